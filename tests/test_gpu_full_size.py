"""Full-size workloads in the launch configuration bench.py times, checked on sampled outputs
the oracle computes one by one, and on properties that hold at any size.

Inputs of every oracle call come from the seeded generators (or from another oracle call);
nothing the CUDA path produced is fed to the oracle.
"""
import numpy as np
import pytest
import torch

from oracle import grpo_oracle as O
from paper_2507_01663_b200 import workloads as wl
from gpu_util import ADV_TOL, GRAD_RTOL, LOGP_TOL, LOSS_RTOL, device, f32, i32, np_of, rel, sample_rows

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2507_01663_b200 import binding as B
    c = B.Context(0)
    yield c
    c.close()


def oracle_rows(H_rows, W_bits, y_rows, chunk=128):
    """Oracle log-prob / entropy / lse of the given rows at the full vocabulary."""
    outs = [O.token_logprob_ref(wl.bf16_bits(H_rows[s:s + chunk]), W_bits, y_rows[s:s + chunk])
            for s in range(0, H_rows.shape[0], chunk)]
    return [np.concatenate([o[k] for o in outs]) for k in range(3)]


def build_store(w, dev):
    H, y = wl.gen_hidden(w, dev), wl.gen_target(w, dev)
    W = wl.gen_weight(w, dev)
    centre = wl.centre_logp_estimate(w, H, W, y)
    old = centre + wl.gen_noise(w, wl.S_OLD, w.total_tokens, dev)
    ref = centre + wl.gen_noise(w, wl.S_REF, w.total_tokens, dev)
    return {"hidden": H, "target": y, "old_logp": old, "ref_logp": ref}, W, wl.gen_reward(w, dev)


def packed_out(T, B, d, dev):
    return {"cu_seqlens": torch.zeros(B + 1, dtype=torch.int32, device=dev),
            "hidden": torch.empty(T, d, dtype=torch.bfloat16, device=dev),
            "target": torch.empty(T, dtype=torch.int32, device=dev),
            "old_logp": torch.empty(T, device=dev), "ref_logp": torch.empty(T, device=dev),
            "adv_seq": torch.empty(B, device=dev), "seq_id": torch.empty(T, dtype=torch.int32, device=dev)}


def check_pack_everywhere(w, store, adv, idx, out, T):
    """Pack is checked on every row by its definition (device-side slicing, bitwise) and through
    the oracle on the scalar columns and on sampled sequences of the hidden column."""
    off = w.tok_offset
    host = {k: np_of(store[k]) for k in ("target", "old_logp", "ref_logp")}
    ref = O.pack_microbatch_ref(off, idx, host, np_of(adv))
    cu = ref["cu_seqlens"].astype(np.int64)
    assert T == int(cu[-1])
    assert np.array_equal(np_of(out["cu_seqlens"])[:len(idx) + 1], ref["cu_seqlens"])
    for k in host:
        assert np_of(out[k][:T]).tobytes() == ref[k].tobytes(), k
    assert np.array_equal(np_of(out["seq_id"][:T]), ref["seq_id"])
    assert np_of(out["adv_seq"][:len(idx)]).tobytes() == ref["adv_seq"].astype(np.float32).tobytes()
    Hs, Hp = store["hidden"].view(torch.int16), out["hidden"].view(torch.int16)
    for j, i in enumerate(idx):
        assert torch.equal(Hp[cu[j]:cu[j + 1]], Hs[off[i]:off[i + 1]]), j
    lens = np.diff(cu)
    for j in {0, len(idx) - 1, int(np.argmax(lens)), int(np.argmin(lens))}:
        i = int(idx[j])
        sub = O.pack_microbatch_ref(np.array([0, off[i + 1] - off[i]]), [0],
                                    {"hidden": wl.bf16_bits(store["hidden"][off[i]:off[i + 1]])})
        assert np.array_equal(wl.bf16_bits(out["hidden"][cu[j]:cu[j + 1]]), sub["hidden"])
    return cu


def scored_chain_check(ctx, w, store, W, reward, idx, n_rows, seed, agg_mode=0):
    """advantage -> pack -> log-prob -> loss on one micro-batch; sampled rows against the oracle."""
    from paper_2507_01663_b200 import binding as B
    dev = device()
    adv = torch.empty(w.N, device=dev)
    ctx.grpo_advantage(reward, None, w.n_prompts, adv)
    adv_ref = O.grpo_advantage_ref(np_of(reward), w.group_id, w.n_prompts)
    assert np.abs(np_of(adv) - adv_ref).max() <= ADV_TOL
    T_cap = int(w.lengths[idx].sum())
    out = packed_out(T_cap, len(idx), w.d, dev)
    T = ctx.pack_microbatch({"tok_offset_host": w.tok_offset, "d": w.d, "adv": adv, **store}, idx, out)
    cu = check_pack_everywhere(w, store, adv, idx, out, T)
    logp, ent, lse, g = (torch.empty(T, device=dev) for _ in range(4))
    ctx.token_logprob(out["hidden"], W, out["target"], logp, ent, lse)
    lo = B.new_loss_out(dev)
    ctx.policy_loss(logp, out["old_logp"], out["ref_logp"], out["adv_seq"], out["cu_seqlens"], lo, g, ent,
                    w.clip_eps, w.clip_eps, w.kl_coef, agg_mode, 1.0)
    res = B.read_loss_out(lo)
    assert ctx.check_device_errors() == 0
    # sampled rows: regenerate nothing, read the very bits the kernel saw
    rows = sample_rows(cu, T, n_rows, seed)
    rt = torch.as_tensor(rows, device=dev)
    W_bits = wl.bf16_bits(W)
    seq_of = np.searchsorted(cu, rows, side="right") - 1
    src_rows = w.tok_offset[idx[seq_of]] + (rows - cu[seq_of])          # store rows, by the definition of pack
    src_t = torch.as_tensor(src_rows, device=dev)
    o_logp, o_ent, o_lse = oracle_rows(store["hidden"][src_t].cpu(), W_bits, np_of(store["target"][src_t]))
    assert np.abs(np_of(logp[rt]) - o_logp).max() <= LOGP_TOL
    assert np.abs(np_of(ent[rt]) - o_ent).max() <= LOGP_TOL
    assert np.abs(np_of(lse[rt]) - o_lse).max() <= LOGP_TOL
    # per-token gradient of the loss at the sampled rows, from oracle quantities only
    A = adv_ref[idx[seq_of]]
    L = np.diff(cu)[seq_of].astype(np.float64)
    wt = 1.0 / (len(idx) * L) if agg_mode == 0 else np.full(len(rows), 1.0 / T)
    old, ref = np_of(store["old_logp"][src_t]).astype(np.float64), np_of(store["ref_logp"][src_t]).astype(np.float64)
    rho = np.exp(o_logp - old)
    s1, s2 = rho * A, np.clip(rho, 1 - w.clip_eps, 1 + w.clip_eps) * A
    g_ref = wt * (np.where(s2 < s1, 0.0, -A * rho) + w.kl_coef * (1.0 - np.exp(ref - o_logp)))
    near = (np.abs(rho - (1 - w.clip_eps)) < 2 * LOGP_TOL) | (np.abs(rho - (1 + w.clip_eps)) < 2 * LOGP_TOL)
    err = np.abs(np_of(g[rt]) - g_ref)[~near]
    assert err.max() <= 5e-3 * np.abs(g_ref).max() + 1e-12
    # properties at full size: finite outputs, entropy range, loss aggregates its own tokens
    lp = np_of(logp)
    assert np.isfinite(lp).all() and (lp <= 1e-5).all()
    e = np_of(ent)
    assert (e >= -1e-4).all() and (e <= np.log(w.V) + 1e-4).all()
    assert rel(res["entropy_mean"], float(e.astype(np.float64).mean())) <= 1e-5
    assert res["n_tokens"] == T and np.isfinite(res["loss"])
    return res


@pytest.mark.parametrize("name,n_rows", [("cfg2", 192), ("cfg3", 128)])
def test_forward_workloads_full_size(ctx, name, n_rows):
    w = wl.make_workload(name)
    dev = device()
    store, W, reward = build_store(w, dev)
    scored_chain_check(ctx, w, store, W, reward, wl.arrival_order(w), n_rows, seed=w.seed)


def test_streaming_store_full_size(ctx):
    """cfg5: arrival-ordered micro-batches with a 32768-token budget, packed, scored and
    loss-reduced back to back on one stream; first, a middle and the last batch are checked."""
    from paper_2507_01663_b200 import binding as B
    w = wl.make_workload("cfg5")
    dev = device()
    store, W, reward = build_store(w, dev)
    mbs = wl.microbatches(w)
    assert all(int(w.lengths[m].sum()) <= w.token_budget or len(m) == 1 for m in mbs)
    for k in (0, len(mbs) // 2, len(mbs) - 1):
        scored_chain_check(ctx, w, store, W, reward, mbs[k], 48, seed=k)
    # back-to-back on one stream with shared buffers: every batch ends with finite, sane scalars
    adv = torch.empty(w.N, device=dev)
    ctx.grpo_advantage(reward, None, w.n_prompts, adv)
    cap = max(int(w.lengths[m].sum()) for m in mbs)
    out = packed_out(cap, max(len(m) for m in mbs), w.d, dev)
    logp, ent, lse, g = (torch.empty(cap, device=dev) for _ in range(4))
    louts = [B.new_loss_out(dev) for _ in mbs]
    total = 0
    for m, lo in zip(mbs, louts):
        T = ctx.pack_microbatch({"tok_offset_host": w.tok_offset, "d": w.d, "adv": adv, **store}, m, out)
        ctx.token_logprob(out["hidden"], W, out["target"], logp, ent, lse, T=T)
        ctx.policy_loss(logp, out["old_logp"], out["ref_logp"], out["adv_seq"], out["cu_seqlens"], lo, g, ent,
                        w.clip_eps, w.clip_eps, w.kl_coef, B=len(m), T=T)
        total += T
    assert ctx.check_device_errors() == 0 and total == w.total_tokens
    for m, lo in zip(mbs, louts):
        r = B.read_loss_out(lo)
        assert r["n_tokens"] == int(w.lengths[m].sum()) and np.isfinite(r["loss"]) and 0 <= r["clip_frac"] <= 1


def test_loss_stage_full_size(ctx):
    """The loss kernel alone at 1.1 M tokens against the oracle, on generator-made inputs."""
    from paper_2507_01663_b200 import binding as B
    w = wl.make_workload("cfg2")
    dev = device()
    T = w.total_tokens
    idx = wl.arrival_order(w)
    cu = np.concatenate([[0], np.cumsum(w.lengths[idx])])
    logp = wl.gen_surrogate_logp(w, T)
    old = logp + wl.gen_noise(w, wl.S_OLD, T)
    ref = logp + wl.gen_noise(w, wl.S_REF, T)
    ent = torch.abs(wl.normal01(w.seed, wl.S_MISC, 0, T)) + 5.0
    adv = O.grpo_advantage_ref(np_of(wl.gen_reward(w)), w.group_id, w.n_prompts)[idx].astype(np.float32)
    for agg_mode in (0, 1):
        lo = B.new_loss_out(dev)
        g = torch.empty(T, device=dev)
        ctx.policy_loss(logp.to(dev), old.to(dev), ref.to(dev), f32(adv), i32(cu), lo, g, ent.to(dev),
                        w.clip_eps, w.clip_eps, w.kl_coef, agg_mode, 1.0)
        res = B.read_loss_out(lo)
        oref = O.policy_loss_ref(logp.numpy(), old.numpy(), ref.numpy(), adv, cu, w.clip_eps, w.clip_eps, w.kl_coef,
                                 agg_mode, 1.0, entropy=ent.numpy())
        for k in ("loss", "pg_loss", "kl_mean", "entropy_mean"):
            assert rel(res[k], oref[k]) <= LOSS_RTOL, (k, res[k], oref[k])
        near = (np.abs(oref["rho"] - 0.8) < 1e-5) | (np.abs(oref["rho"] - 1.2) < 1e-5)
        assert abs(res["clip_frac"] - oref["clip_frac"]) <= (near.sum() + 0.5) / T
        assert np.abs(np_of(g) - oref["dlogp"])[~near].max() <= 1e-5 * np.abs(oref["dlogp"]).max()
    assert ctx.check_device_errors() == 0


def test_backward_full_size(ctx):
    """cfg4: one 65536-token micro-batch, d = 3584, V = 152064.  dH on sampled rows and dW on
    sampled vocabulary rows against the oracle; column sums and the <dW,W> = <dH,H> identity
    over the whole result.  The stage's lse input is synthetic (the oracle uses the same)."""
    w = wl.make_workload("cfg4")
    dev = device()
    T = w.total_tokens
    H, y, W = wl.gen_hidden(w, dev), wl.gen_target(w, dev), wl.gen_weight(w, dev)
    # lse: the Gaussian estimate of a random head's normaliser, jittered; g ~ N(0, 1/T^2)
    hh = (H.float() ** 2).sum(1)
    lse = (np.log(w.V) + 0.5 * w.w_std ** 2 * hh + 0.05 * wl.normal01(w.seed, wl.S_MISC, 0, T, dev)).contiguous()
    g = (wl.normal01(w.seed, wl.S_G, 0, T, dev) / T).contiguous()
    dH = torch.empty(T, w.d, dtype=torch.bfloat16, device=dev)
    dW = torch.empty(w.V, w.d, device=dev)
    ctx.policy_loss_backward(H, W, y, lse, g, dH, dW)
    assert ctx.check_device_errors() == 0
    W_bits = wl.bf16_bits(W)
    cu = w.tok_offset
    rows = sample_rows(cu, T, 96, seed=1)
    rt = torch.as_tensor(rows, device=dev)
    dH_ref = np.concatenate([
        O.policy_loss_backward_ref(wl.bf16_bits(H[rt[s:s + 32]]), W_bits, np_of(y[rt[s:s + 32]]),
                                   np_of(lse[rt[s:s + 32]]), np_of(g[rt[s:s + 32]]))[0]
        for s in range(0, len(rows), 32)])
    got = np_of(dH[rt].float())
    nH = np.linalg.norm(dH_ref)
    assert abs(np.linalg.norm(got) - nH) <= GRAD_RTOL * nH
    assert np.linalg.norm(got - dH_ref) <= GRAD_RTOL * nH
    # dW rows: ids that occur as targets, tile edges, the last row
    ys = np_of(y)
    vs = sorted({0, 127, 128, 255, 256, w.V - 1, w.V - 129, int(ys[0]), int(ys[T // 2]), int(ys[-1])}
                | set(np.random.default_rng(2).integers(0, w.V, 54).tolist()))
    dW_ref = O.policy_loss_backward_ref(wl.bf16_bits(H), W_bits, ys, np_of(lse), np_of(g), vocab_rows=vs)
    gotW = np_of(dW[torch.as_tensor(vs, device=dev)])
    nW = np.linalg.norm(dW_ref)
    assert abs(np.linalg.norm(gotW) - nW) <= GRAD_RTOL * nW
    assert np.linalg.norm(gotW - dW_ref) <= GRAD_RTOL * nW
    # whole-result properties.  sum_v dZ_tv = g_t (1 - sum_v p_tv): with the synthetic lse the
    # "probabilities" do not sum to one, so the column-sum identity reads sum_v dW[v] = c^T H
    # with c_t = g_t (1 - S_t); S_t comes from the oracle on the sampled rows only, so check the
    # trace identity instead, which needs no S: <dW, W> - <dH, H> = 0 up to bf16 rounding
    lhs = float((dW.double() * W.double()).sum())
    rhs = float((dH.double() * H.double()).sum())
    scale = float(dW.double().norm() * W.double().norm())
    assert abs(lhs - rhs) <= 2e-3 * scale


def test_vocabulary_parallel_head_full_size(ctx):
    """The 7B head split over two ranks' worth of vocabulary rows at 65536 tokens (the shards are
    scored one after the other on this GPU): merged result against the unsharded call on every
    token, and against the oracle on sampled rows."""
    w = wl.make_workload("cfg4")
    dev = device()
    T = w.total_tokens
    H, y, W = wl.gen_hidden(w, dev), wl.gen_target(w, dev), wl.gen_weight(w, dev)
    cuts = [0, 76032, w.V]
    partials = torch.empty(2, T, 4, device=dev)
    for r in range(2):
        ctx.token_logprob_shard(H, W[cuts[r]:cuts[r + 1]], y, cuts[r], partials[r])
    logp, ent, lse = (torch.empty(T, device=dev) for _ in range(3))
    ctx.merge_logprob_shards(partials, y, w.V, logp, ent, lse)
    one = [torch.empty(T, device=dev) for _ in range(3)]
    ctx.token_logprob(H, W, y, *one)
    assert ctx.check_device_errors() == 0
    for got, ref in zip((logp, ent, lse), one):
        assert float((got - ref).abs().max()) <= 1e-4
    # exactly one shard holds every token's target
    assert bool((torch.isfinite(partials[:, :, 3]).sum(0) == 1).all())
    rows = sample_rows(w.tok_offset, T, 64, seed=5)
    rt = torch.as_tensor(rows, device=dev)
    o_logp, o_ent, o_lse = oracle_rows(H[rt].cpu(), wl.bf16_bits(W), np_of(y[rt]))
    assert np.abs(np_of(logp[rt]) - o_logp).max() <= LOGP_TOL
    assert np.abs(np_of(ent[rt]) - o_ent).max() <= LOGP_TOL
    assert np.abs(np_of(lse[rt]) - o_lse).max() <= LOGP_TOL


def test_fused_update_full_size(ctx):
    """cfg4 through af_policy_update against the same micro-batch through the three separate
    calls (which the tests above tie to the oracle): log-probs, loss record and dlogp agree to
    fp32 rounding, the gradients within the bf16 rounding of dZ."""
    from paper_2507_01663_b200 import binding as B
    w = wl.make_workload("cfg4")
    dev = device()
    T = w.total_tokens
    store, W, reward = build_store(w, dev)
    H, y, old, ref = store["hidden"], store["target"], store["old_logp"], store["ref_logp"]
    adv = torch.empty(w.N, device=dev)
    ctx.grpo_advantage(reward, None, w.n_prompts, adv)
    cu = torch.as_tensor(w.tok_offset.astype(np.int32), device=dev)
    # three calls
    logp, ent, lse, g = (torch.empty(T, device=dev) for _ in range(4))
    lo = B.new_loss_out(dev)
    ctx.token_logprob(H, W, y, logp, ent, lse)
    ctx.policy_loss(logp, old, ref, adv, cu, lo, g, ent, w.clip_eps, w.clip_eps, w.kl_coef)
    dH = torch.empty(T, w.d, dtype=torch.bfloat16, device=dev)
    dW = torch.empty(w.V, w.d, device=dev)
    ctx.policy_loss_backward(H, W, y, lse, g, dH, dW)
    res = B.read_loss_out(lo)
    # one call
    logp2, ent2, lse2, g2 = (torch.empty(T, device=dev) for _ in range(4))
    lo2 = B.new_loss_out(dev)
    dH2 = torch.empty_like(dH)
    dW2 = torch.empty_like(dW)
    ctx.policy_update(H, W, y, old, ref, adv, cu, lo2, logp2, lse2, dH2, dW2, entropy=ent2, dlogp=g2,
                      clip_lo=w.clip_eps, clip_hi=w.clip_eps, kl_coef=w.kl_coef)
    res2 = B.read_loss_out(lo2)
    assert ctx.check_device_errors() == 0
    assert float((logp2 - logp).abs().max()) <= 1e-4 and float((lse2 - lse).abs().max()) <= 1e-4
    assert float((ent2 - ent).abs().max()) <= 1e-4
    for k in ("loss", "pg_loss", "kl_mean", "entropy_mean"):
        assert rel(res2[k], res[k]) <= 1e-4, k
    assert res2["n_tokens"] == T
    assert float((g2 - g).abs().max()) <= 1e-3 * float(g.abs().max())
    assert float((dW2 - dW).norm() / dW.norm()) <= 2e-3
    assert float((dH2.float() - dH.float()).norm() / dH.float().norm()) <= 2e-3
    # trace identity over the whole fused result: <dW, W> = <dH, H> up to bf16 rounding
    lhs = float((dW2.double() * W.double()).sum())
    rhs = float((dH2.double() * H.double()).sum())
    assert abs(lhs - rhs) <= 2e-3 * float(dW2.double().norm() * W.double().norm())
