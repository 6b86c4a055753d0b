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
from gpu_util import (ADV_TOL, GRAD_RTOL, LOGP_TOL, LOSS_RTOL, device, f32, i32, np_of, off_the_clip_bounds, rel,
                      sample_rows)

N_ROWS = 2048        # token rows scored by the oracle per full-size batch (every row over the full vocabulary)
N_ROWS_MB = 256      # the same per micro-batch of the streaming store
N_VOCAB_ROWS = 256   # rows of dW formed by the oracle (each a sum over every token of the batch)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2507_01663_b200 import binding as B
    c = B.Context(0)
    yield c
    c.close()


def oracle_rows(H_rows, W_bits, y_rows, chunk=512):
    """Oracle log-prob / entropy / lse of the given rows at the full vocabulary (in chunks of rows:
    every call of the oracle widens the whole weight matrix to fp64 first)."""
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


def vocab_rows_sample(V, targets, n, seed):
    """Vocabulary ids for sampled rows of dW: ids that occur as targets, both sides of the 128- and
    256-row tile edges at either end of the vocabulary, the last row, then seeded random ids."""
    last256 = (V - 1) // 256 * 256
    vs = {0, 127, 128, 255, 256, 257, last256 - 1, last256, last256 + 127, last256 + 128, V - 2, V - 1}
    vs = {min(max(int(v), 0), V - 1) for v in vs}
    vs.update(int(t) for t in targets)
    rng = np.random.default_rng(seed)
    while len(vs) < n:
        vs.add(int(rng.integers(0, V)))
    return sorted(vs)


def token_gradient_ref(o_logp, old, ref, A, wt, clip_eps, kl_coef):
    """dL/dlogp of the given tokens from oracle quantities only, through the oracle's loss: every
    token becomes a sequence of its own (length 1) in token-mean mode, where the oracle's weight is
    1/n; the token's real weight `wt` (from the batch it sits in) replaces it."""
    n = len(o_logp)
    r = O.policy_loss_ref(o_logp, old, ref, A, np.arange(n + 1), clip_eps, clip_eps, kl_coef, agg_mode=1, loss_scale=1.0)
    return r["dlogp"] * n * wt, r


def scored_chain_check(ctx, w, store, W, reward, idx, n_rows, seed, agg_mode=0):
    """advantage -> pack -> log-prob -> loss on one micro-batch; sampled rows against the oracle.
    At the sampled rows the store's old / ref log-probs are, as the workload defines them, the
    oracle's log-prob plus noise (moved off the clip bounds); elsewhere they are centred on the
    estimate of the generator module."""
    from paper_2507_01663_b200 import binding as B
    dev = device()
    idx = np.asarray(idx)
    cu = np.concatenate([[0], np.cumsum(w.lengths[idx])]).astype(np.int64)
    T_host = int(cu[-1])
    rows = sample_rows(cu, T_host, n_rows, seed)
    rt = torch.as_tensor(rows, device=dev)
    seq_of = np.searchsorted(cu, rows, side="right") - 1
    src_rows = w.tok_offset[idx[seq_of]] + (rows - cu[seq_of])          # store rows, by the definition of pack
    src_t = torch.as_tensor(src_rows, device=dev)
    W_bits = wl.bf16_bits(W)
    # the oracle reads the very bits the kernel will see
    o_logp, o_ent, o_lse = oracle_rows(store["hidden"][src_t].cpu(), W_bits, np_of(store["target"][src_t]))
    n_old = np_of(wl.gen_noise(w, wl.S_OLD, w.total_tokens, dev)[src_t]).astype(np.float64)
    n_ref = np_of(wl.gen_noise(w, wl.S_REF, w.total_tokens, dev)[src_t]).astype(np.float64)
    old = off_the_clip_bounds(o_logp, (o_logp + n_old).astype(np.float32), w.clip_eps, w.clip_eps)
    ref = (o_logp + n_ref).astype(np.float32).astype(np.float64)
    store["old_logp"][src_t] = f32(old)
    store["ref_logp"][src_t] = f32(ref)

    adv = torch.empty(w.N, device=dev)
    ctx.grpo_advantage(reward, None, w.n_prompts, adv)
    adv_ref = O.grpo_advantage_ref(np_of(reward), w.group_id, w.n_prompts)
    assert np.abs(np_of(adv) - adv_ref).max() <= ADV_TOL
    out = packed_out(T_host, len(idx), w.d, dev)
    T = ctx.pack_microbatch({"tok_offset_host": w.tok_offset, "d": w.d, "adv": adv, **store}, idx, out)
    assert np.array_equal(check_pack_everywhere(w, store, adv, idx, out, T), cu)
    logp, ent, lse, g = (torch.empty(T, device=dev) for _ in range(4))
    ctx.token_logprob(out["hidden"], W, out["target"], logp, ent, lse)
    lo = B.new_loss_out(dev)
    ctx.policy_loss(logp, out["old_logp"], out["ref_logp"], out["adv_seq"], out["cu_seqlens"], lo, g, ent,
                    w.clip_eps, w.clip_eps, w.kl_coef, agg_mode, 1.0)
    res = B.read_loss_out(lo)
    assert ctx.check_device_errors() == 0
    assert np.abs(np_of(logp[rt]) - o_logp).max() <= LOGP_TOL
    assert np.abs(np_of(ent[rt]) - o_ent).max() <= LOGP_TOL
    assert np.abs(np_of(lse[rt]) - o_lse).max() <= LOGP_TOL
    # per-token gradient of the loss at the sampled rows, from oracle quantities only
    A = adv_ref[idx[seq_of]]
    L = np.diff(cu)[seq_of].astype(np.float64)
    wt = 1.0 / (len(idx) * L) if agg_mode == 0 else np.full(len(rows), 1.0 / T)
    g_ref, _ = token_gradient_ref(o_logp, old, ref, A, wt, w.clip_eps, w.kl_coef)
    assert np.abs(np_of(g[rt]) - g_ref).max() <= 5e-3 * np.abs(g_ref).max() + 1e-12
    # properties at full size: finite outputs, entropy range, loss aggregates its own tokens
    lp = np_of(logp)
    assert np.isfinite(lp).all() and (lp <= 1e-5).all()
    e = np_of(ent)
    assert (e >= -1e-4).all() and (e <= np.log(w.V) + 1e-4).all()
    assert rel(res["entropy_mean"], float(e.astype(np.float64).mean())) <= 1e-5
    assert res["n_tokens"] == T and np.isfinite(res["loss"])
    return res


@pytest.mark.parametrize("name", ["cfg2", "cfg3"])
def test_forward_workloads_full_size(ctx, name):
    w = wl.make_workload(name)
    dev = device()
    store, W, reward = build_store(w, dev)
    scored_chain_check(ctx, w, store, W, reward, wl.arrival_order(w), N_ROWS, seed=w.seed)


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
        scored_chain_check(ctx, w, store, W, reward, mbs[k], N_ROWS_MB, seed=k)
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


def test_closed_streaming_loop_full_size():
    """cfg5 through the benchmark's two-task loop (controller get -> pack -> log-prob -> write-back with
    status bits; get on those bits -> pack -> log-prob -> loss; weight swap at an iteration boundary):
    the column actor inference wrote back against the oracle on sampled store rows, every sample
    served once per task, every loss record finite with nothing clipped."""
    import bench
    w = wl.make_workload("cfg5")
    dev = device()
    job = bench.ScoringJob(w, dev)
    try:
        job.make_closed_loop()
        scored = job.step_closed_loop(refresh_weights=True)
        torch.cuda.synchronize()
        assert scored == 2 * w.total_tokens and job.ctx.check_device_errors() == 0 and job.w_swaps == 1
        col = job.cl_old_col
        assert bool(torch.isfinite(col).all())
        rows = sample_rows(w.tok_offset, w.total_tokens, N_ROWS_MB, seed=11)
        rt = torch.as_tensor(rows, device=dev)
        o_logp, _, _ = oracle_rows(job.store["hidden"][rt].cpu(), wl.bf16_bits(job.W), np_of(job.store["target"][rt]))
        assert np.abs(np_of(col[rt]) - o_logp).max() <= LOGP_TOL
        both = job.COL_RESPONSE | job.COL_OLD_LOGP
        assert bool((job.cl_tab["ready"] == both).all())
        assert bool((job.cl_tab["consumed"] == (job.TASK_INFER | job.TASK_UPDATE)).all())
        for task in (job.TASK_INFER, job.TASK_UPDATE):
            seen = np.concatenate([mb for t, mb in job.cl_history if t == task])
            assert np.array_equal(np.sort(seen), np.arange(w.N))
        for _, mb in job.cl_history:
            assert int(w.lengths[mb].sum()) <= w.token_budget or len(mb) == 1
        records = [job.B.read_loss_out(lo) for lo in job.cl_loss_outs[:job.cl_loss_count]]
        assert sum(r["n_tokens"] for r in records) == w.total_tokens
        assert all(np.isfinite(r["loss"]) and r["clip_frac"] == 0.0 for r in records)
    finally:
        job.ctx.close()


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


def dH_rows_ref(H_rows, W_bits, y_rows, lse_rows, g_rows, chunk=256):
    """Oracle dH of the given token rows (each row needs the whole vocabulary, nothing else)."""
    return np.concatenate([
        O.policy_loss_backward_ref(wl.bf16_bits(H_rows[s:s + chunk]), W_bits, y_rows[s:s + chunk],
                                   lse_rows[s:s + chunk], g_rows[s:s + chunk])[0]
        for s in range(0, H_rows.shape[0], chunk)])


def assert_grad_close(got, ref, what):
    n = np.linalg.norm(ref)
    assert abs(np.linalg.norm(got) - n) <= GRAD_RTOL * n, what          # gradient norm (the stated bar)
    assert np.linalg.norm(got - ref) <= GRAD_RTOL * n, what            # and the direction, element-wise


def test_backward_full_size(ctx):
    """cfg4: one 65536-token micro-batch, d = 3584, V = 152064.  dH on sampled rows and dW on
    sampled vocabulary rows against the oracle; the <dW,W> = <dH,H> identity over the whole result.
    The stage's lse input is synthetic (the oracle uses the same)."""
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
    rows = sample_rows(w.tok_offset, T, N_ROWS, seed=1)
    rt = torch.as_tensor(rows, device=dev)
    dH_ref = dH_rows_ref(H[rt].cpu(), W_bits, np_of(y[rt]), np_of(lse[rt]), np_of(g[rt]))
    assert_grad_close(np_of(dH[rt].float()), dH_ref, "dH")
    # dW rows: ids that occur as targets, tile edges, the last row
    ys = np_of(y)
    vs = vocab_rows_sample(w.V, ys[[0, T // 2, T - 1, 255, 256]], N_VOCAB_ROWS, seed=2)
    dW_ref = O.policy_loss_backward_ref(wl.bf16_bits(H), W_bits, ys, np_of(lse), np_of(g), vocab_rows=vs)
    assert_grad_close(np_of(dW[torch.as_tensor(vs, device=dev)]), dW_ref, "dW")
    # whole-result property.  With a synthetic lse the "probabilities" do not sum to one, so the
    # column sums of dZ are not zero; the trace identity needs no such assumption:
    # <dW, W> - <dH, H> = 0 up to bf16 rounding
    lhs = float((dW.double() * W.double()).sum())
    rhs = float((dH.double() * H.double()).sum())
    scale = float(dW.double().norm() * W.double().norm())
    assert abs(lhs - rhs) <= 2e-3 * scale


def test_vocabulary_parallel_head_full_size(ctx):
    """The 7B head split over two ranks' worth of vocabulary rows at 65536 tokens (the shards are
    scored one after the other on this GPU): merged result against the oracle on sampled rows, and
    against the unsharded call on every token."""
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
    rows = sample_rows(w.tok_offset, T, N_ROWS_MB, seed=5)
    rt = torch.as_tensor(rows, device=dev)
    o_logp, o_ent, o_lse = oracle_rows(H[rt].cpu(), wl.bf16_bits(W), np_of(y[rt]))
    assert np.abs(np_of(logp[rt]) - o_logp).max() <= LOGP_TOL
    assert np.abs(np_of(ent[rt]) - o_ent).max() <= LOGP_TOL
    assert np.abs(np_of(lse[rt]) - o_lse).max() <= LOGP_TOL
    # the two CUDA paths sum the vocabulary in different groupings (fp32, approximate exp2): a loose
    # consistency check beside the oracle comparison above
    for got, ref in zip((logp, ent, lse), one):
        assert float((got - ref).abs().max()) <= 3e-4
    # exactly one shard holds every token's target
    assert bool((torch.isfinite(partials[:, :, 3]).sum(0) == 1).all())


# ------------------------------------------------------------------------------------------
# the actor update as a chain at full size: log-prob -> loss -> backward, three calls or one
# ------------------------------------------------------------------------------------------
_ORACLE_CACHE = {}      # oracle results of a chain workload (generator inputs only), shared by both modes


def run_actor_update(ctx, mode, w, H, W, y, old, ref, reward, kl_coef):
    """The cfg4-shaped micro-batch (samples in index order) through the three calls or the fused one."""
    from paper_2507_01663_b200 import binding as B
    dev = device()
    T = w.total_tokens
    adv = torch.empty(w.N, device=dev)
    ctx.grpo_advantage(reward, None, w.n_prompts, adv)
    cu = torch.as_tensor(w.tok_offset.astype(np.int32), device=dev)
    logp, ent, lse, g = (torch.empty(T, device=dev) for _ in range(4))
    lo = B.new_loss_out(dev)
    dH = torch.empty(T, w.d, dtype=torch.bfloat16, device=dev)
    dW = torch.empty(w.V, w.d, device=dev)
    if mode == "three_calls":
        ctx.token_logprob(H, W, y, logp, ent, lse)
        ctx.policy_loss(logp, old, ref, adv, cu, lo, g, ent, w.clip_eps, w.clip_eps, kl_coef)
        ctx.policy_loss_backward(H, W, y, lse, g, dH, dW)       # the forward's own lse
    else:
        ctx.policy_update(H, W, y, old, ref, adv, cu, lo, logp, lse, dH, dW, entropy=ent, dlogp=g,
                          clip_lo=w.clip_eps, clip_hi=w.clip_eps, kl_coef=kl_coef)
    res = B.read_loss_out(lo)
    assert ctx.check_device_errors() == 0
    return res, adv, logp, ent, lse, g, dH, dW


@pytest.mark.parametrize("mode", ["three_calls", "fused"])
def test_actor_update_chain_full_size(ctx, mode):
    """cfg4 as stated (Bernoulli(0.5) rewards, eps 0.2, KL coefficient 0.04): on 2048 sampled rows
    the log-prob, entropy, lse, dL/dlogp and dH of the CUDA chain against the oracle chain
    advantage -> log-prob -> loss -> backward, whose inputs are the generators' alone."""
    w = wl.make_workload("cfg4")
    dev = device()
    T = w.total_tokens
    H, y, W = wl.gen_hidden(w, dev), wl.gen_target(w, dev), wl.gen_weight(w, dev)
    reward = wl.gen_reward(w, dev)
    cu = w.tok_offset
    rows = sample_rows(cu, T, N_ROWS, seed=7)
    rt = torch.as_tensor(rows, device=dev)
    if "cfg4" not in _ORACLE_CACHE:
        W_bits = wl.bf16_bits(W)
        o = oracle_rows(H[rt].cpu(), W_bits, np_of(y[rt]))
        adv_ref = O.grpo_advantage_ref(np_of(reward), w.group_id, w.n_prompts)
        n_old = np_of(wl.gen_noise(w, wl.S_OLD, T, dev)[rt]).astype(np.float64)
        n_ref = np_of(wl.gen_noise(w, wl.S_REF, T, dev)[rt]).astype(np.float64)
        old_r = off_the_clip_bounds(o[0], (o[0] + n_old).astype(np.float32), w.clip_eps, w.clip_eps)
        ref_r = (o[0] + n_ref).astype(np.float32).astype(np.float64)
        seq_of = np.searchsorted(cu, rows, side="right") - 1
        wt = 1.0 / (w.N * np.diff(cu)[seq_of].astype(np.float64))
        g_ref, _ = token_gradient_ref(o[0], old_r, ref_r, adv_ref[seq_of], wt, w.clip_eps, w.kl_coef)
        dH_ref = dH_rows_ref(H[rt].cpu(), W_bits, np_of(y[rt]), o[2], g_ref)
        _ORACLE_CACHE["cfg4"] = (o, adv_ref, old_r, ref_r, g_ref, dH_ref)
    (o_logp, o_ent, o_lse), adv_ref, old_r, ref_r, g_ref, dH_ref = _ORACLE_CACHE["cfg4"]
    # store columns: centred on the generator module's estimate, the oracle's log-prob + noise at the sampled rows
    centre = wl.centre_logp_estimate(w, H, W, y)
    old = centre + wl.gen_noise(w, wl.S_OLD, T, dev)
    ref = centre + wl.gen_noise(w, wl.S_REF, T, dev)
    old[rt], ref[rt] = f32(old_r), f32(ref_r)
    res, adv, logp, ent, lse, g, dH, dW = run_actor_update(ctx, mode, w, H, W, y, old, ref, reward, w.kl_coef)
    assert np.abs(np_of(adv) - adv_ref).max() <= ADV_TOL
    assert np.abs(np_of(logp[rt]) - o_logp).max() <= LOGP_TOL
    assert np.abs(np_of(ent[rt]) - o_ent).max() <= LOGP_TOL
    assert np.abs(np_of(lse[rt]) - o_lse).max() <= LOGP_TOL
    assert np.abs(np_of(g[rt]) - g_ref).max() <= 5e-3 * np.abs(g_ref).max()
    assert_grad_close(np_of(dH[rt].float()), dH_ref, "dH")
    # whole-result properties: the record counts its tokens, sum_v dW[v,:] = 0 (softmax rows sum to
    # one when lse is the forward's own) and <dW, W> = <dH, H>, both up to the bf16 rounding of dZ
    assert res["n_tokens"] == T and np.isfinite(res["loss"]) and 0.0 <= res["clip_frac"] <= 1.0
    col = dW.double().sum(0)
    assert float(col.abs().max()) <= 2e-2 * float(dW.double().abs().sum(0).max())
    lhs = float((dW.double() * W.double()).sum())
    rhs = float((dH.double() * H.double()).sum())
    assert abs(lhs - rhs) <= 2e-3 * float(dW.double().norm() * W.double().norm())


@pytest.mark.parametrize("mode", ["three_calls", "fused"])
def test_actor_update_chain_sparse_advantages_full_size(ctx, mode):
    """dW -- every row of it a sum over all 65536 tokens -- against the oracle chain at the full
    cfg4 shape.  The oracle cannot score 65536 tokens over 152064 logits in test time, so the batch
    is made to need only some of them: all groups but two get equal rewards (the degenerate case of
    the group normalisation: zero advantages) and the KL coefficient is 0, so that tokens outside
    the two live groups have dL/dlogp = 0 exactly and drop out of dW, dH and the loss.  The oracle
    scores the live tokens (about an eighth of the batch); the CUDA path runs the whole batch in
    the launch configuration of the benchmark."""
    w = wl.make_workload("cfg4")
    dev = device()
    T, G = w.total_tokens, w.group_size
    H, y, W = wl.gen_hidden(w, dev), wl.gen_target(w, dev), wl.gen_weight(w, dev)
    r = np_of(wl.gen_reward(w)).copy()
    mixed = [p for p in range(w.n_prompts) if 0 < r[p * G:(p + 1) * G].sum() < G]
    live_groups = [mixed[0], mixed[-1]]
    for p in range(w.n_prompts):
        if p not in live_groups:
            r[p * G:(p + 1) * G] = r[p * G]
    reward = f32(r)
    cu = w.tok_offset
    live_samples = np.concatenate([np.arange(p * G, (p + 1) * G) for p in live_groups])
    live_tok = np.concatenate([np.arange(cu[i], cu[i + 1]) for i in live_samples])
    lt = torch.as_tensor(live_tok, device=dev)
    ys = np_of(y)
    vs = vocab_rows_sample(w.V, ys[live_tok[[0, len(live_tok) // 2, -1]]], N_VOCAB_ROWS, seed=8)
    if "sparse" not in _ORACLE_CACHE:
        W_bits = wl.bf16_bits(W)
        H_live = H[lt].cpu()
        o = oracle_rows(H_live, W_bits, ys[live_tok])
        adv_ref = O.grpo_advantage_ref(r, w.group_id, w.n_prompts)
        assert np.count_nonzero(adv_ref) == len(live_samples)
        n_old = np_of(wl.gen_noise(w, wl.S_OLD, T, dev)[lt]).astype(np.float64)
        old_l = off_the_clip_bounds(o[0], (o[0] + n_old).astype(np.float32), w.clip_eps, w.clip_eps)
        # the live responses as a batch of their own, each weighing 1/N as in the whole batch
        cu_live = np.concatenate([[0], np.cumsum(w.lengths[live_samples])])
        lref = O.policy_loss_ref(o[0], old_l, o[0], adv_ref[live_samples], cu_live, w.clip_eps, w.clip_eps, 0.0,
                                 0, len(live_samples) / w.N)
        dW_ref = O.policy_loss_backward_ref(wl.bf16_bits(H_live), W_bits, ys[live_tok], o[2], lref["dlogp"], vocab_rows=vs)
        pick = sample_rows(cu_live, len(live_tok), 512, seed=9)
        dH_ref = dH_rows_ref(H_live[pick], W_bits, ys[live_tok[pick]], o[2][pick], lref["dlogp"][pick])
        _ORACLE_CACHE["sparse"] = (o, adv_ref, old_l, lref, dW_ref, pick, dH_ref)
    (o_logp, o_ent, o_lse), adv_ref, old_l, lref, dW_ref, pick, dH_ref = _ORACLE_CACHE["sparse"]
    centre = wl.centre_logp_estimate(w, H, W, y)
    old = centre + wl.gen_noise(w, wl.S_OLD, T, dev)
    ref = centre + wl.gen_noise(w, wl.S_REF, T, dev)
    old[lt] = f32(old_l)
    res, adv, logp, ent, lse, g, dH, dW = run_actor_update(ctx, mode, w, H, W, y, old, ref, reward, 0.0)
    assert np.abs(np_of(adv) - adv_ref).max() <= ADV_TOL
    dead = torch.ones(T, dtype=torch.bool, device=dev)
    dead[lt] = False
    assert int(torch.count_nonzero(g[dead])) == 0 and int(torch.count_nonzero(dH[dead].float())) == 0
    assert np.abs(np_of(logp[lt]) - o_logp).max() <= LOGP_TOL
    assert np.abs(np_of(lse[lt]) - o_lse).max() <= LOGP_TOL
    assert np.abs(np_of(ent[lt]) - o_ent).max() <= LOGP_TOL
    assert np.abs(np_of(g[lt]) - lref["dlogp"]).max() <= 5e-3 * np.abs(lref["dlogp"]).max()
    for k in ("loss", "pg_loss"):
        assert rel(res[k], lref["pg_loss"]) <= LOSS_RTOL, (k, res[k], lref["pg_loss"])
    assert abs(res["clip_frac"] - lref["clipped"].sum() / T) <= 0.5 / T
    assert_grad_close(np_of(dW[torch.as_tensor(vs, device=dev)]), dW_ref, "dW")
    assert_grad_close(np_of(dH[lt[torch.as_tensor(pick, device=dev)]].float()), dH_ref, "dH")
