"""Seeded sweep over random shapes, split counts, token blocks and GEMM variants: pack -> log-prob
-> loss -> backward and the fused update against the fp64 oracle.  The fixed parameter lists of the
other GPU tests place sizes on the tile edges; this one draws sizes nobody chose."""
import math

import numpy as np
import pytest
import torch

from oracle import grpo_oracle as O
from paper_2507_01663_b200 import workloads as wl
from gpu_util import GRAD_RTOL, LOGP_TOL, LOSS_RTOL, device, f32, np_of, rel

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2507_01663_b200 import binding as B
    c = B.Context(0)
    yield c
    c.close()


def draw_case(seed):
    rng = np.random.default_rng(1000 + seed)
    large = seed >= 100                               # a few cases several tiles wide in every dimension
    B = int(rng.integers(1, 24))
    lengths = rng.integers(0, 500 if large else 140, size=B)            # empty sequences allowed
    if lengths.sum() == 0:
        lengths[0] = 1
    d = 8 * int(rng.integers(1, 200 if large else 90))
    V = 8 * int(rng.integers(1, 3000 if large else 1100))
    return {"B": B, "lengths": lengths, "d": d, "V": V,
            "splits": int(rng.choice([0, 0, 1, 2, 3, 5, 8, 13])),
            "token_block": int(rng.choice([0, 128, 256, 384, 1024])),
            "variant": int(rng.choice([1, 2])),
            "agg_mode": int(rng.integers(0, 2)),
            "clip": (float(rng.uniform(0.05, 0.3)), float(rng.uniform(0.05, 0.4))),
            "kl": float(rng.choice([0.0, 0.04, 0.5])),
            "n_store": B + int(rng.integers(0, 9)), "seed": seed}


@pytest.mark.parametrize("seed", list(range(64)) + list(range(100, 112)))
def test_random_chain(ctx, seed):
    from paper_2507_01663_b200 import binding as Bn
    c = draw_case(seed)
    dev = device()
    rng = np.random.default_rng(5000 + seed)
    B, d, V = c["B"], c["d"], c["V"]
    # a store of n_store samples; the micro-batch takes B of them in a random order
    store_len = np.concatenate([c["lengths"], rng.integers(1, 50, size=c["n_store"] - B)])
    perm = rng.permutation(c["n_store"])
    store_len = store_len[perm]
    idx = np.argsort(perm)[:B].astype(np.int32)       # store rows that hold the B chosen lengths, in order
    off = np.concatenate([[0], np.cumsum(store_len)]).astype(np.int64)
    Ttot = int(off[-1])
    H = wl._normal_matrix(seed, wl.S_HIDDEN, Ttot, d, 1.0, "cpu")
    W = wl._normal_matrix(seed, wl.S_W, V, d, 1.0 / math.sqrt(d), "cpu")
    y = wl.randint(seed, wl.S_TARGET, 0, Ttot, V).to(torch.int32)
    adv_store = rng.standard_normal(c["n_store"]).astype(np.float32)

    # oracle: pack, then score, then everything downstream
    cols = {"hidden": wl.bf16_bits(H), "target": y.numpy()}
    packed_ref = O.pack_microbatch_ref(off, idx, cols)
    cu = packed_ref["cu_seqlens"]
    T = int(cu[-1])
    lp, ent_r, lse_r = O.token_logprob_ref(packed_ref["hidden"], wl.bf16_bits(W), packed_ref["target"])
    old = (lp + 0.15 * rng.standard_normal(T)).astype(np.float32)
    ref = (lp + 0.15 * rng.standard_normal(T)).astype(np.float32)
    old_store, ref_store = np.zeros(Ttot, np.float32), np.zeros(Ttot, np.float32)
    for j, i in enumerate(idx):
        old_store[off[i]:off[i + 1]] = old[cu[j]:cu[j + 1]]
        ref_store[off[i]:off[i + 1]] = ref[cu[j]:cu[j + 1]]

    # device: pack
    store = {"tok_offset_host": off, "d": d, "hidden": H.to(dev), "target": y.to(dev), "old_logp": f32(old_store),
             "ref_logp": f32(ref_store), "adv": f32(adv_store)}
    from gpu_util import packed_buffers
    out = packed_buffers(T + 3, B + 1, d)
    ctx.set_tuning(c["splits"], c["token_block"], c["variant"])
    assert ctx.pack_microbatch(store, idx, out) == T
    assert np.array_equal(np_of(out["cu_seqlens"])[:B + 1], cu)
    assert np.array_equal(wl.bf16_bits(out["hidden"][:T].cpu()), packed_ref["hidden"])
    assert np.array_equal(np_of(out["target"])[:T], packed_ref["target"])
    assert np.array_equal(np_of(out["old_logp"])[:T], old) and np.array_equal(np_of(out["adv_seq"])[:B], adv_store[idx])

    # device: three calls
    Wd = W.to(dev)
    logp, ent, lse, g = (torch.full((T,), 9.0, device=dev) for _ in range(4))
    loss_out = Bn.new_loss_out(dev)
    ctx.token_logprob(out["hidden"], Wd, out["target"], logp, ent, lse, T=T)
    ctx.policy_loss(logp, out["old_logp"], out["ref_logp"], out["adv_seq"], out["cu_seqlens"], loss_out, g, ent,
                    c["clip"][0], c["clip"][1], c["kl"], c["agg_mode"], 1.0, B=B, T=T)
    dH = torch.full((T, d), 7.0, dtype=torch.bfloat16, device=dev)
    dW = torch.full((V, d), 7.0, device=dev)
    ctx.policy_loss_backward(out["hidden"], Wd, out["target"], lse, g, dH, dW, False, T=T)
    # device: the fused call
    logp_f, ent_f, lse_f, g_f = (torch.full((T,), 9.0, device=dev) for _ in range(4))
    loss_out_f = Bn.new_loss_out(dev)
    dH_f, dW_f = torch.full_like(dH, 3.0), torch.full_like(dW, 3.0)
    ctx.policy_update(out["hidden"], Wd, out["target"], out["old_logp"], out["ref_logp"], out["adv_seq"],
                      out["cu_seqlens"], loss_out_f, logp_f, lse_f, dH_f, dW_f, entropy=ent_f, dlogp=g_f,
                      clip_lo=c["clip"][0], clip_hi=c["clip"][1], kl_coef=c["kl"], agg_mode=c["agg_mode"], B=B, T=T)
    flags = ctx.check_device_errors()
    ctx.set_tuning(0, 0)
    assert flags == 0, c

    for name, got, want in (("logp", logp, lp), ("ent", ent, ent_r), ("lse", lse, lse_r), ("logp_f", logp_f, lp),
                            ("ent_f", ent_f, ent_r), ("lse_f", lse_f, lse_r)):
        assert np.abs(np_of(got) - want).max() <= LOGP_TOL, (name, c)
    # loss stage fed with the device's own log-probs (stage isolation)
    oref = O.policy_loss_ref(np_of(logp), old, ref, adv_store[idx], cu, c["clip"][0], c["clip"][1], c["kl"],
                             c["agg_mode"], 1.0, entropy=np_of(ent))
    res, res_f = Bn.read_loss_out(loss_out), Bn.read_loss_out(loss_out_f)
    scale = max(abs(oref["pg_loss"]), abs(oref["kl_mean"]), 1e-3)
    for k in ("loss", "pg_loss", "kl_mean"):
        assert abs(res[k] - oref[k]) <= LOSS_RTOL * max(abs(oref[k]), scale), (k, c)
    assert rel(res["entropy_mean"], oref["entropy_mean"]) <= LOSS_RTOL
    assert res["n_tokens"] == T
    near = (np.abs(oref["rho"] - (1 - c["clip"][0])) < 1e-5) | (np.abs(oref["rho"] - (1 + c["clip"][1])) < 1e-5)
    gmax = max(np.abs(oref["dlogp"]).max(), 1e-30)
    assert np.abs(np_of(g) - oref["dlogp"])[~near].max(initial=0.0) <= 1e-5 * gmax, c
    # backward fed with the device's lse and dlogp
    dH_ref, dW_ref = O.policy_loss_backward_ref(packed_ref["hidden"], wl.bf16_bits(W), packed_ref["target"], np_of(lse),
                                                np_of(g))
    nH, nW = max(np.linalg.norm(dH_ref), 1e-30), max(np.linalg.norm(dW_ref), 1e-30)
    assert np.linalg.norm(np_of(dH.float()) - dH_ref) <= GRAD_RTOL * nH, c
    assert np.linalg.norm(np_of(dW) - dW_ref) <= GRAD_RTOL * nW, c
    # the fused call: same record given the same log-probs; gradients against its own lse / dlogp
    if torch.equal(logp_f, logp) and torch.equal(ent_f, ent):
        assert res_f == res and torch.equal(g_f, g), c
    dH_ref_f, dW_ref_f = O.policy_loss_backward_ref(packed_ref["hidden"], wl.bf16_bits(W), packed_ref["target"],
                                                    np_of(lse_f), np_of(g_f))
    assert np.linalg.norm(np_of(dH_f.float()) - dH_ref_f) <= GRAD_RTOL * nH, c
    assert np.linalg.norm(np_of(dW_f) - dW_ref_f) <= GRAD_RTOL * nW, c
