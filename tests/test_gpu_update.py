"""af_policy_update (forward + loss + backward in one call) against the oracle chain and against
the three separate calls it replaces."""
import numpy as np
import pytest
import torch

from oracle import grpo_oracle as O
from paper_2507_01663_b200 import workloads as wl
from gpu_util import GRAD_RTOL, LOGP_TOL, LOSS_RTOL, device, f32, np_of, off_the_clip_bounds, rel

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2507_01663_b200 import binding as B
    c = B.Context(0)
    yield c
    c.close()


def chain_inputs(name, seed_shift=0):
    """Packed micro-batch of a workload with old / ref log-probs around the oracle's own."""
    w = wl.make_workload(name)
    H, W, y = wl.gen_hidden(w), wl.gen_weight(w), wl.gen_target(w)
    T = w.total_tokens
    cu = w.tok_offset
    adv = O.grpo_advantage_ref(np_of(wl.gen_reward(w)), w.group_id, w.n_prompts).astype(np.float32)
    lp, ent, lse = O.token_logprob_ref(wl.bf16_bits(H), wl.bf16_bits(W), y.numpy())
    old = torch.tensor(lp, dtype=torch.float32) + wl.gen_noise(w, wl.S_OLD, T)
    old = torch.tensor(off_the_clip_bounds(lp, old.numpy(), w.clip_eps, w.clip_eps), dtype=torch.float32)
    ref = torch.tensor(lp, dtype=torch.float32) + wl.gen_noise(w, wl.S_REF, T)
    return w, H, W, y, cu, adv, old, ref, (lp, ent, lse)


def run_fused(ctx, w, H, W, y, cu, adv, old, ref, variant, token_block=0, agg_mode=0, accumulate=False, dW_init=None):
    from paper_2507_01663_b200 import binding as B
    dev = device()
    T = H.shape[0]
    out = B.new_loss_out(dev)
    logp, ent, lse, g = (torch.full((T,), 9.0, device=dev) for _ in range(4))
    dH = torch.full((T, w.d), 7.0, dtype=torch.bfloat16, device=dev)
    dW = torch.full((w.V, w.d), 7.0, device=dev) if dW_init is None else dW_init.clone()
    ctx.set_tuning(0, token_block, variant)
    ctx.policy_update(H.to(dev), W.to(dev), y.to(dev), old.to(dev), ref.to(dev), f32(adv),
                      torch.as_tensor(cu.astype(np.int32), device=dev), out, logp, lse, dH, dW, entropy=ent, dlogp=g,
                      accumulate_dW=accumulate, clip_lo=w.clip_eps, clip_hi=w.clip_eps, kl_coef=w.kl_coef,
                      agg_mode=agg_mode)
    flags = ctx.check_device_errors()
    ctx.set_tuning(0, 0)
    assert flags == 0
    return B.read_loss_out(out), logp, ent, lse, g, dH, dW


@pytest.mark.parametrize("variant", [1, 2], ids=["cta", "pair"])
@pytest.mark.parametrize("name,token_block,agg_mode", [("cfg4_mini", 0, 0), ("cfg4_mini", 256, 1), ("cfg1", 128, 0)])
def test_fused_update_matches_oracle_chain(ctx, name, token_block, agg_mode, variant):
    w, H, W, y, cu, adv, old, ref, (lp, ent_r, lse_r) = chain_inputs(name)
    res, logp, ent, lse, g, dH, dW = run_fused(ctx, w, H, W, y, cu, adv, old, ref, variant, token_block, agg_mode)
    assert np.abs(np_of(logp) - lp).max() <= LOGP_TOL
    assert np.abs(np_of(ent) - ent_r).max() <= LOGP_TOL and np.abs(np_of(lse) - lse_r).max() <= LOGP_TOL
    # loss and per-token gradient: the oracle fed with the device's log-probs (stage isolation)
    oref = O.policy_loss_ref(np_of(logp), old.numpy(), ref.numpy(), adv, cu, w.clip_eps, w.clip_eps, w.kl_coef,
                             agg_mode, 1.0, entropy=np_of(ent))
    for k in ("loss", "pg_loss", "kl_mean", "entropy_mean"):
        assert rel(res[k], oref[k]) <= LOSS_RTOL, k
    near = (np.abs(oref["rho"] - (1 - w.clip_eps)) < 1e-5) | (np.abs(oref["rho"] - (1 + w.clip_eps)) < 1e-5)
    assert np.abs(np_of(g) - oref["dlogp"])[~near].max() <= 1e-5 * np.abs(oref["dlogp"]).max()
    # gradients: the oracle's backward fed with the device's lse and dlogp
    dH_ref, dW_ref = O.policy_loss_backward_ref(wl.bf16_bits(H), wl.bf16_bits(W), y.numpy(), np_of(lse), np_of(g))
    nH, nW = np.linalg.norm(dH_ref), np.linalg.norm(dW_ref)
    assert np.linalg.norm(np_of(dH.float()) - dH_ref) <= GRAD_RTOL * nH
    assert np.linalg.norm(np_of(dW) - dW_ref) <= GRAD_RTOL * nW
    assert abs(np.linalg.norm(np_of(dH.float())) - nH) <= GRAD_RTOL * nH
    assert abs(np.linalg.norm(np_of(dW)) - nW) <= GRAD_RTOL * nW
    # and the whole chain from the oracle's own log-probs and lse (no device value enters): no token
    # sits near a clip bound (chain_inputs), so both sides clip the same tokens
    cref = O.policy_loss_ref(lp, old.numpy(), ref.numpy(), adv, cu, w.clip_eps, w.clip_eps, w.kl_coef, agg_mode, 1.0,
                             entropy=ent_r)
    assert res["clip_frac"] == pytest.approx(cref["clip_frac"], abs=1e-7)
    assert np.abs(np_of(g) - cref["dlogp"]).max() <= 5e-3 * np.abs(cref["dlogp"]).max()
    # a log-prob error e moves a token's loss by at most (|A| rho + kl_coef |exp(delta) - 1|) |e|
    slack = LOGP_TOL * float(np.abs(cref["dlogp"]).sum())
    for k in ("loss", "pg_loss"):
        assert abs(res[k] - cref[k]) <= LOSS_RTOL * abs(cref[k]) + slack, k
    dH_c, dW_c = O.policy_loss_backward_ref(wl.bf16_bits(H), wl.bf16_bits(W), y.numpy(), lse_r, cref["dlogp"])
    assert np.linalg.norm(np_of(dH.float()) - dH_c) <= GRAD_RTOL * np.linalg.norm(dH_c)
    assert np.linalg.norm(np_of(dW) - dW_c) <= GRAD_RTOL * np.linalg.norm(dW_c)


@pytest.mark.parametrize("variant", [1, 2], ids=["cta", "pair"])
def test_fused_update_equals_the_three_calls(ctx, variant):
    """Same token block, same accumulators, same per-token arithmetic: the loss record and dlogp
    agree to the last bit whenever the log-probs do; gradients within bf16 rounding of dZ."""
    from paper_2507_01663_b200 import binding as B
    dev = device()
    w, H, W, y, cu, adv, old, ref, _ = chain_inputs("cfg4_mini")
    res, logp, ent, lse, g, dH, dW = run_fused(ctx, w, H, W, y, cu, adv, old, ref, variant, 256)
    Hd, Wd, yd = H.to(dev), W.to(dev), y.to(dev)
    ctx.set_tuning(0, 256, variant)
    # the separate loss call on the fused call's log-probs reproduces its record and gradient
    out2, g2 = B.new_loss_out(dev), torch.empty_like(g)
    ctx.policy_loss(logp, old.to(dev), ref.to(dev), f32(adv), torch.as_tensor(cu.astype(np.int32), device=dev), out2,
                    g2, ent, w.clip_eps, w.clip_eps, w.kl_coef)
    assert B.read_loss_out(out2) == res and torch.equal(g2, g)
    # and the separate backward on (lse, dlogp) the same gradients up to the recomputed logits
    dH2 = torch.empty_like(dH)
    dW2 = torch.empty_like(dW)
    ctx.policy_loss_backward(Hd, Wd, yd, lse, g, dH2, dW2)
    ctx.set_tuning(0, 0)
    assert float((dW2 - dW).norm() / dW.norm()) <= 1e-3
    assert float((dH2.float() - dH.float()).norm() / dH.float().norm()) <= 1e-3
    assert ctx.check_device_errors() == 0


def test_fused_update_accumulates_and_handles_empty_batches(ctx):
    from paper_2507_01663_b200 import binding as B
    dev = device()
    w, H, W, y, cu, adv, old, ref, _ = chain_inputs("cfg1")
    base = wl._normal_matrix(9, wl.S_MISC, w.V, w.d, 1.0, "cpu").float().to(dev)
    _, _, _, _, _, _, dW0 = run_fused(ctx, w, H, W, y, cu, adv, old, ref, 0)
    _, _, _, _, _, _, dW1 = run_fused(ctx, w, H, W, y, cu, adv, old, ref, 0, accumulate=True, dW_init=base)
    assert float((dW1 - base - dW0).abs().max()) <= 2e-6            # fp32 rounding of base + dW at |base| ~ 4
    # T = 0: gradients zero, record empty
    out = B.new_loss_out(dev)
    dW = torch.full((16, 8), 3.0, device=dev)
    z = torch.zeros(0, device=dev)
    ctx.policy_update(torch.zeros(0, 8, dtype=torch.bfloat16, device=dev), torch.zeros(16, 8, dtype=torch.bfloat16, device=dev),
                      torch.zeros(0, dtype=torch.int32, device=dev), z, z, z, torch.zeros(1, dtype=torch.int32, device=dev),
                      out, z, z, torch.zeros(0, 8, dtype=torch.bfloat16, device=dev), dW, B=0, T=0)
    assert float(dW.abs().max()) == 0.0 and B.read_loss_out(out)["n_tokens"] == 0
    with pytest.raises(B.AfError):                      # V must be a multiple of 8
        ctx.policy_update(torch.zeros(4, 8, dtype=torch.bfloat16, device=dev), torch.zeros(12, 8, dtype=torch.bfloat16, device=dev),
                          torch.zeros(4, dtype=torch.int32, device=dev), torch.zeros(4, device=dev), torch.zeros(4, device=dev),
                          torch.zeros(1, device=dev), torch.tensor([0, 4], dtype=torch.int32, device=dev), out,
                          torch.zeros(4, device=dev), torch.zeros(4, device=dev),
                          torch.zeros(4, 8, dtype=torch.bfloat16, device=dev), torch.zeros(12, 8, device=dev))
    assert ctx.check_device_errors() == 0
