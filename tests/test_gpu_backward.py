"""af_policy_loss_backward against the fp64 oracle (dense at sizes the oracle can afford)."""
import math

import numpy as np
import pytest
import torch

from oracle import grpo_oracle as O
from paper_2507_01663_b200 import workloads as wl
from gpu_util import GRAD_RTOL, device, f32, np_of

pytestmark = pytest.mark.gpu


VARIANT = 0    # which GEMM variant the helpers below select (0 = library default)


@pytest.fixture(autouse=True, params=[1, 2], ids=["cta", "pair"])
def gemm_variant(request):
    """Every test of this module runs on both tensor-core main loops: one CTA per 128 x 256
    tile and a CTA pair per 256 x 256 tile (the default)."""
    global VARIANT
    VARIANT = request.param
    yield
    VARIANT = 0


@pytest.fixture(scope="module")
def ctx():
    from paper_2507_01663_b200 import binding as B
    c = B.Context(0)
    yield c
    c.close()


def inputs(T, d, V, seed):
    H = wl._normal_matrix(seed, wl.S_HIDDEN, T, d, 1.0, "cpu")
    W = wl._normal_matrix(seed, wl.S_W, V, d, 1.0 / math.sqrt(d), "cpu")
    y = wl.randint(seed, wl.S_TARGET, 0, T, V).to(torch.int32)
    g = wl.normal01(seed, wl.S_G, 0, T) / max(T, 1)
    _, _, lse = O.token_logprob_ref(wl.bf16_bits(H), wl.bf16_bits(W), y.numpy())
    return H, W, y, g, lse


def run_bwd(ctx, H, W, y, g, lse, token_block=0, accumulate=False, dW_init=None):
    dev = device()
    T, d = H.shape
    V = W.shape[0]
    dH = torch.full((max(T, 1), d), 7.0, dtype=torch.bfloat16, device=dev)
    dW = torch.full((V, d), 7.0, device=dev) if dW_init is None else dW_init.clone()
    ctx.set_tuning(0, token_block, VARIANT)
    ctx.policy_loss_backward(H.to(dev), W.to(dev), y.to(dev), f32(lse), g.to(dev), dH, dW, accumulate, T=T)
    flags = ctx.check_device_errors()
    ctx.set_tuning(0, 0)
    assert flags == 0
    return np_of(dH.float())[:T], np_of(dW)


def compare(dH, dW, dH_ref, dW_ref):
    nH, nW = np.linalg.norm(dH_ref), np.linalg.norm(dW_ref)
    assert abs(np.linalg.norm(dH) - nH) <= GRAD_RTOL * nH          # gradient norms (the stated bar)
    assert abs(np.linalg.norm(dW) - nW) <= GRAD_RTOL * nW
    assert np.linalg.norm(dH - dH_ref) <= GRAD_RTOL * nH           # and the direction, element-wise
    assert np.linalg.norm(dW - dW_ref) <= GRAD_RTOL * nW
    # bf16 rounding of dZ and of dH bounds the element error by a small multiple of the largest entry
    assert np.abs(dH - dH_ref).max() <= 2e-2 * np.abs(dH_ref).max()
    assert np.abs(dW - dW_ref).max() <= 2e-2 * np.abs(dW_ref).max()


@pytest.mark.parametrize("T,d,V,tb", [(128, 64, 256, 0), (300, 128, 512, 128), (1, 8, 8, 0), (77, 72, 1000, 0),
                                      (1024, 512, 8192, 0), (1000, 264, 3000, 256), (700, 3584, 1024, 384)])
def test_dense_against_oracle(ctx, T, d, V, tb):
    H, W, y, g, lse = inputs(T, d, V, seed=T + V)
    dH, dW = run_bwd(ctx, H, W, y, g, lse, tb)
    dH_ref, dW_ref = O.policy_loss_backward_ref(wl.bf16_bits(H), wl.bf16_bits(W), y.numpy(), lse, g.numpy())
    compare(dH, dW, dH_ref, dW_ref)


def test_cfg4_mini_chain(ctx):
    """Whole chain on the reduced actor-update workload: oracle log-probs -> loss -> dlogp ->
    gradients, against the GPU chain run on the same packed inputs."""
    from paper_2507_01663_b200 import binding as B
    dev = device()
    w = wl.make_workload("cfg4_mini")
    H, W, y = wl.gen_hidden(w), wl.gen_weight(w), wl.gen_target(w)
    T = w.total_tokens
    cu = w.tok_offset
    r = np_of(wl.gen_reward(w))
    adv = O.grpo_advantage_ref(r, w.group_id, w.n_prompts)
    lp, ent, lse = O.token_logprob_ref(wl.bf16_bits(H), wl.bf16_bits(W), y.numpy())
    old = torch.tensor(lp, dtype=torch.float32) + wl.gen_noise(w, wl.S_OLD, T)
    ref = torch.tensor(lp, dtype=torch.float32) + wl.gen_noise(w, wl.S_REF, T)
    oref = O.policy_loss_ref(lp, old.numpy(), ref.numpy(), adv.astype(np.float32), cu, w.clip_eps, w.clip_eps, w.kl_coef)
    dH_ref, dW_ref = O.policy_loss_backward_ref(wl.bf16_bits(H), wl.bf16_bits(W), y.numpy(), lse, oref["dlogp"])
    # GPU chain
    Hd, Wd, yd = H.to(dev), W.to(dev), y.to(dev)
    logp_d, ent_d, lse_d, g_d = (torch.empty(T, device=dev) for _ in range(4))
    ctx.set_tuning(0, 0, VARIANT)
    ctx.token_logprob(Hd, Wd, yd, logp_d, ent_d, lse_d)
    out = B.new_loss_out(dev)
    ctx.policy_loss(logp_d, old.to(dev), ref.to(dev), f32(adv), torch.as_tensor(cu.astype(np.int32), device=dev), out,
                    g_d, ent_d, w.clip_eps, w.clip_eps, w.kl_coef)
    dH = torch.empty(T, w.d, dtype=torch.bfloat16, device=dev)
    dW = torch.empty(w.V, w.d, device=dev)
    ctx.policy_loss_backward(Hd, Wd, yd, lse_d, g_d, dH, dW)
    ctx.set_tuning(0, 0)
    res = B.read_loss_out(out)
    assert ctx.check_device_errors() == 0
    assert abs(res["loss"] - oref["loss"]) <= 1e-3 * abs(oref["loss"])
    # tokens whose ratio sits within the log-prob tolerance of a clip bound may flip sides between
    # the two chains; their rows are excluded from the element-wise check, the norms keep them
    rho = oref["rho"]
    near = (np.abs(rho - 0.8) < 4e-3) | (np.abs(rho - 1.2) < 4e-3)
    dHg = np_of(dH.float())
    nH = np.linalg.norm(dH_ref[~near])
    assert np.linalg.norm(dHg[~near] - dH_ref[~near]) <= GRAD_RTOL * nH
    if not near.any():
        compare(dHg, np_of(dW), dH_ref, dW_ref)
    else:
        nW = np.linalg.norm(dW_ref)
        assert abs(np.linalg.norm(np_of(dW)) - nW) <= 5 * GRAD_RTOL * nW


def test_accumulate_and_zero_gradient(ctx):
    H, W, y, g, lse = inputs(260, 64, 520, seed=5)
    dev = device()
    base = wl._normal_matrix(8, wl.S_MISC, 520, 64, 1.0, "cpu").float().to(dev)
    _, dW_plain = run_bwd(ctx, H, W, y, g, lse)
    _, dW_acc = run_bwd(ctx, H, W, y, g, lse, accumulate=True, dW_init=base)
    assert np.allclose(dW_acc, dW_plain + np_of(base), rtol=0, atol=1e-6)
    # token blocks change only the fp32 summation order of dW
    _, dW_blk = run_bwd(ctx, H, W, y, g, lse, token_block=128)
    assert np.abs(dW_blk - dW_plain).max() <= 1e-5 * np.abs(dW_plain).max()
    # zero upstream gradient gives exact zeros
    dH0, dW0 = run_bwd(ctx, H, W, y, torch.zeros_like(g), lse)
    assert not dH0.any() and not dW0.any()
    # T = 0: dW is zeroed (or left alone when accumulating)
    _, dWz = run_bwd(ctx, H[:0], W, y[:0], g[:0], lse[:0])
    assert not dWz.any()
    _, dWk = run_bwd(ctx, H[:0], W, y[:0], g[:0], lse[:0], accumulate=True, dW_init=base)
    assert np.array_equal(dWk, np_of(base))


def test_bitwise_reproducible(ctx):
    H, W, y, g, lse = inputs(500, 128, 1024, seed=9)
    a = run_bwd(ctx, H, W, y, g, lse)
    b = run_bwd(ctx, H, W, y, g, lse)
    assert a[0].tobytes() == b[0].tobytes() and a[1].tobytes() == b[1].tobytes()


def test_host_argument_errors(ctx):
    from paper_2507_01663_b200.binding import AfError
    dev = device()
    H = torch.zeros(4, 16, dtype=torch.bfloat16, device=dev)
    W = torch.zeros(12, 16, dtype=torch.bfloat16, device=dev)       # V % 8 != 0
    y = torch.zeros(4, dtype=torch.int32, device=dev)
    v = torch.zeros(4, device=dev)
    with pytest.raises(AfError) as e:
        ctx.policy_loss_backward(H, W, y, v, v, torch.zeros_like(H), torch.zeros(12, 16, device=dev))
    assert e.value.status == -3


@pytest.mark.parametrize("cuts", [[0, 8192], [0, 3000, 8192], [0, 8, 264, 4096, 8184, 8192]])
def test_vocabulary_shards_of_the_backward(ctx, cuts):
    """The head split by vocabulary rows: every shard's dH contribution and dW rows against the
    oracle's shard backward; the contributions add up to the unsharded call's dH, the rows stack to
    its dW."""
    dev = device()
    w = wl.make_workload("cfg4_mini")                       # d = 512, V = 8192
    H, W, y = wl.gen_hidden(w), wl.gen_weight(w), wl.gen_target(w)
    T = H.shape[0]
    g = wl.normal01(w.seed, wl.S_G, 0, T) / T
    _, _, lse = O.token_logprob_ref(wl.bf16_bits(H), wl.bf16_bits(W), y.numpy())
    Hd, Wd, yd, gd, lsed = H.to(dev), W.to(dev), y.to(dev), g.to(dev), f32(lse)
    ctx.set_tuning(0, 256, VARIANT)
    dH_sum = np.zeros((T, w.d))
    rows = []
    for a, b in zip(cuts[:-1], cuts[1:]):
        dH_p = torch.full((T, w.d), 7.0, dtype=torch.bfloat16, device=dev)
        dW_s = torch.full((b - a, w.d), 7.0, device=dev)
        ctx.policy_loss_backward_shard(Hd, Wd[a:b].contiguous(), yd, lsed, gd, a, dH_p, dW_s)
        dH_ref, dW_ref = O.policy_loss_backward_shard_ref(wl.bf16_bits(H), wl.bf16_bits(W[a:b]), y.numpy(), lse,
                                                          g.numpy(), a)
        nH, nW = np.linalg.norm(dH_ref), np.linalg.norm(dW_ref)
        assert np.linalg.norm(np_of(dH_p.float()) - dH_ref) <= GRAD_RTOL * nH
        assert np.linalg.norm(np_of(dW_s) - dW_ref) <= GRAD_RTOL * nW
        dH_sum += np_of(dH_p.float())
        rows.append(np_of(dW_s))
    dH_full = torch.empty(T, w.d, dtype=torch.bfloat16, device=dev)
    dW_full = torch.empty(w.V, w.d, device=dev)
    ctx.policy_loss_backward(Hd, Wd, yd, lsed, gd, dH_full, dW_full)
    flags = ctx.check_device_errors()
    ctx.set_tuning(0, 0)
    assert flags == 0
    ref_H, ref_W = O.policy_loss_backward_ref(wl.bf16_bits(H), wl.bf16_bits(W), y.numpy(), lse, g.numpy())
    compare(dH_sum, np.concatenate(rows), ref_H, ref_W)
    # each dW row is computed from the same dZ column whichever shard it sits in
    assert np.abs(np.concatenate(rows) - np_of(dW_full)).max() <= 1e-6 * np.abs(np_of(dW_full)).max() + 1e-12
    assert np.linalg.norm(dH_sum - np_of(dH_full.float())) <= GRAD_RTOL * np.linalg.norm(ref_H)


def test_shard_backward_argument_errors(ctx):
    from paper_2507_01663_b200 import binding as B
    dev = device()
    H = torch.zeros(4, 8, dtype=torch.bfloat16, device=dev)
    z4 = torch.zeros(4, device=dev)
    y = torch.zeros(4, dtype=torch.int32, device=dev)
    with pytest.raises(B.AfError):                       # shard rows must be a multiple of 8
        ctx.policy_loss_backward_shard(H, torch.zeros(12, 8, dtype=torch.bfloat16, device=dev), y, z4, z4, 0,
                                       torch.zeros_like(H), torch.zeros(12, 8, device=dev))
    with pytest.raises(B.AfError):                       # negative offset
        ctx.policy_loss_backward_shard(H, torch.zeros(16, 8, dtype=torch.bfloat16, device=dev), y, z4, z4, -8,
                                       torch.zeros_like(H), torch.zeros(16, 8, device=dev))
    assert ctx.check_device_errors() == 0


@pytest.mark.parametrize("fused", [False, True], ids=["backward", "update"])
def test_dw_ready_event_marks_the_complete_gradient(ctx, fused):
    """With a "d_W ready" event registered, a second stream that waits on it sees the finished d_W
    (the data-parallel all-reduce starts there, beside the last block's dH product), and the
    results are those of the default order bit for bit."""
    from paper_2507_01663_b200 import binding as B
    dev = device()
    H, W, y, g, lse = inputs(1000, 264, 3000, seed=77)
    Hd, Wd, yd, gd, lsed = H.to(dev), W.to(dev), y.to(dev), g.to(dev), f32(lse)
    cu = torch.as_tensor(np.array([0, 400, 1000], dtype=np.int32), device=dev)
    adv = f32([0.7, -1.1])
    old = lsed * 0 - 8.0
    ctx.set_tuning(0, 256, VARIANT)

    def run():
        dH = torch.full((1000, 264), 7.0, dtype=torch.bfloat16, device=dev)
        dW = torch.full((3000, 264), 7.0, device=dev)
        if fused:
            lo = B.new_loss_out(dev)
            logp, lse_o = torch.empty(1000, device=dev), torch.empty(1000, device=dev)
            ctx.policy_update(Hd, Wd, yd, old, old, adv, cu, lo, logp, lse_o, dH, dW)
        else:
            ctx.policy_loss_backward(Hd, Wd, yd, lsed, gd, dH, dW)
        return dH, dW

    dH0, dW0 = run()
    torch.cuda.synchronize()
    ev = torch.cuda.Event()
    ev.record()                                   # creates the underlying CUDA event
    ctx.set_dw_ready_event(ev)
    side = torch.cuda.Stream()
    try:
        dH1, dW1 = run()
        with torch.cuda.stream(side):
            side.wait_event(ev)
            snap = dW1.clone()                    # reads d_W as soon as the event allows
        torch.cuda.synchronize()
    finally:
        ctx.set_dw_ready_event(None)
        ctx.set_tuning(0, 0)
    assert ctx.check_device_errors() == 0
    assert torch.equal(snap, dW1) and torch.equal(dW1, dW0) and torch.equal(dH1, dH0)


def test_backward_with_die_aware_dealing(ctx):
    """gemm_variant 3 on the backward's three products (the dZ and dH products have enough units for
    the mode to switch on at this size): dense against the oracle."""
    if VARIANT != 2:
        pytest.skip("one run is enough: the test selects its own variant")
    dev = device()
    T, d, V = 12000, 264, 2048
    H, W, y, g, lse = inputs(T, d, V, seed=91)
    dH = torch.full((T, d), 7.0, dtype=torch.bfloat16, device=dev)
    dW = torch.full((V, d), 7.0, device=dev)
    ctx.set_tuning(0, 0, 3)
    ctx.policy_loss_backward(H.to(dev), W.to(dev), y.to(dev), f32(lse), g.to(dev), dH, dW)
    flags = ctx.check_device_errors()
    ctx.set_tuning(0, 0)
    assert flags == 0
    dH_ref, dW_ref = O.policy_loss_backward_ref(wl.bf16_bits(H), wl.bf16_bits(W), y.numpy(), lse, g.numpy())
    compare(np_of(dH.float()), np_of(dW), dH_ref, dW_ref)
