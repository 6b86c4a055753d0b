"""Sizes at and beyond what the entry points accept, and the largest shapes along each axis that a
test can afford: many token rows (65536 pair tiles), a very wide vocabulary (4097 column tiles), a
deep reduction -- each against the oracle on all or on sampled rows."""
import math

import numpy as np
import pytest
import torch

from oracle import grpo_oracle as O
from paper_2507_01663_b200 import workloads as wl
from gpu_util import GRAD_RTOL, LOGP_TOL, device, np_of, sample_rows

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2507_01663_b200 import binding as B
    c = B.Context(0)
    yield c
    c.close()


def test_sizes_beyond_the_limits_are_refused_on_the_host(ctx):
    """T, N >= 2^31 never reach a kernel (32-bit token indices): AF_ERR_SHAPE, nothing launched."""
    from paper_2507_01663_b200 import binding as B
    dev = device()
    H = torch.zeros(8, 16, dtype=torch.bfloat16, device=dev)
    W = torch.zeros(16, 16, dtype=torch.bfloat16, device=dev)
    y = torch.zeros(8, dtype=torch.int32, device=dev)
    f = torch.zeros(8, device=dev)
    dW = torch.zeros(16, 16, device=dev)
    lo = B.new_loss_out(dev)
    big = 1 << 31
    with pytest.raises(B.AfError) as e:
        ctx.token_logprob(H, W, y, f, T=big)
    assert e.value.status == -2
    with pytest.raises(B.AfError) as e:
        ctx.token_logprob_shard(H, W, y, 0, torch.zeros(8, 4, device=dev), T=big)
    assert e.value.status == -2
    with pytest.raises(B.AfError) as e:
        ctx.policy_loss_backward(H, W, y, f, f, H.clone(), dW, T=big)
    assert e.value.status == -2
    with pytest.raises(B.AfError) as e:
        ctx.policy_loss(f, f, f, f, torch.zeros(2, dtype=torch.int32, device=dev), lo, T=big)
    assert e.value.status == -2
    with pytest.raises(B.AfError) as e:
        ctx.policy_update(H, W, y, f, f, f, torch.zeros(2, dtype=torch.int32, device=dev), lo, f, f, H.clone(), dW, T=big)
    assert e.value.status == -2
    with pytest.raises(B.AfError) as e:
        ctx.grpo_advantage(f, y, 4, f, N=big)                      # membership by id: 32-bit member counts
    assert e.value.status == -2
    with pytest.raises(B.AfError) as e:
        ctx.reserve(big, 4, 16, 16)
    assert e.value.status == -2
    assert ctx.check_device_errors() == 0


def test_many_token_rows(ctx):
    """T = 2^24 + 77 rows at d = 64 (2.1 GB of hidden states, 65537 pair tiles, a ragged last tile)."""
    dev = device()
    T, d, V = (1 << 24) + 77, 64, 520
    H = wl._normal_matrix(51, wl.S_HIDDEN, T, d, 1.0, dev)
    W = wl._normal_matrix(51, wl.S_W, V, d, 1.0 / math.sqrt(d), dev)
    y = wl.randint(51, wl.S_TARGET, 0, T, V, dev).to(torch.int32)
    logp, ent, lse = (torch.full((T,), 9.0, device=dev) for _ in range(3))
    ctx.token_logprob(H, W, y, logp, ent, lse)
    assert ctx.check_device_errors() == 0
    rows = sample_rows(np.array([0, T]), T, 4096, seed=52)
    rt = torch.as_tensor(rows, device=dev)
    want = O.token_logprob_ref(wl.bf16_bits(H[rt]), wl.bf16_bits(W), np_of(y[rt]))
    for got, ref in zip((logp, ent, lse), want):
        assert np.abs(np_of(got[rt]) - ref).max() <= LOGP_TOL
    assert bool(torch.isfinite(logp).all()) and float(logp.max()) <= 1e-5
    assert float(ent.min()) >= -1e-4 and float(ent.max()) <= math.log(V) + 1e-4


def test_very_wide_vocabulary(ctx):
    """V = 2^20 + 8 (4097 column tiles) at T = 300, d = 64: forward on every row, backward on all of dH
    and sampled rows of dW."""
    dev = device()
    T, d, V = 300, 64, (1 << 20) + 8
    H = wl._normal_matrix(53, wl.S_HIDDEN, T, d, 1.0, "cpu")
    W = wl._normal_matrix(53, wl.S_W, V, d, 1.0 / math.sqrt(d), "cpu")
    y = wl.randint(53, wl.S_TARGET, 0, T, V).to(torch.int32)
    y[0], y[1], y[2] = V - 1, 0, V - 9
    want = O.token_logprob_ref(wl.bf16_bits(H), wl.bf16_bits(W), y.numpy())
    Hd, Wd, yd = H.to(dev), W.to(dev), y.to(dev)
    logp, ent, lse = (torch.full((T,), 9.0, device=dev) for _ in range(3))
    ctx.token_logprob(Hd, Wd, yd, logp, ent, lse)
    for got, ref in zip((logp, ent, lse), want):
        assert np.abs(np_of(got) - ref).max() <= LOGP_TOL
    g = (wl.normal01(53, wl.S_G, 0, T) / T)
    dH = torch.empty(T, d, dtype=torch.bfloat16, device=dev)
    dW = torch.empty(V, d, device=dev)
    ctx.policy_loss_backward(Hd, Wd, yd, torch.as_tensor(want[2], dtype=torch.float32, device=dev), g.to(dev), dH, dW)
    assert ctx.check_device_errors() == 0
    dH_ref, _ = O.policy_loss_backward_ref(wl.bf16_bits(H), wl.bf16_bits(W), y.numpy(), want[2].astype(np.float32), g.numpy())
    n = np.linalg.norm(dH_ref)
    assert np.linalg.norm(np_of(dH.float()) - dH_ref) <= GRAD_RTOL * n
    vs = sorted({0, 255, 256, V - 1, V - 8, V - 9, 1 << 19} | {int(v) for v in y[:40]})
    dW_ref = O.policy_loss_backward_ref(wl.bf16_bits(H), wl.bf16_bits(W), y.numpy(), want[2].astype(np.float32), g.numpy(),
                                        vocab_rows=vs)
    got = np_of(dW[torch.as_tensor(vs, device=dev)])
    assert np.linalg.norm(got - dW_ref) <= GRAD_RTOL * np.linalg.norm(dW_ref)


def test_deep_reduction(ctx):
    """d = 16384 (256 K blocks per tile) at T = 200, V = 1000."""
    T, d, V = 200, 16384, 1000
    H = wl._normal_matrix(54, wl.S_HIDDEN, T, d, 1.0, "cpu")
    W = wl._normal_matrix(54, wl.S_W, V, d, 1.0 / math.sqrt(d), "cpu")
    y = wl.randint(54, wl.S_TARGET, 0, T, V).to(torch.int32)
    want = O.token_logprob_ref(wl.bf16_bits(H), wl.bf16_bits(W), y.numpy())
    dev = device()
    logp, ent, lse = (torch.full((T,), 9.0, device=dev) for _ in range(3))
    ctx.token_logprob(H.to(dev), W.to(dev), y.to(dev), logp, ent, lse)
    assert ctx.check_device_errors() == 0
    for got, ref in zip((logp, ent, lse), want):
        assert np.abs(np_of(got) - ref).max() <= LOGP_TOL
