"""af_token_logprob_static: the allocation-free scoring call must reproduce af_token_logprob.

This file sorts last on purpose: a run that stops at the first failure has by then exercised
every other test.  It does not depend on them -- it also passes alone in a fresh process, where
its first call is the one that performs the per-device set-up.
"""
import math

import numpy as np
import pytest
import torch

from paper_2507_01663_b200 import workloads as wl
from gpu_util import LOGP_TOL, device, np_of

pytestmark = pytest.mark.gpu


def _case(T, d, V, seed):
    dev = device()
    H = wl._normal_matrix(seed, wl.S_HIDDEN, T, d, 1.0, dev)
    W = wl._normal_matrix(seed, wl.S_W, V, d, 1.0 / math.sqrt(d), dev)
    y = wl.randint(seed, wl.S_TARGET, 0, T, V, dev).to(torch.int32)
    return H, W, y


def _both(ctx, H, W, y):
    from paper_2507_01663_b200 import binding as B
    dev = device()
    T = H.shape[0]
    ref = [torch.full((T,), 5.0, device=dev) for _ in range(3)]
    got = [torch.full((T,), 6.0, device=dev) for _ in range(3)]
    flags = torch.zeros(1, dtype=torch.int32, device=dev)
    ctx.token_logprob(H, W, y, *ref)
    B.token_logprob_static(H, W, y, *got, device_flags=flags)
    torch.cuda.synchronize()
    assert ctx.check_device_errors() == 0 and int(flags.item()) == 0
    return [np_of(t) for t in ref], [np_of(t) for t in got]


def test_static_entry_matches_context_entry_on_two_calls_in_a_row():
    from paper_2507_01663_b200 import binding as B
    ctx = B.Context(0)
    try:
        # call 1 fills the shared scratch with a large batch; call 2 is a smaller, differently
        # split batch that must not be disturbed by what call 1 left behind
        for T, d, V, seed in [(3000, 256, 5000, 31), (257, 512, 8200, 32)]:
            ref, got = _both(ctx, *_case(T, d, V, seed))
            for r, g in zip(ref, got):
                assert np.isfinite(g).all()
                assert np.abs(g - r).max() <= LOGP_TOL
    finally:
        ctx.close()


def test_static_entry_limits_and_flags():
    from paper_2507_01663_b200 import binding as B
    dev = device()
    H, W, y = _case(64, 64, 300, 33)
    out = torch.zeros(64, device=dev)
    # beyond the fixed scratch: refused with a clear status, nothing launched
    with pytest.raises(B.AfError) as e:
        B.token_logprob_static(H, W, y, out, T=32769)
    assert e.value.status == -4
    B.token_logprob_static(H, W, y, out, T=0)                     # empty batch: no-op
    # a bad target is reported through the caller's flag word and as NaN
    y2 = y.clone()
    y2[7] = 300
    flags = torch.zeros(1, dtype=torch.int32, device=dev)
    B.token_logprob_static(H, W, y2, out, device_flags=flags)
    torch.cuda.synchronize()
    assert int(flags.item()) & B.DEVERR_TARGET_RANGE and bool(torch.isnan(out[7])) and int(torch.isnan(out).sum()) == 1
