"""af_token_logprob_static: the scoring call for callers that cannot allocate.

It is checked against the CPU oracle and against af_token_logprob (the entry point with a context),
on two calls in a row that share the fixed scratch array, at its capacity limit, on a stream of the
caller's, and for what it must not do: allocate, or touch outputs that were not asked for.

This file sorts last on purpose: a run that stops at the first failure has by then exercised
every other test.  It does not depend on them -- it also passes alone in a fresh process, where
its first call is the one that performs the per-device set-up.
"""
import math

import numpy as np
import pytest
import torch

from oracle import grpo_oracle as O
from paper_2507_01663_b200 import workloads as wl
from gpu_util import LOGP_TOL, device, np_of

pytestmark = pytest.mark.gpu


def _case(T, d, V, seed):
    dev = device()
    H = wl._normal_matrix(seed, wl.S_HIDDEN, T, d, 1.0, dev)
    W = wl._normal_matrix(seed, wl.S_W, V, d, 1.0 / math.sqrt(d), dev)
    y = wl.randint(seed, wl.S_TARGET, 0, T, V, dev).to(torch.int32)
    return H, W, y


def _oracle(H, W, y, rows=None):
    """Oracle log-prob, entropy, lse of all rows (or the given ones), from the bits the kernel saw."""
    if rows is not None:
        rt = torch.as_tensor(rows, device=H.device)
        H, y = H[rt], y[rt]
    return O.token_logprob_ref(wl.bf16_bits(H), wl.bf16_bits(W), np_of(y))


def _both(ctx, H, W, y, stream=None):
    from paper_2507_01663_b200 import binding as B
    dev = device()
    T = H.shape[0]
    ref = [torch.full((T,), 5.0, device=dev) for _ in range(3)]
    got = [torch.full((T,), 6.0, device=dev) for _ in range(3)]
    flags = torch.zeros(1, dtype=torch.int32, device=dev)
    ctx.token_logprob(H, W, y, *ref)
    torch.cuda.synchronize()
    B.token_logprob_static(H, W, y, *got, device_flags=flags, stream=stream)
    torch.cuda.synchronize()
    assert ctx.check_device_errors() == 0 and int(flags.item()) == 0
    return [np_of(t) for t in ref], [np_of(t) for t in got]


def test_static_entry_matches_oracle_and_context_entry_on_two_calls_in_a_row():
    from paper_2507_01663_b200 import binding as B
    ctx = B.Context(0)
    try:
        # call 1 fills the shared scratch with a large batch; call 2 is a smaller, differently
        # split batch that must not be disturbed by what call 1 left behind
        for T, d, V, seed in [(3000, 256, 5000, 31), (257, 512, 8200, 32)]:
            H, W, y = _case(T, d, V, seed)
            ref, got = _both(ctx, H, W, y)
            want = _oracle(H, W, y)
            for o, r, g in zip(want, ref, got):
                assert np.isfinite(g).all()
                assert np.abs(g - o).max() <= LOGP_TOL          # the oracle
                assert np.abs(g - r).max() <= LOGP_TOL          # the entry point with a context
    finally:
        ctx.close()


def test_static_entry_at_its_capacity_limit():
    """T = 32768 exactly: the point where vocabulary ranges x tokens meets the fixed scratch, so the
    number of ranges is cut down to what fits."""
    from paper_2507_01663_b200 import binding as B
    ctx = B.Context(0)
    try:
        H, W, y = _case(32768, 64, 600, 34)
        ref, got = _both(ctx, H, W, y)
        want = _oracle(H, W, y)
        for o, r, g in zip(want, ref, got):
            assert np.abs(g - o).max() <= LOGP_TOL and np.abs(g - r).max() <= LOGP_TOL
    finally:
        ctx.close()


def test_static_entry_on_a_side_stream_leaves_unrequested_outputs_alone():
    from paper_2507_01663_b200 import binding as B
    dev = device()
    H, W, y = _case(1500, 128, 3000, 35)
    logp, ent, lse = (torch.full((1500,), 6.0, device=dev) for _ in range(3))
    B.token_logprob_static(H, W, y, logp, ent, lse)                 # first call: per-device set-up
    torch.cuda.synchronize()
    want = _oracle(H, W, y)
    # second call on a stream of the caller's, log-probs only: the outputs that were not requested
    # keep their contents, and a read queued behind the call on that stream sees its result
    logp2 = torch.full((1500,), 7.0, device=dev)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    B.token_logprob_static(H, W, y, logp2, stream=side)
    with torch.cuda.stream(side):
        doubled = logp2 * 2.0                                       # a dependent read on the same stream
    side.synchronize()
    torch.cuda.synchronize()
    assert np.abs(np_of(logp2) - want[0]).max() <= LOGP_TOL
    assert torch.equal(doubled, logp2 * 2.0)
    assert torch.equal(logp2, logp)                                 # same call, same bits
    assert np.abs(np_of(ent) - want[1]).max() <= LOGP_TOL and np.abs(np_of(lse) - want[2]).max() <= LOGP_TOL


def test_static_entry_free_memory_unchanged_by_a_call():
    """The driver reports the same free device memory before and after a call (after the first one,
    which loads the kernels): nothing was allocated on the device, by the library or for it."""
    from paper_2507_01663_b200 import binding as B
    H, W, y = _case(2048, 128, 2048, 36)
    logp = torch.empty(2048, device=device())
    B.token_logprob_static(H, W, y, logp)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    B.token_logprob_static(H, W, y, logp)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before


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
