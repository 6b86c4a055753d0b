"""Helpers shared by the GPU parity tests (device buffers in, numpy out)."""
import numpy as np
import torch

from paper_2507_01663_b200 import workloads as wl

LOGP_TOL = 2e-3      # |delta logp|, |delta entropy|: bf16 inputs, fp32 accumulation
LOSS_RTOL = 1e-3     # relative error of loss scalars
GRAD_RTOL = 1e-2     # relative error of gradient norms
ADV_TOL = 1e-5       # absolute error of advantages


def device():
    return torch.device("cuda:0")


def f32(x):
    return torch.as_tensor(np.asarray(x, dtype=np.float32), device=device())


def i32(x):
    return torch.as_tensor(np.asarray(x, dtype=np.int32), device=device())


def np_of(t):
    return t.detach().cpu().numpy()


def packed_buffers(T_cap, B_cap, d, with_cols=True):
    dev = device()
    out = {"cu_seqlens": torch.full((B_cap + 1,), -7, dtype=torch.int32, device=dev),
           "hidden": torch.zeros(max(T_cap, 1), d, dtype=torch.bfloat16, device=dev)}
    if with_cols:
        out.update(target=torch.full((max(T_cap, 1),), -7, dtype=torch.int32, device=dev),
                   old_logp=torch.zeros(max(T_cap, 1), device=dev),
                   ref_logp=torch.zeros(max(T_cap, 1), device=dev),
                   adv_seq=torch.zeros(max(B_cap, 1), device=dev),
                   seq_id=torch.full((max(T_cap, 1),), -7, dtype=torch.int32, device=dev))
    return out


def rel(a, b):
    return abs(a - b) / max(abs(b), 1e-30)


def sample_rows(cu, T, n, seed):
    """Token rows for sampled checks: first/last token of the batch and of some sequences (the
    longest, the shortest, the first, the last), the rows on either side of the 128-row tile edges
    and of the 256-row edges of a CTA pair's tile, the first and last row of the last (partial)
    128-row and 256-row tile, then seeded random rows up to `n`."""
    cu = np.asarray(cu, dtype=np.int64)
    last128, last256 = (T - 1) // 128 * 128, (T - 1) // 256 * 256
    edges = [0, T - 1, 127, 128, 129, 255, 256, 257, 383, 384, 511, 512, last128 - 1, last128, last128 + 1,
             last256 - 1, last256, last256 + 1]
    rows = {min(max(int(r), 0), T - 1) for r in edges}
    lens = np.diff(cu)
    for j in (int(np.argmax(lens)), int(np.argmin(np.where(lens > 0, lens, lens.max() + 1))), 0, len(lens) - 1):
        if lens[j] > 0:
            rows.update({int(cu[j]), int(cu[j + 1] - 1)})
    rng = np.random.default_rng(seed)
    while len(rows) < min(n, T):
        rows.add(int(rng.integers(0, T)))
    return np.array(sorted(rows), dtype=np.int64)


def off_the_clip_bounds(logp, old, clip_lo, clip_hi, margin=5e-3, shift=0.02):
    """Test-input recipe for chained checks: the kernel takes the clip decision in fp32 from its own
    log-prob (within 2e-3 of the oracle's), the oracle in fp64 from its own.  Where the oracle's
    ratio exp(logp - old) lies within `margin` of a clip bound the two could decide differently, so
    those tokens get their old log-prob moved by `shift` (ratio changes by 2 %), away from the bound.
    Returns the adjusted copy of `old` (float32 values, float64 container)."""
    logp = np.asarray(logp, dtype=np.float64)
    old = np.asarray(old, dtype=np.float32).astype(np.float64).copy()
    for _ in range(2):
        rho = np.exp(logp - old)
        near = (np.abs(rho - (1.0 - clip_lo)) < margin) | (np.abs(rho - (1.0 + clip_hi)) < margin)
        old[near] = (old[near] + shift).astype(np.float32)
    rho = np.exp(logp - old)
    assert not ((np.abs(rho - (1.0 - clip_lo)) < margin) | (np.abs(rho - (1.0 + clip_hi)) < margin)).any()
    return old
