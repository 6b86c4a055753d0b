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
    """Token rows for sampled checks: first/last token of the batch and of some sequences, rows on
    128-row tile edges, the last (partial) tile, then seeded random rows."""
    cu = np.asarray(cu, dtype=np.int64)
    rows = {0, T - 1, min(127, T - 1), min(128, T - 1), (T - 1) // 128 * 128}
    lens = np.diff(cu)
    for j in (int(np.argmax(lens)), int(np.argmin(np.where(lens > 0, lens, lens.max() + 1))), 0, len(lens) - 1):
        if lens[j] > 0:
            rows.update({int(cu[j]), int(cu[j + 1] - 1)})
    rng = np.random.default_rng(seed)
    while len(rows) < min(n, T):
        rows.add(int(rng.integers(0, T)))
    return np.array(sorted(rows), dtype=np.int64)
