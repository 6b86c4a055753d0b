"""Seeded synthetic workloads for the GRPO scoring path.

This module only *draws inputs*: response lengths, hidden states, LM-head weights, target
tokens, rewards and noise.  It holds none of the method's arithmetic (no softmax, no
advantage, no loss) so that both the CUDA path and the CPU oracle can be fed from it
without sharing any code of the method itself.

Every value is a pure function of ``(seed, stream, element index)``: a SplitMix64 hash of the
counter (Steele, Lea & Flood, "Fast splittable pseudorandom number generators", 2014), so
any row of a multi-GB tensor can be regenerated anywhere without storing it.  The hash is
evaluated with torch integer ops and therefore runs on CPU or on a CUDA device unchanged.

The shapes, length mixes and reward laws follow the five evaluation workloads (Qwen2.5-7B /
32B heads as in the paper's Evaluation, "Experiment Setup"; response lengths with high
variance as in "Load-Balancing Strategies").  They stand in for the paper's DeepScaleR +
Qwen2.5 runs, which need a dataset and trained weights.
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Optional, Sequence

import numpy as np
import torch

# ----------------------------------------------------------------------------------------
# counter-based generator
# ----------------------------------------------------------------------------------------
_MASK64 = (1 << 64) - 1


def _s64(x: int) -> int:
    """Two's-complement view of an unsigned 64-bit constant as a Python int in int64 range."""
    x &= _MASK64
    return x - (1 << 64) if x >= (1 << 63) else x


_GOLDEN = _s64(0x9E3779B97F4A7C15)
_M1 = _s64(0xBF58476D1CE4E5B9)
_M2 = _s64(0x94D049BB133111EB)


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical shift right of int64 lanes (torch's >> is arithmetic)."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def _splitmix64(x: torch.Tensor) -> torch.Tensor:
    z = (x ^ _lsr(x, 30)) * _M1
    z = (z ^ _lsr(z, 27)) * _M2
    return z ^ _lsr(z, 31)


def _stream_key(seed: int, stream: int) -> int:
    """Scalar key for (seed, stream), itself a SplitMix64 finaliser evaluated in Python ints."""
    z = (seed * 0x9E3779B97F4A7C15 + stream * 0xD1B54A32D192ED03 + 0x2545F4914F6CDD1D) & _MASK64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _MASK64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _MASK64
    return _s64(z ^ (z >> 31))


def counter_bits(seed: int, stream: int, start: int, count: int, device="cpu") -> torch.Tensor:
    """64 hash bits for counters ``start .. start+count-1`` of stream ``(seed, stream)``."""
    idx = torch.arange(start, start + count, dtype=torch.int64, device=device)
    return _splitmix64(idx * _GOLDEN + _stream_key(seed, stream))


def uniform01(seed: int, stream: int, start: int, count: int, device="cpu") -> torch.Tensor:
    """float32 uniforms strictly inside (0, 1): (top 24 bits + 0.5) / 2^24."""
    bits = _lsr(counter_bits(seed, stream, start, count, device), 40)
    return (bits.to(torch.float32) + 0.5) * (1.0 / 16777216.0)


def normal01(seed: int, stream: int, start: int, count: int, device="cpu") -> torch.Tensor:
    """float32 standard normals by Box-Muller; element i uses counters 2i and 2i+1."""
    u = uniform01(seed, stream, 2 * start, 2 * count, device).view(count, 2)
    r = torch.sqrt(-2.0 * torch.log(u[:, 0]))
    return r * torch.cos((2.0 * math.pi) * u[:, 1])


def randint(seed: int, stream: int, start: int, count: int, n: int, device="cpu") -> torch.Tensor:
    """int64 integers in [0, n) (n < 2^31) from the top 32 hash bits."""
    hi = _lsr(counter_bits(seed, stream, start, count, device), 32)
    return (hi * n) >> 32


# stream ids (one per tensor)
S_LEN, S_HIDDEN, S_W, S_TARGET, S_REWARD, S_OLD, S_REF, S_ORDER, S_MISC, S_LOGP, S_G = range(1, 12)


# ----------------------------------------------------------------------------------------
# workload description
# ----------------------------------------------------------------------------------------
@dataclasses.dataclass
class Workload:
    """A synthetic sample store: N responses in groups of G, response i has ``lengths[i]`` rows."""

    name: str
    seed: int
    d: int
    V: int
    n_prompts: int
    group_size: int
    lengths: np.ndarray                 # [N] int64
    reward_law: str                     # "bernoulli:<p>" | "uniform"
    clip_eps: float = 0.2
    kl_coef: float = 0.04
    noise_std: float = 0.1
    hidden_std: float = 1.0
    w_std: float = 0.02
    token_budget: Optional[int] = None  # streaming micro-batch budget (None: one batch)
    backward: bool = False

    @property
    def N(self) -> int:
        return self.n_prompts * self.group_size

    @property
    def tok_offset(self) -> np.ndarray:
        off = np.zeros(self.N + 1, dtype=np.int64)
        np.cumsum(self.lengths, out=off[1:])
        return off

    @property
    def total_tokens(self) -> int:
        return int(self.lengths.sum())

    @property
    def group_id(self) -> np.ndarray:
        """Sample i answers prompt i // G (the store is indexed prompt-major)."""
        return (np.arange(self.N, dtype=np.int64) // self.group_size).astype(np.int32)


def _uniform_lengths(seed, n, lo, hi):
    return (randint(seed, S_LEN, 0, n, hi - lo + 1) + lo).numpy().astype(np.int64)


def _lognormal_lengths(seed, n, median, sigma, lo, hi):
    z = normal01(seed, S_LEN, 0, n).double()
    L = torch.round(torch.exp(math.log(median) + sigma * z)).clamp(lo, hi)
    return L.numpy().astype(np.int64)


def _pareto_lengths(seed, n, x_m, alpha, cap):
    u = uniform01(seed, S_LEN, 0, n).double()
    L = torch.floor(x_m * (1.0 - u) ** (-1.0 / alpha)).clamp(x_m, cap)
    return L.numpy().astype(np.int64)


def _fixed_total_lengths(seed, n, lo, hi, total):
    """n lengths drawn uniform in [lo, hi], rescaled to sum exactly to ``total`` inside [lo, hi]."""
    L = _uniform_lengths(seed, n, lo, hi).astype(np.float64)
    L = np.clip(np.rint(L * (total / L.sum())), lo, hi).astype(np.int64)
    i = 0
    while L.sum() != total:
        step = 1 if L.sum() < total else -1
        if lo <= L[i % n] + step <= hi:
            L[i % n] += step
        i += 1
    return L


def make_workload(name: str, seed_offset: int = 0) -> Workload:
    """The five evaluation workloads (``cfg1`` .. ``cfg5``) and reduced test variants (``*_mini``).

    ``cfg2_mid`` and ``cfg4_mid`` are profiling-sized forward and actor-update batches (a few GB on the device).  Mini variants keep the structure (group sizes, length law, ragged tails) at sizes a CPU
    oracle evaluates in seconds; their V is deliberately not a multiple of the GEMM tile.
    ``seed_offset`` derives an independent draw of the same shape (one per data-parallel rank).
    """
    base = {"cfg1": 0, "cfg2": 1, "cfg3": 2, "cfg4": 3, "cfg5": 4,
            "cfg2_mini": 11, "cfg3_mini": 12, "cfg4_mini": 13, "cfg5_mini": 14, "cfg4_mid": 23, "cfg2_mid": 21}
    if name not in base:
        raise KeyError(name)
    sd = base[name] + seed_offset
    if name == "cfg1":
        return Workload(name, sd, 256, 4096, 8, 4, _uniform_lengths(sd, 32, 16, 64), "bernoulli:0.5")
    if name == "cfg2":
        return Workload(name, sd, 3584, 152064, 64, 8, _uniform_lengths(sd, 512, 256, 4096), "bernoulli:0.3")
    if name == "cfg3":
        return Workload(name, sd, 5120, 152064, 32, 16, _lognormal_lengths(sd, 512, 1024, 1.0, 64, 8192), "uniform")
    if name == "cfg4":
        return Workload(name, sd, 3584, 152064, 16, 8, _fixed_total_lengths(sd, 128, 64, 1024, 65536),
                        "bernoulli:0.5", backward=True)
    if name == "cfg5":
        return Workload(name, sd, 3584, 152064, 64, 64, _pareto_lengths(sd, 4096, 128, 1.5, 16384),
                        "bernoulli:0.3", token_budget=32768)
    if name == "cfg2_mid":   # the 7B head on a profiling-sized forward batch (about 65 k tokens, a few GB on the device)
        return Workload(name, sd, 3584, 152064, 4, 8, _uniform_lengths(sd, 32, 1024, 3072), "bernoulli:0.3")
    if name == "cfg4_mid":   # one backward token block at the 7B hidden size, a quarter-size vocabulary
        return Workload(name, sd, 3584, 32768, 2, 8, _fixed_total_lengths(sd, 16, 64, 1024, 9472),
                        "bernoulli:0.5", backward=True)
    if name == "cfg2_mini":
        return Workload(name, sd, 512, 8200, 8, 8, _uniform_lengths(sd, 64, 32, 300), "bernoulli:0.3")
    if name == "cfg3_mini":
        return Workload(name, sd, 640, 5000, 4, 16, _lognormal_lengths(sd, 64, 96, 1.0, 8, 700), "uniform")
    if name == "cfg4_mini":
        return Workload(name, sd, 512, 8192, 4, 8, _fixed_total_lengths(sd, 32, 8, 64, 1024),
                        "bernoulli:0.5", backward=True)
    return Workload(name, sd, 256, 4104, 8, 16, _pareto_lengths(sd, 128, 8, 1.5, 512),
                    "bernoulli:0.3", token_budget=1024)


# ----------------------------------------------------------------------------------------
# tensors of a workload
# ----------------------------------------------------------------------------------------
_CHUNK = 1 << 24


def _normal_matrix(seed, stream, rows, cols, std, device, row_start=0) -> torch.Tensor:
    """bf16 [rows, cols] with element (r, c) = std * normal(counter (row_start + r) * cols + c)."""
    out = torch.empty((rows, cols), dtype=torch.bfloat16, device=device)
    flat = out.view(-1)
    base = row_start * cols
    total = rows * cols
    for s in range(0, total, _CHUNK):
        n = min(_CHUNK, total - s)
        flat[s:s + n] = (normal01(seed, stream, base + s, n, device) * std).to(torch.bfloat16)
    return out


def gen_hidden(w: Workload, device="cpu", row_start: int = 0, rows: Optional[int] = None) -> torch.Tensor:
    """Store column ``hidden`` [sum L, d] bf16 (or the row range ``row_start .. row_start+rows``)."""
    rows = w.total_tokens - row_start if rows is None else rows
    return _normal_matrix(w.seed, S_HIDDEN, rows, w.d, w.hidden_std, device, row_start)


def gen_hidden_rows(w: Workload, rows: Sequence[int], device="cpu") -> torch.Tensor:
    """Regenerate the given store rows of ``hidden`` (any order) without building the column."""
    return torch.cat([gen_hidden(w, device, int(r), 1) for r in rows], 0)


def gen_weight(w: Workload, device="cpu") -> torch.Tensor:
    """LM-head weight [V, d] bf16, one row per vocabulary id."""
    return _normal_matrix(w.seed, S_W, w.V, w.d, w.w_std, device)


def gen_target(w: Workload, device="cpu", row_start: int = 0, rows: Optional[int] = None) -> torch.Tensor:
    """Store column ``target`` [sum L] int32, uniform over the vocabulary (or the given row range)."""
    rows = w.total_tokens - row_start if rows is None else rows
    return randint(w.seed, S_TARGET, row_start, rows, w.V, device).to(torch.int32)


def gen_reward(w: Workload, device="cpu") -> torch.Tensor:
    """Per-response reward [N] float32."""
    u = uniform01(w.seed, S_REWARD, 0, w.N, device)
    if w.reward_law == "uniform":
        return u
    p = float(w.reward_law.split(":")[1])
    return (u < p).to(torch.float32)


def gen_noise(w: Workload, stream: int, count: int, device="cpu", start: int = 0) -> torch.Tensor:
    """float32 N(0, noise_std^2) draws (streams S_OLD / S_REF perturb the current log-probs)."""
    return normal01(w.seed, stream, start, count, device) * w.noise_std


def gen_surrogate_logp(w: Workload, count: int, device="cpu") -> torch.Tensor:
    """Stand-in per-token log-probs for stage-isolated loss checks at sizes where no CPU
    scorer is affordable: -(ln V + |N(0,1.5)|), the magnitude a random head produces."""
    return -(math.log(w.V) + torch.abs(normal01(w.seed, S_LOGP, 0, count, device)) * 1.5)


def arrival_order(w: Workload) -> np.ndarray:
    """Seeded permutation of the sample indices: the order in which responses arrive."""
    keys = counter_bits(w.seed, S_ORDER, 0, w.N)
    return torch.argsort(keys, stable=True).numpy().astype(np.int32)


def microbatches(w: Workload, order: Optional[np.ndarray] = None) -> List[np.ndarray]:
    """Greedy arrival-ordered micro-batches: append the next response while the running token
    total stays within ``token_budget`` (a response longer than the budget forms its own batch)."""
    order = arrival_order(w) if order is None else order
    if w.token_budget is None:
        return [np.asarray(order, dtype=np.int32)]
    out, cur, tot = [], [], 0
    for i in order:
        L = int(w.lengths[i])
        if cur and tot + L > w.token_budget:
            out.append(np.asarray(cur, dtype=np.int32))
            cur, tot = [], 0
        cur.append(int(i))
        tot += L
    if cur:
        out.append(np.asarray(cur, dtype=np.int32))
    return out


def shard_prompts(n_prompts: int, world_size: int, rank: int) -> range:
    """Data-parallel split by prompt: whole groups stay on one rank so that group statistics
    need no exchange.  Rank r owns prompts [r*n/W, (r+1)*n/W)."""
    lo = (n_prompts * rank) // world_size
    hi = (n_prompts * (rank + 1)) // world_size
    return range(lo, hi)


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """Raw bf16 bit patterns of a tensor as a numpy uint16 array (numpy has no bf16 dtype)."""
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def centre_logp_estimate(w: Workload, hidden: torch.Tensor, weight: torch.Tensor,
                         target: torch.Tensor, chunk: int = 1 << 16) -> torch.Tensor:
    """A cheap stand-in for "the current log-prob" used only to centre synthetic old / ref
    log-probs where scoring every token on the CPU is out of reach: the target logit (one dot
    product per token) minus the Gaussian estimate ln V + |h|^2 w_std^2 / 2 of the normaliser a
    random head produces.  Inputs are perturbed around it by ``gen_noise``; nothing is checked
    against it."""
    out = torch.empty(hidden.shape[0], dtype=torch.float32, device=hidden.device)
    for s in range(0, hidden.shape[0], chunk):
        h = hidden[s:s + chunk].float()
        zy = (h * weight[target[s:s + chunk].long()].float()).sum(1)
        out[s:s + chunk] = zy - (math.log(w.V) + 0.5 * (w.w_std ** 2) * (h * h).sum(1))
    return out
