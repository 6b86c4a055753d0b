#!/usr/bin/env python
"""Benchmark of the GRPO scoring hot path on B200.

One *step* = one pass of the whole path over one synthetic batch shaped like the Qwen2.5-7B
workload (512 responses, ~1.1 M scored tokens): group advantages -> pack by sample index ->
fused LM-head log-prob / entropy -> clipped policy loss + k3 KL (with dL/dlogp).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload cfg2]

Prints ONE JSON line (rank 0).  ``value`` is scored tokens/s over all ranks with the inputs
resident in HBM; ``e2e`` is the same metric with the store columns starting in pinned host
memory: every step's host->device copies (on a second stream, into the device copy the previous
step is not reading) and the device->host read of the step's results (per-token log-probs and the
loss record) are inside the timed region.  With the default workload on one GPU the line also
carries ``configs``: short timed legs of the other four workloads (cfg1, cfg3, cfg4, cfg5).
``--gpus N`` (N > 1) without a launcher's RANK in the environment starts N ranks itself, one per
GPU, through ``torch.distributed.run``.  ``--impl reference`` times the fp64 CPU oracle on a
bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import ctypes
import json
import os
import socket
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2507_01663_b200 import workloads as wl  # noqa: E402

METRIC = "scored tokens/sec (logprob+GRPO loss) at Qwen-7B head; % dense-BF16 peak"
UNIT = "tokens/s"
KERNELS_PER_MICROBATCH = 4  # pack (rows by bulk copy + the 4-byte columns), fused LM-head GEMM, partial merge, loss
PACK_INLINE_SEQS = 512      # beyond this many sequences a pack also launches the fetch of its sequence table
# DRAM bytes per scored token of the fused LM-head kernel (dram__bytes_read of one ncu capture of the
# CTA-pair kernel, row tiles dealt by die, two vocabulary ranges -- what the library picks at the
# bench size -- on `--workload cfg2_mid --v-splits 2`: T = 62989, d = 3584, V = 152064; 8.306 and
# 8.838 GB for two launches on a part with 70 + 78 SMs per die, 8.46-8.47 GB on one with 72 + 76; writes
# are 7-10 MB; traffic grows with the number of waves of row tiles, i.e. in proportion to T).  Valid
# for the 7B head shape and the default kernel only; None whenever the kernel or its work
# decomposition has changed since the counters were taken.
GEMM_DRAM_BYTES_PER_TOKEN_7B = (8.572e9 + 8.5e6) / 62989
BWD_TOKEN_BLOCK = 9472  # the library's default backward block (3 GEMM launches per block)


# ------------------------------------------------------------------------------------------
# helpers
# ------------------------------------------------------------------------------------------
def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.QUERY}",
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._pump, daemon=True).start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def head_name(w) -> str:
    return {(3584, 152064): "Qwen2.5-7B-shaped", (5120, 152064): "Qwen2.5-32B-shaped"}.get((w.d, w.V), "synthetic")


# Set by --dp-single-rank: run the data-parallel exchanges (reward all-gather, overlapped dW
# all-reduce) through a process group of ONE rank, so that their code path -- NCCL calls, streams,
# events -- runs on a single GPU.
EXCHANGE_WITH_ONE_RANK = False


def exchanging(world: int) -> bool:
    return world > 1 or EXCHANGE_WITH_ONE_RANK


def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def rank_workload(name: str, rank: int) -> wl.Workload:
    """Draw number `rank` of a workload: the same shape, its own seed (own lengths and values)."""
    return wl.make_workload(name, seed_offset=1000 * rank)


class DataParallelShare:
    """One rank's share of a data-parallel step (Section 4.1: the batch is streamed to the DP groups
    of a task; Section 4.4, last paragraph: the controller gives every DP group the same number of
    samples and balances their token totals with Karmarkar-Karp).

    The global batch is `world` draws of the workload (weak scaling: the per-GPU work stays fixed).
    Its responses are dealt to the ranks by af_balance_partitions with equal sample counts, so the
    responses to one prompt end up on different ranks; each rank therefore contributes the rewards
    of its own responses to one all-gather, computes the group-normalised advantages of the whole
    batch from the gathered vector (group ids in arbitrary order) and keeps its own slice.  The
    metadata (lengths, group ids, the partition) is computed by every rank alike from the seeds;
    hidden states, targets and rewards are generated only for the rank's own responses.
    """

    def __init__(self, name: str, world: int, rank: int, balance: bool = True):
        self.name, self.world, self.rank = name, world, rank
        self.sources = [rank_workload(name, s) for s in range(world)]
        w0 = self.sources[0]
        self.n_per_source = w0.N
        self.lengths = np.concatenate([w.lengths for w in self.sources]).astype(np.int64)
        self.source = np.repeat(np.arange(world), w0.N)
        self.local_index = np.tile(np.arange(w0.N), world)
        self.group_id = (self.source * w0.n_prompts + self.local_index // w0.group_size).astype(np.int32)
        self.n_groups = world * w0.n_prompts
        self.N_global = world * w0.N
        contiguous = np.repeat(np.arange(world), w0.N).astype(np.int32)      # dealt by prompt index
        if balance and world > 1:
            from paper_2507_01663_b200 import binding as B
            part, _ = B.balance_partitions(self.lengths.astype(np.int32), world, True)
        else:
            part = contiguous
        self.part = np.asarray(part, dtype=np.int32)
        self.tokens_per_rank = np.bincount(self.part, weights=self.lengths, minlength=world).astype(np.int64)
        self.tokens_per_rank_by_prompt = np.bincount(contiguous, weights=self.lengths, minlength=world).astype(np.int64)
        # responses of rank r in increasing global index; all ranks' lists back to back = the order of
        # the gathered reward vector
        self.members = [np.nonzero(self.part == r)[0] for r in range(world)]
        counts = {len(m) for m in self.members}
        if len(counts) != 1:
            raise RuntimeError(f"ranks got unequal sample counts {sorted(counts)}")
        self.mine = self.members[rank]
        self.gathered_order = np.concatenate(self.members)
        self.gathered_group_id = self.group_id[self.gathered_order].astype(np.int32)
        self.n_mine = len(self.mine)
        self.loss_scale = self.n_mine / self.N_global        # B_rank / B_global: rank losses and gradients add up

    def rank_view(self) -> wl.Workload:
        """The rank's responses as a workload of their own (lengths only; group structure lives here)."""
        w0 = self.sources[0]
        import dataclasses
        return dataclasses.replace(w0, lengths=self.lengths[self.mine].copy(), seed=w0.seed + 7919 * (self.rank + 1))

    def build_columns(self, device):
        """hidden / target rows and rewards of the rank's own responses, from their sources' generators."""
        H, y, r = [], [], []
        rewards = [wl.gen_reward(w).numpy() for w in self.sources]
        for g in self.mine:
            w, i = self.sources[self.source[g]], int(self.local_index[g])
            off = w.tok_offset
            H.append(wl.gen_hidden(w, device, int(off[i]), int(off[i + 1] - off[i])))
            y.append(wl.gen_target(w, device, int(off[i]), int(off[i + 1] - off[i])))
            r.append(rewards[self.source[g]][i])
        return torch.cat(H, 0), torch.cat(y, 0), torch.as_tensor(np.asarray(r, dtype=np.float32), device=device)

    def gather_rewards(self, mine: torch.Tensor) -> torch.Tensor:
        """All ranks' reward slices back to back (rank-major): 4 bytes per response cross the links."""
        if not exchanging(self.world):
            return mine
        import torch.distributed as dist
        out = torch.empty(self.N_global, dtype=mine.dtype, device=mine.device)
        dist.all_gather_into_tensor(out, mine.contiguous())
        return out

    def report(self) -> dict:
        t, b = self.tokens_per_rank, self.tokens_per_rank_by_prompt
        return {"ranks": self.world, "responses_per_rank": int(self.n_mine), "tokens_per_rank": [int(x) for x in t],
                "token_spread_balanced": int(t.max() - t.min()), "token_spread_by_prompt_index": int(b.max() - b.min()),
                "how": "af_balance_partitions (Karmarkar-Karp, equal sample counts) over the global batch; rewards "
                       "all-gathered, advantages by group id on every rank"}


def reduce_over_ranks(ms_local: float, tokens_local: int, world: int):
    """(max over ranks of the step time, sum over ranks of the tokens)."""
    if world == 1:
        return ms_local, tokens_local
    import torch.distributed as dist
    dev = torch.device("cuda", torch.cuda.current_device()) if dist.get_backend() == "nccl" else torch.device("cpu")
    t = torch.tensor([ms_local], dtype=torch.float64, device=dev)
    n = torch.tensor([tokens_local], dtype=torch.int64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(n, op=dist.ReduceOp.SUM)
    return float(t.item()), int(n.item())


def allreduce_sum_(t: torch.Tensor, world: int) -> torch.Tensor:
    """Actor update under data parallelism: every rank scores its own prompts with
    loss_scale = B_rank / B_global, so the weight gradients of the ranks ADD UP to the gradient of
    the global batch; the one exchange of the path is this sum (NCCL on GPUs, gloo in CPU tests)."""
    if exchanging(world):
        import torch.distributed as dist
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return t


def vocab_shard(V: int, world: int, rank: int):
    """Rows [lo, hi) of the LM head held by `rank` under vocabulary parallelism (multiples of 8)."""
    per = -(-V // world)
    per = -(-per // 8) * 8
    return min(rank * per, V), min((rank + 1) * per, V)


def allgather_partials(mine: torch.Tensor, world: int) -> torch.Tensor:
    """The one exchange of vocabulary-parallel scoring: every rank contributes its [T, 4] shard
    statistics (16 bytes per token) and receives all of them as [R, T, 4]."""
    if world == 1:
        return mine.unsqueeze(0)
    import torch.distributed as dist
    out = torch.empty((world,) + tuple(mine.shape), dtype=mine.dtype, device=mine.device)
    dist.all_gather(list(out.unbind(0)), mine.contiguous())     # the slices are contiguous views of `out`
    return out


# ------------------------------------------------------------------------------------------
# the CUDA arm
# ------------------------------------------------------------------------------------------
class ScoringJob:
    """Device buffers of one rank and the step function that runs the path through the C ABI."""

    def __init__(self, w: wl.Workload, device: torch.device, gemm_variant: int = 0, world: int = 1, v_splits: int = 0,
                 vocab_parallel: bool = False, rank: int = 0, bwd_token_block: int = 0,
                 dp: "DataParallelShare | None" = None):
        from paper_2507_01663_b200 import binding as B
        self.B, self.dev, self.world, self.rank, self.dp = B, device, world, rank, dp
        self.ctx = B.Context(device.index or 0)
        self.ctx.set_tuning(v_splits, bwd_token_block, gemm_variant)
        if dp is not None:
            # this rank's token-balanced share of the global batch; the head is replicated
            w = dp.rank_view()
            hidden, target, self.reward = dp.build_columns(device)
            self.store = {"hidden": hidden, "target": target}
            self.W = wl.gen_weight(dp.sources[0], device)
            self.gid = torch.as_tensor(dp.gathered_group_id, device=device)
            self.adv_all = torch.empty(dp.N_global, device=device)
        else:
            self.store = {"hidden": wl.gen_hidden(w, device), "target": wl.gen_target(w, device)}
            self.W = wl.gen_weight(w, device)
            self.reward = wl.gen_reward(w, device)
        self.w = w
        T = w.total_tokens
        self.T = T
        self.vocab_parallel = vocab_parallel
        # data parallel: the rank's batch weighs B_rank / B_global; vocabulary parallel: one batch
        self.loss_scale = 1.0 if vocab_parallel else (dp.loss_scale if dp is not None else 1.0 / world)
        self.v_lo, self.v_hi = vocab_shard(w.V, world, rank) if vocab_parallel else (0, w.V)
        centre = wl.centre_logp_estimate(w, self.store["hidden"], self.W, self.store["target"])
        self.store["old_logp"] = centre + wl.gen_noise(w, wl.S_OLD, T, device)
        self.store["ref_logp"] = centre + wl.gen_noise(w, wl.S_REF, T, device)
        del centre
        self.adv = self.adv_all[rank * dp.n_mine:(rank + 1) * dp.n_mine] if dp is not None else torch.empty(w.N, device=device)
        # micro-batches: the whole arrival-ordered batch, or (streaming store) greedy arrival-ordered
        # index lists under the workload's token budget, issued back to back on one stream
        self.mbs = wl.microbatches(w)
        self.idx = self.mbs[0]
        self.off = w.tok_offset
        cap_T = max(int(w.lengths[m].sum()) for m in self.mbs)
        cap_B = max(len(m) for m in self.mbs)
        self.packed = {
            "cu_seqlens": torch.zeros(cap_B + 1, dtype=torch.int32, device=device),
            "hidden": torch.empty(cap_T, w.d, dtype=torch.bfloat16, device=device),
            "target": torch.empty(cap_T, dtype=torch.int32, device=device),
            "old_logp": torch.empty(cap_T, device=device), "ref_logp": torch.empty(cap_T, device=device),
            "adv_seq": torch.empty(cap_B, device=device),
        }
        self.logp, self.ent, self.lse, self.dlogp = (torch.empty(cap_T, device=device) for _ in range(4))
        if vocab_parallel:     # this rank keeps only its rows of the head; statistics are exchanged per micro-batch
            self.W_shard = self.W[self.v_lo:self.v_hi].contiguous()
            self.partial = torch.empty(cap_T, 4, device=device)
        self.loss_outs = [B.new_loss_out(device) for _ in self.mbs]
        self.loss_out = self.loss_outs[-1]
        self.overlap_dw = False
        if w.backward:
            self.d_hidden = torch.empty(cap_T, w.d, dtype=torch.bfloat16, device=device)
            self.d_W = torch.empty(w.V, w.d, device=device)
            if exchanging(world) and not vocab_parallel:
                # the gradient all-reduce runs on its own stream, started by the event the backward
                # records as soon as d_W is complete (its last block runs the dW product first)
                self.overlap_dw = True
                self.comm_stream = torch.cuda.Stream()
                self.dw_ready, self.dw_reduced = torch.cuda.Event(), torch.cuda.Event()
                self.dw_ready.record()
                self.dw_reduced.record()
                self.ctx.set_dw_ready_event(self.dw_ready)
        self.e2e_logp_host = None
        self.ctx.reserve(cap_T, cap_B, w.d, w.V, with_backward=2 if w.backward else False)
        self.gemm_events, self.pack_events, self.bwd_events = [], [], []
        per_mb = KERNELS_PER_MICROBATCH + (3 * -(-cap_T // BWD_TOKEN_BLOCK) if w.backward else 0)
        self.launches_per_step = (1 + per_mb * len(self.mbs)                      # 1: the advantage kernel
                                  + sum(len(mb) > PACK_INLINE_SEQS for mb in self.mbs))

    def advantages(self, reward=None):
        """Group-normalised advantages of this rank's responses (into self.adv)."""
        w, c = self.w, self.ctx
        reward = self.reward if reward is None else reward
        if self.dp is None:
            c.grpo_advantage(reward, None, w.n_prompts, self.adv)
        else:
            # groups are spread over the ranks: gather every rank's rewards, normalise the whole
            # batch by group id, keep the own slice (self.adv is a view of it)
            c.grpo_advantage(self.dp.gather_rewards(reward), self.gid, self.dp.n_groups, self.adv_all)

    def sum_dW_over_ranks(self):
        """The one exchange of a data-parallel actor update.  With the overlap set up, the all-reduce
        waits for the backward's "d_W complete" event on the communication stream and runs beside
        the last block's dH product; the compute stream waits for it only before d_W is next written."""
        if not exchanging(self.world):
            return
        if not self.overlap_dw:
            allreduce_sum_(self.d_W, self.world)
            return
        with torch.cuda.stream(self.comm_stream):
            self.comm_stream.wait_event(self.dw_ready)
            allreduce_sum_(self.d_W, self.world)
            self.dw_reduced.record(self.comm_stream)

    def step(self, time_gemm: bool = False, store_cols=None, reward=None):
        w, c = self.w, self.ctx
        self.advantages(reward)
        store = {"tok_offset_host": self.off, "d": w.d, "adv": self.adv, **(self.store if store_cols is None else store_cols)}
        total = 0
        for mb, loss_out in zip(self.mbs, self.loss_outs):
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(6)] if time_gemm else None
            if ev:
                ev[0].record()
            T = c.pack_microbatch(store, mb, self.packed)
            if ev:
                ev[1].record()
                ev[2].record()
            if self.vocab_parallel:
                c.token_logprob_shard(self.packed["hidden"], self.W_shard, self.packed["target"], self.v_lo,
                                      self.partial, T=T)
                gathered = allgather_partials(self.partial[:T], self.world)
                c.merge_logprob_shards(gathered, self.packed["target"], w.V, self.logp, self.ent, self.lse, T=T)
            else:
                c.token_logprob(self.packed["hidden"], self.W, self.packed["target"], self.logp, self.ent, self.lse, T=T)
            if ev:
                ev[3].record()
            c.policy_loss(self.logp, self.packed["old_logp"], self.packed["ref_logp"], self.packed["adv_seq"],
                          self.packed["cu_seqlens"], loss_out, self.dlogp, self.ent,
                          w.clip_eps, w.clip_eps, w.kl_coef, 0, self.loss_scale, B=len(mb), T=T)
            if self.e2e_logp_host is not None:      # end-to-end steps return the task's result to the host
                self.e2e_logp_host[total:total + T].copy_(self.logp[:T], non_blocking=True)
            if w.backward:
                if ev:
                    ev[4].record()
                if self.overlap_dw:
                    torch.cuda.current_stream().wait_event(self.dw_reduced)   # the previous sum has read d_W
                if self.vocab_parallel:
                    # this rank's rows of dW stay here; the ranks' contributions to dH are summed
                    c.policy_loss_backward_shard(self.packed["hidden"], self.W_shard, self.packed["target"], self.lse,
                                                 self.dlogp, self.v_lo, self.d_hidden, self.d_W[self.v_lo:self.v_hi],
                                                 False, T=T)
                else:
                    c.policy_loss_backward(self.packed["hidden"], self.W, self.packed["target"], self.lse, self.dlogp,
                                           self.d_hidden, self.d_W, False, T=T)
                if ev:
                    ev[5].record()
                    self.bwd_events.append((ev[4], ev[5]))
                if self.vocab_parallel:
                    allreduce_sum_(self.d_hidden[:T], self.world)
                else:
                    self.sum_dW_over_ranks()
            if ev:
                self.pack_events.append((ev[0], ev[1]))
                self.gemm_events.append((ev[2], ev[3]))
            total += T
        return total

    def hbm_kernels_at_scale(self, peak_gbs: float, log2_n: int = 28) -> dict:
        """The memory-bound kernels timed alone, before the long GEMM loop heats the part (the
        condition the measured copy bandwidth was taken under): pack at the workload's own size,
        loss, advantage and the controller's scan at 2^log2_n tokens / responses / samples, where
        bandwidth rather than launch latency decides (the default, 2^28, moves 2-5 GB per call like the
        4 GB copy that defines the measured peak; at 2^26 the same kernels read 3-7 % lower, and so
        does a plain copy of that size)."""
        dev, c, B = self.dev, self.ctx, self.B
        out = {}

        def avg_ms(fn, n=10):
            for _ in range(3):
                fn()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(n):
                fn()
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) / n

        w = self.w
        store = {"tok_offset_host": self.off, "d": w.d, "adv": self.adv, **self.store}
        ms = avg_ms(lambda: c.pack_microbatch(store, self.idx, self.packed))
        t_mb = int(w.lengths[self.idx].sum())
        nbytes = 2.0 * t_mb * (2 * w.d + 12) + 8.0 * len(self.idx)
        gbs = nbytes / ms / 1e6
        out["pack_microbatch"] = {"tokens": t_mb, "bytes_per_token": 2 * (2 * w.d + 12), "ms": ms, "gbs": gbs,
                                  "frac": gbs / peak_gbs, "where": "timed alone, 10 calls (one launch each up to 512 sequences, else table fetch + gather)"}
        # results written back by the same index list: 4 B read + 4 B written per token of one column
        col = torch.empty(int(self.off[-1]), device=dev)
        ms = avg_ms(lambda: c.unpack_microbatch(self.off, self.idx, [self.logp], [col]))
        out["unpack_microbatch"] = {"tokens": t_mb, "bytes_per_token": 8, "ms": ms, "gbs": 8.0 * t_mb / ms / 1e6,
                                    "where": "one log-prob column of the same micro-batch back to the store; "
                                             "launch-bound at this size (2 kernels + metadata copy)"}
        del col
        n = 1 << log2_n
        seq = 1024
        logp = wl.gen_surrogate_logp(self.w, 1 << 20, dev).repeat(n >> 20)
        old, ref, ent = logp + 0.1, logp - 0.1, -logp
        adv = wl.normal01(self.w.seed, wl.S_MISC, 0, n // seq, dev)
        cu = torch.arange(n // seq + 1, device=dev, dtype=torch.int32) * seq
        g, lo = torch.empty(n, device=dev), B.new_loss_out(dev)
        ms = avg_ms(lambda: c.policy_loss(logp, old, ref, adv, cu, lo, g, ent))
        gbs = 20.0 * n / ms / 1e6
        out["policy_loss"] = {"tokens": n, "bytes_per_token": 20, "ms": ms, "gbs": gbs, "frac": gbs / peak_gbs}
        del logp, old, ref, ent, g
        r = wl.uniform01(self.w.seed, wl.S_REWARD, 0, 1 << 20, dev).repeat(n >> 20)
        a = torch.empty(n, device=dev)
        G = self.w.group_size
        ms = avg_ms(lambda: c.grpo_advantage(r, None, n // G, a))
        gbs = 8.0 * n / ms / 1e6
        out["grpo_advantage"] = {"responses": n, "group_size": G, "bytes_per_response": 8, "ms": ms, "gbs": gbs,
                                 "frac": gbs / peak_gbs}
        # the same call with membership by group id (any order): exact fixed-point sums with integer
        # atomics, four streaming passes; ids in index order (a warp's lanes share groups and combine
        # before the atomics) and ids drawn at random (every atomic lands on its own line of a table
        # larger than L2)
        n_id = min(n, 1 << 26)
        for label, ids in (("ids_in_order", (torch.arange(n_id, device=dev, dtype=torch.int32) // G)),
                           ("ids_shuffled", wl.randint(self.w.seed, wl.S_MISC, 0, n_id, n_id // G, dev).to(torch.int32))):
            ms = avg_ms(lambda: c.grpo_advantage(r[:n_id], ids, n_id // G, a[:n_id]), n=5)
            gbs = 36.0 * n_id / ms / 1e6
            out["grpo_advantage_" + label] = {"responses": n_id, "groups": n_id // G, "bytes_per_response": 36, "ms": ms,
                                              "gbs": gbs, "frac": gbs / peak_gbs,
                                              "bound": "integer atomics on a table of 64 B per group (537 MB here, beyond "
                                                       "L2): read-modify-write of accumulator lines, not streaming; "
                                                       "microseconds at workload sizes (N <= 4096)"}
        del r, a, ids
        # controller: one read request against a 2^log2_n-sample status table (12 B read per sample:
        # ready, consumed, length) that hands out the first 4096 eligible samples
        tab = {"ready": torch.ones(n, dtype=torch.int32, device=dev),
               "consumed": torch.zeros(n, dtype=torch.int32, device=dev),
               "length": torch.full((n,), 300, dtype=torch.int32, device=dev)}
        tab["ready"][: n - 100000] = 0          # the eligible samples sit at the far end of the table
        out_idx, res = torch.empty(4096, dtype=torch.int32, device=dev), B.new_get_result(dev)

        def get_once():
            c.controller_get(tab, 1, 1, 4096, 1 << 20, out_idx, res)
            c.controller_clear(tab, 0, 1)       # hand the same samples out again next time

        ms_pair = avg_ms(get_once)
        ms_clear = avg_ms(lambda: c.controller_clear(tab, 0, 1))
        ms = ms_pair - ms_clear
        gbs = 12.0 * n / ms / 1e6
        out["controller_get"] = {"samples": n, "bytes_per_sample": 12, "ms": ms, "gbs": gbs, "frac": gbs / peak_gbs,
                                 "returned": B.read_get_result(res)["count"],
                                 "clear": {"ms": ms_clear, "bytes_per_sample": 8, "gbs": 8.0 * n / ms_clear / 1e6},
                                 "where": "2 launches (count, select); time of a get + clear pair minus a clear"}
        return out

    def balance_report(self) -> dict:
        """Token balancing of the workload's responses over 8 data-parallel groups (host call):
        spread of the groups' token totals against dealing the responses out in arrival order."""
        w, B = self.w, self.B
        L = w.lengths.astype(np.int32)
        k = 8
        t0 = time.perf_counter()
        part, sums = B.balance_partitions(L, k, True)
        ms_dp = 1e3 * (time.perf_counter() - t0)
        t0 = time.perf_counter()
        _, sums_pp = B.balance_partitions(L, k, False)
        ms_pp = 1e3 * (time.perf_counter() - t0)
        order = wl.arrival_order(w)
        rr = np.zeros(k, dtype=np.int64)
        np.add.at(rr, np.arange(w.N) % k, w.lengths[order])
        return {"groups": k, "samples": int(w.N), "host_ms_equal_counts": ms_dp, "host_ms_free_counts": ms_pp,
                "token_spread_arrival_order": int(rr.max() - rr.min()),
                "token_spread_equal_counts": int(sums.max() - sums.min()),
                "token_spread_free_counts": int(sums_pp.max() - sums_pp.min()),
                "mean_tokens_per_group": float(sums.mean())}

    # -- actor update in one call ------------------------------------------------------------
    def step_fused_update(self):
        """advantage -> pack -> af_policy_update (forward + loss + backward, logits evaluated once)."""
        w, c = self.w, self.ctx
        self.advantages()
        store = {"tok_offset_host": self.off, "d": w.d, "adv": self.adv, **self.store}
        total = 0
        for mb, loss_out in zip(self.mbs, self.loss_outs):
            T = c.pack_microbatch(store, mb, self.packed)
            if self.overlap_dw:
                torch.cuda.current_stream().wait_event(self.dw_reduced)
            c.policy_update(self.packed["hidden"], self.W, self.packed["target"], self.packed["old_logp"],
                            self.packed["ref_logp"], self.packed["adv_seq"], self.packed["cu_seqlens"], loss_out,
                            self.logp, self.lse, self.d_hidden, self.d_W, entropy=self.ent, dlogp=self.dlogp,
                            clip_lo=w.clip_eps, clip_hi=w.clip_eps, kl_coef=w.kl_coef, loss_scale=self.loss_scale,
                            B=len(mb), T=T)
            self.sum_dW_over_ranks()
            total += T
        return total

    # -- streaming with the controller in the loop ------------------------------------------
    def make_live_controller(self, wave: int = 512):
        """Status table beside the store; responses become ready in arrival order, `wave` at a time."""
        w, dev, B = self.w, self.dev, self.B
        self.tab = {"ready": torch.zeros(w.N, dtype=torch.int32, device=dev),
                    "consumed": torch.zeros(w.N, dtype=torch.int32, device=dev),
                    "length": torch.as_tensor(w.lengths.astype(np.int32), device=dev)}
        self.arrival_dev = torch.as_tensor(wl.arrival_order(w).astype(np.int32), device=dev)
        self.wave = wave
        self.req_idx = [torch.empty(w.N, dtype=torch.int32, device=dev) for _ in range(2)]
        self.req_res = [B.new_get_result(dev) for _ in range(2)]
        self.req_idx_host = [torch.empty(w.N, dtype=torch.int32, pin_memory=True) for _ in range(2)]
        self.req_res_host = [torch.empty(self.req_res[0].shape, dtype=torch.uint8, pin_memory=True) for _ in range(2)]
        self.req_done = [torch.cuda.Event() for _ in range(2)]
        cap_T = max(self.packed["hidden"].shape[0], int(w.token_budget))
        self.packed_live = {
            "cu_seqlens": torch.zeros(w.N + 1, dtype=torch.int32, device=dev),
            "hidden": self.packed["hidden"] if cap_T == self.packed["hidden"].shape[0]
            else torch.empty(cap_T, w.d, dtype=torch.bfloat16, device=dev),
            "target": torch.empty(cap_T, dtype=torch.int32, device=dev),
            "old_logp": torch.empty(cap_T, device=dev), "ref_logp": torch.empty(cap_T, device=dev),
            "adv_seq": torch.empty(w.N, device=dev),
        }
        self.live_logp, self.live_ent, self.live_lse, self.live_g = (torch.empty(cap_T, device=dev) for _ in range(4))
        self.ctx.reserve(cap_T, w.N, w.d, w.V)
        self.live_requests = 0

    def _request(self, slot: int):
        """Queue: the next wave of arrivals marked ready, one read request, its answer to pinned memory."""
        c, w = self.ctx, self.w
        if self.next_wave < w.N:
            c.controller_put(self.tab, self.arrival_dev[self.next_wave:self.next_wave + self.wave], 1)
            self.next_wave += self.wave
        c.controller_get(self.tab, 1, 1, w.N, int(w.token_budget), self.req_idx[slot], self.req_res[slot])
        self.req_idx_host[slot].copy_(self.req_idx[slot], non_blocking=True)
        self.req_res_host[slot].copy_(self.req_res[slot], non_blocking=True)
        self.req_done[slot].record()

    def step_live_controller(self):
        """The streaming step with live production and consumption: every micro-batch is whatever
        the controller hands out (ready, not yet consumed, within the token budget).  The request
        for micro-batch k+1 is queued before the kernels of micro-batch k, so its answer is on the
        host long before the GPU needs the next index list."""
        w, c, B = self.w, self.ctx, self.B
        c.controller_clear(self.tab, 0xFFFFFFFF, 0xFFFFFFFF)
        c.grpo_advantage(self.reward, None, w.n_prompts, self.adv)
        store = {"tok_offset_host": self.off, "d": w.d, "adv": self.adv, **self.store}
        self.next_wave, slot, total, k = 0, 0, 0, 0
        self._request(slot)
        while True:
            self.req_done[slot].synchronize()
            count = B.GetResult.from_buffer_copy(self.req_res_host[slot].numpy().tobytes()).count
            if count == 0 and self.next_wave >= w.N:
                break
            mb = self.req_idx_host[slot][:count].numpy().copy()
            self._request(slot ^ 1)
            if count:
                T = c.pack_microbatch(store, mb, self.packed_live)
                c.token_logprob(self.packed_live["hidden"], self.W, self.packed_live["target"], self.live_logp,
                                self.live_ent, self.live_lse, T=T)
                c.policy_loss(self.live_logp, self.packed_live["old_logp"], self.packed_live["ref_logp"],
                              self.packed_live["adv_seq"], self.packed_live["cu_seqlens"],
                              self.loss_outs[k % len(self.loss_outs)], self.live_g, self.live_ent,
                              w.clip_eps, w.clip_eps, w.kl_coef, 0, 1.0, B=count, T=T)
                total += T
                k += 1
            slot ^= 1
        self.live_requests = k
        if total != self.T:
            raise RuntimeError(f"the controller handed out {total} tokens of {self.T}")
        return total

    # -- the streaming pieces as one path: two tasks, one store, one status table -----------
    COL_RESPONSE, COL_OLD_LOGP = 1, 2         # column bits of the status table
    TASK_INFER, TASK_UPDATE = 1, 2            # consumption bits: actor inference, actor-update forward

    def make_closed_loop(self, wave: int = 512):
        """Section 4.2's interaction, end to end on one device.  Responses become ready (hidden
        states and targets written) `wave` at a time in arrival order.  Actor inference asks the
        controller for ready samples, fetches them, scores them and writes its per-token log-probs
        back to the store's old_logp column by the same index list, which also marks that column
        written.  The loss task asks for samples whose response AND old_logp columns are written,
        fetches them -- old_logp now being what the first task stored -- scores them and reduces
        the loss.  Every micro-batch of either task is whatever af_controller_get hands out."""
        w, dev, B = self.w, self.dev, self.B
        if not hasattr(self, "W_host"):
            self.make_weight_refresh()
        self.cl_tab = {"ready": torch.zeros(w.N, dtype=torch.int32, device=dev),
                       "consumed": torch.zeros(w.N, dtype=torch.int32, device=dev),
                       "length": torch.as_tensor(w.lengths.astype(np.int32), device=dev)}
        self.cl_arrival = torch.as_tensor(wl.arrival_order(w).astype(np.int32), device=dev)
        self.cl_wave = wave

        def channel():
            return {"idx": [torch.empty(w.N, dtype=torch.int32, device=dev) for _ in range(2)],
                    "res": [B.new_get_result(dev) for _ in range(2)],
                    "idx_host": [torch.empty(w.N, dtype=torch.int32, pin_memory=True) for _ in range(2)],
                    "res_host": [torch.empty(ctypes.sizeof(B.GetResult), dtype=torch.uint8, pin_memory=True) for _ in range(2)]}

        self.cl_req = {self.TASK_INFER: channel(), self.TASK_UPDATE: channel()}
        self.cl_done = [torch.cuda.Event() for _ in range(2)]
        budget = int(w.token_budget or w.total_tokens)
        cap_T = max(budget, int(w.lengths.max()))
        self.cl_budget = budget
        self.cl_packed1 = {"cu_seqlens": torch.zeros(w.N + 1, dtype=torch.int32, device=dev),
                           "hidden": torch.empty(cap_T, w.d, dtype=torch.bfloat16, device=dev),
                           "target": torch.empty(cap_T, dtype=torch.int32, device=dev)}
        self.cl_packed2 = {"cu_seqlens": torch.zeros(w.N + 1, dtype=torch.int32, device=dev),
                           "hidden": torch.empty(cap_T, w.d, dtype=torch.bfloat16, device=dev),
                           "target": torch.empty(cap_T, dtype=torch.int32, device=dev),
                           "old_logp": torch.empty(cap_T, device=dev), "ref_logp": torch.empty(cap_T, device=dev),
                           "adv_seq": torch.empty(w.N, device=dev)}
        self.cl_logp1 = torch.empty(cap_T, device=dev)
        self.cl_logp2, self.cl_ent2, self.cl_lse2, self.cl_g2 = (torch.empty(cap_T, device=dev) for _ in range(4))
        self.cl_old_col = torch.empty(w.total_tokens, device=dev)     # the column actor inference fills
        self.cl_loss_outs = []
        self.ctx.reserve(cap_T, w.N, w.d, w.V)
        self.cl_iterations = 0

    def _cl_request(self, slot: int):
        """Queue: the next wave of arrivals marked written, one read request per task, answers to pinned memory."""
        c, w = self.ctx, self.w
        if self.cl_next_wave < w.N:
            c.controller_put(self.cl_tab, self.cl_arrival[self.cl_next_wave:self.cl_next_wave + self.cl_wave],
                             self.COL_RESPONSE)
            self.cl_next_wave += self.cl_wave
        for task, mask in ((self.TASK_INFER, self.COL_RESPONSE), (self.TASK_UPDATE, self.COL_RESPONSE | self.COL_OLD_LOGP)):
            ch = self.cl_req[task]
            c.controller_get(self.cl_tab, mask, task, w.N, self.cl_budget, ch["idx"][slot], ch["res"][slot])
            ch["idx_host"][slot].copy_(ch["idx"][slot], non_blocking=True)
            ch["res_host"][slot].copy_(ch["res"][slot], non_blocking=True)
        self.cl_done[slot].record()

    def step_closed_loop(self, refresh_weights: bool = True):
        """One pass of the whole store through both tasks.  Requests are queued one iteration ahead
        of the kernels that use their answers, so the host never waits for the GPU to drain; a loss
        request therefore sees the log-probs written up to the previous iteration.  With
        `refresh_weights` a new LM-head weight is loaded on a second stream meanwhile and swapped in
        at an iteration boundary (Section 5.2)."""
        w, c, B = self.w, self.ctx, self.B
        main = torch.cuda.current_stream()
        pending = False
        if refresh_weights:
            with torch.cuda.stream(self.w_stream):
                self.w_stream.wait_event(self.w_released)
                self.W_standby.copy_(self.W_host, non_blocking=True)
                self.w_loaded.record(self.w_stream)
            pending = True
        c.controller_clear(self.cl_tab, 0xFFFFFFFF, 0xFFFFFFFF)
        self.cl_old_col.fill_(float("nan"))       # a row read before it was written would poison its loss
        self.advantages()
        store1 = {"tok_offset_host": self.off, "d": w.d, "hidden": self.store["hidden"], "target": self.store["target"]}
        store2 = {"tok_offset_host": self.off, "d": w.d, "adv": self.adv, "hidden": self.store["hidden"],
                  "target": self.store["target"], "old_logp": self.cl_old_col, "ref_logp": self.store["ref_logp"]}
        self.cl_next_wave, slot, tot1, tot2, it, k2 = 0, 0, 0, 0, 0, 0
        self.cl_history = []                      # (task, index list) of every micro-batch handed out
        self._cl_request(slot)
        while tot1 < self.T or tot2 < self.T:
            it += 1
            if it > 8 * w.N + 64:
                raise RuntimeError("the closed loop made no progress")
            self.cl_done[slot].synchronize()
            mbs = {}
            for task, ch in self.cl_req.items():
                n = B.GetResult.from_buffer_copy(ch["res_host"][slot].numpy().tobytes()).count
                mbs[task] = ch["idx_host"][slot][:n].numpy().copy()
            self._cl_request(slot ^ 1)
            if pending and (self.w_loaded.query() or (tot1 >= self.T)):
                main.wait_event(self.w_loaded)
                self.W, self.W_standby = self.W_standby, self.W
                self.w_released.record(main)
                self.w_swaps += 1
                pending = False
            mb = mbs[self.TASK_INFER]
            if len(mb):      # actor inference: fetch, score, write the log-probs back, mark them written
                self.cl_history.append((self.TASK_INFER, mb))
                T1 = c.pack_microbatch(store1, mb, self.cl_packed1)
                c.token_logprob(self.cl_packed1["hidden"], self.W, self.cl_packed1["target"], self.cl_logp1, T=T1)
                c.unpack_microbatch(self.off, mb, [self.cl_logp1], [self.cl_old_col], self.cl_tab, self.COL_OLD_LOGP)
                tot1 += T1
            mb = mbs[self.TASK_UPDATE]
            if len(mb):      # loss task: its old_logp column is what actor inference stored
                self.cl_history.append((self.TASK_UPDATE, mb))
                while len(self.cl_loss_outs) <= k2:
                    self.cl_loss_outs.append(B.new_loss_out(self.dev))
                T2 = c.pack_microbatch(store2, mb, self.cl_packed2)
                c.token_logprob(self.cl_packed2["hidden"], self.W, self.cl_packed2["target"], self.cl_logp2,
                                self.cl_ent2, self.cl_lse2, T=T2)
                c.policy_loss(self.cl_logp2, self.cl_packed2["old_logp"], self.cl_packed2["ref_logp"],
                              self.cl_packed2["adv_seq"], self.cl_packed2["cu_seqlens"], self.cl_loss_outs[k2],
                              self.cl_g2, self.cl_ent2, w.clip_eps, w.clip_eps, w.kl_coef, 0, 1.0, B=len(mb), T=T2)
                tot2 += T2
                k2 += 1
            slot ^= 1
        if pending:          # nothing was left to score when the load finished: swap for the next step
            main.wait_event(self.w_loaded)
            self.W, self.W_standby = self.W_standby, self.W
            self.w_released.record(main)
            self.w_swaps += 1
        self.cl_iterations, self.cl_loss_count = it, k2
        if tot1 != self.T or tot2 != self.T:
            raise RuntimeError(f"the two tasks saw {tot1} and {tot2} tokens of {self.T}")
        return tot1 + tot2

    # -- delayed parameter update: new weights arrive while scoring goes on -----------------
    def make_weight_refresh(self):
        """A pinned host copy of the LM-head weight (the "received new parameters"), a standby
        device buffer and a copy stream.  Scoring keeps using the old weight while the new one is
        loaded; the buffers are swapped at the first micro-batch boundary after the load."""
        self.W_host = torch.empty(self.W.shape, dtype=self.W.dtype, pin_memory=True)
        self.W_host.copy_(self.W)
        self.W_standby = torch.empty_like(self.W)
        self.w_stream = torch.cuda.Stream()
        self.w_loaded = torch.cuda.Event()
        self.w_released = torch.cuda.Event()      # last kernel that read the standby buffer has run
        torch.cuda.synchronize()
        self.w_released.record()
        self.w_swaps = 0

    def step_with_weight_refresh(self):
        w, c = self.w, self.ctx
        main = torch.cuda.current_stream()
        with torch.cuda.stream(self.w_stream):
            self.w_stream.wait_event(self.w_released)
            self.W_standby.copy_(self.W_host, non_blocking=True)
            self.w_loaded.record(self.w_stream)
        pending = True
        c.grpo_advantage(self.reward, None, w.n_prompts, self.adv)
        store = {"tok_offset_host": self.off, "d": w.d, "adv": self.adv, **self.store}
        total = 0
        for i, (mb, loss_out) in enumerate(zip(self.mbs, self.loss_outs)):
            if pending and (self.w_loaded.query() or i == len(self.mbs) - 1):
                main.wait_event(self.w_loaded)                 # no-op when the load has finished
                self.W, self.W_standby = self.W_standby, self.W
                self.w_released.record(main)                   # kernels enqueued so far read the old buffer
                self.w_swaps += 1
                pending = False
            T = c.pack_microbatch(store, mb, self.packed)
            c.token_logprob(self.packed["hidden"], self.W, self.packed["target"], self.logp, self.ent, self.lse, T=T)
            c.policy_loss(self.logp, self.packed["old_logp"], self.packed["ref_logp"], self.packed["adv_seq"],
                          self.packed["cu_seqlens"], loss_out, self.dlogp, self.ent,
                          w.clip_eps, w.clip_eps, w.kl_coef, 0, 1.0 / self.world, B=len(mb), T=T)
            total += T
        return total

    # -- end-to-end: store columns start in pinned host memory ------------------------------
    def make_host_store(self):
        """Pinned host copies of the store columns and rewards, a second device copy of the store
        and a copy stream: the host->device copies of step k+1 run while step k computes."""
        self.host = {k: torch.empty(v.shape, dtype=v.dtype, pin_memory=True) for k, v in self.store.items()}
        self.host["reward"] = torch.empty(self.reward.shape, dtype=self.reward.dtype, pin_memory=True)
        for k, v in self.store.items():
            self.host[k].copy_(v)
        self.host["reward"].copy_(self.reward)
        self.dev_store = [self.store, {k: torch.empty_like(v) for k, v in self.store.items()}]
        self.dev_reward = [self.reward, torch.empty_like(self.reward)]
        self.copy_stream = torch.cuda.Stream()
        self.buf_ready = [torch.cuda.Event() for _ in range(2)]
        self.buf_free = [torch.cuda.Event() for _ in range(2)]
        torch.cuda.synchronize()
        for e in self.buf_free:
            e.record()
        self.e2e_steps = 0
        self.h2d_bytes = sum(t.numel() * t.element_size() for t in self.host.values())
        self.host_loss = [torch.empty(lo.shape, dtype=torch.uint8, pin_memory=True) for lo in self.loss_outs]
        # the result of the scoring task: per-token log-probs in packed order, read back every step
        self.e2e_logp_host = torch.empty(self.T, dtype=torch.float32, pin_memory=True)
        self.d2h_bytes = self.e2e_logp_host.numel() * 4 + sum(lo.numel() for lo in self.loss_outs)

    def step_e2e(self):
        b = self.e2e_steps & 1
        self.e2e_steps += 1
        main = torch.cuda.current_stream()
        with torch.cuda.stream(self.copy_stream):
            self.copy_stream.wait_event(self.buf_free[b])       # the step that last read this copy is done
            for k, v in self.dev_store[b].items():
                v.copy_(self.host[k], non_blocking=True)
            self.dev_reward[b].copy_(self.host["reward"], non_blocking=True)
            self.buf_ready[b].record(self.copy_stream)
        main.wait_event(self.buf_ready[b])
        T = self.step(store_cols=self.dev_store[b], reward=self.dev_reward[b])
        self.buf_free[b].record(main)
        for h, lo in zip(self.host_loss, self.loss_outs):
            h.copy_(lo, non_blocking=True)
        return T


def timed_loop(fn, steps: int, world: int):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    torch.cuda.synchronize()
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    marks[0].record()
    for i in range(steps):
        fn()
        marks[i + 1].record()
    torch.cuda.synchronize()
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    timed_loop.last_steps_ms = [marks[i].elapsed_time(marks[i + 1]) for i in range(steps)]
    return marks[0].elapsed_time(marks[-1])


def cpu_oracle_sample(w: wl.Workload, hidden_rows: torch.Tensor, W_bits: np.ndarray, target_rows: np.ndarray,
                      reward: np.ndarray):
    """One pass of the oracle, as it stands, over a sample of `n` tokens forming one sequence of
    the batch: pack -> log-prob -> advantage (all N responses) -> loss.  Returns seconds."""
    from oracle import grpo_oracle as O
    n = hidden_rows.shape[0]
    t0 = time.perf_counter()
    packed = O.pack_microbatch_ref(np.array([0, n]), [0], {"hidden": wl.bf16_bits(hidden_rows), "target": target_rows})
    logp, ent, lse = O.token_logprob_ref(packed["hidden"], W_bits, packed["target"])
    adv = O.grpo_advantage_ref(reward, w.group_id, w.n_prompts)
    O.policy_loss_ref(logp, logp + 0.1, logp - 0.1, adv[:1], packed["cu_seqlens"], w.clip_eps, w.clip_eps,
                      w.kl_coef, entropy=ent)
    return time.perf_counter() - t0


def blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else (os.cpu_count() or 1)
    except Exception:
        return os.cpu_count() or 1


def describe(w, job, name: str) -> str:
    return (f"{name}: {head_name(w)} head d={w.d} V={w.V}, {w.N} responses "
            f"({w.n_prompts} prompts x {w.group_size}), {job.T} scored tokens per GPU, "
            + (f"{len(job.mbs)} arrival-ordered micro-batches of <= {w.token_budget} tokens, packed, "
               "scored and loss-reduced back to back on one stream" if w.token_budget
               else "one arrival-ordered packed micro-batch")
            + (", forward + backward (dH, dW)" if w.backward else ""))


def host_enqueue_us(job, n: int = 20) -> float:
    """Host time of one step's calls (no synchronisation inside the loop): what the CPU pays to
    enqueue a step, which bounds the step rate of a launch-bound workload."""
    job.step()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(n):
        job.step()
    dt = time.perf_counter() - t0
    torch.cuda.synchronize()
    return 1e6 * dt / n


def graph_replay_us(job, n: int = 50) -> float:
    """Device time per scoring step (advantage, log-prob, loss on the packed batch) when the calls
    are recorded once into a CUDA graph and replayed: what a launch-bound workload costs once the
    host's calls are out of the way.  (The pack stages its index list through the host and is not
    recorded.)"""
    w, c = job.w, job.ctx
    T = job.T

    def scoring():
        c.grpo_advantage(job.reward, None, w.n_prompts, job.adv)
        c.token_logprob(job.packed["hidden"], job.W, job.packed["target"], job.logp, job.ent, job.lse, T=T)
        c.policy_loss(job.logp, job.packed["old_logp"], job.packed["ref_logp"], job.packed["adv_seq"],
                      job.packed["cu_seqlens"], job.loss_out, job.dlogp, job.ent, w.clip_eps, w.clip_eps, w.kl_coef,
                      0, job.loss_scale, B=len(job.mbs[-1]), T=T)

    job.step()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        scoring()
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        scoring()
    for _ in range(3):
        graph.replay()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(n):
        graph.replay()
    e1.record()
    torch.cuda.synchronize()
    return 1e3 * e0.elapsed_time(e1) / n


def timed_leg(fn, steps: int, warmup: int, world: int, tokens: int):
    for _ in range(warmup):
        fn()
    ms_total = timed_loop(fn, steps, world)
    ms, _ = reduce_over_ranks(ms_total / steps, tokens, world)
    return ms


def streaming_legs(job, args, world: int, tokens: int, steps: int, warmup: int) -> dict:
    """The streaming store's extra legs: the controller in the loop, the delayed weight update, and
    the two-task closed loop with write-back."""
    out = {}
    w = job.w
    job.make_live_controller()
    ms = timed_leg(job.step_live_controller, steps, warmup, world, tokens)
    out["live_controller"] = {
        "value": job.T / (ms * 1e-3), "unit": UNIT, "ms_per_step": ms, "micro_batches": job.live_requests,
        "what": "the same store scored with the controller in the loop: responses become ready 512 at a "
                "time in arrival order, every micro-batch is the answer to an af_controller_get (ready, "
                "not consumed, <= the token budget) read back to the host, then packed, scored and "
                "loss-reduced; the next request is queued ahead of the current micro-batch's kernels"}
    job.make_weight_refresh()
    ms = timed_leg(job.step_with_weight_refresh, steps, warmup, world, tokens)
    out["weight_refresh"] = {
        "value": tokens / (ms * 1e-3), "unit": UNIT, "ms_per_step": ms,
        "h2d_bytes_per_step": int(job.W.numel() * job.W.element_size()), "swaps": job.w_swaps,
        "what": "every step a new LM-head weight is loaded from pinned host memory on a second stream "
                "while scoring continues with the old one; swapped at a micro-batch boundary"}
    job.make_closed_loop()
    ms = timed_leg(job.step_closed_loop, steps, max(1, warmup - 1), world, tokens)
    losses = [job.B.read_loss_out(lo) for lo in job.cl_loss_outs[:job.cl_loss_count]]
    if not all(np.isfinite(r["loss"]) for r in losses):
        raise RuntimeError("closed loop: a loss record is not finite (a row was read before it was written)")
    out["closed_loop"] = {
        "value": job.T / (ms * 1e-3), "unit": "store tokens/s through both tasks", "ms_per_step": ms,
        "scored_tokens_per_s": 2.0 * job.T / (ms * 1e-3), "iterations": job.cl_iterations,
        "loss_micro_batches": job.cl_loss_count, "max_clip_frac": float(max(r["clip_frac"] for r in losses)),
        "weight_swaps": job.w_swaps,
        "what": "controller get -> pack -> log-prob -> write-back of the log-probs to the store's old_logp column "
                "with its ready bit (actor inference), and controller get on that bit -> pack -> log-prob -> loss "
                "(actor-update forward), interleaved on one stream over one status table, while a new weight "
                "loads and is swapped in at an iteration boundary; every token is scored twice"}
    return out


def side_leg(name: str, args, dev, peaks, steps: int = 5, warmup: int = 3) -> dict:
    """A short timed leg of another workload on one GPU (its own buffers, its own clock record)."""
    w = wl.make_workload(name)
    job = ScoringJob(w, dev, {"default": 0, "single": 1, "pair": 2, "die": 3}[args.gemm])
    out = {"workload": describe(w, job, name), "steps": steps, "warmup": warmup}
    for _ in range(warmup):
        job.step()
    torch.cuda.synchronize()
    sampler = ClockSampler(dev.index or 0)
    sampler.start()
    ms_total = timed_loop(lambda: job.step(time_gemm=True), steps, 1)
    out["clocks"] = sampler.stop()
    ms = ms_total / steps
    gemm_ms = float(np.sum([a.elapsed_time(b) for a, b in job.gemm_events])) / steps
    pack_ms = float(np.sum([a.elapsed_time(b) for a, b in job.pack_events])) / steps
    tf = 2.0 * job.T * w.d * w.V / (gemm_ms * 1e-3) / 1e12
    pack_gbs = (2.0 * job.T * (2 * w.d + 12) + 8.0 * w.N) / (pack_ms * 1e-3) / 1e9
    out.update({"value": job.T / (ms * 1e-3), "unit": UNIT, "ms_per_step": ms,
                "logprob_ms": gemm_ms, "logprob_tflops": tf, "frac_of_sustained": tf / peaks["bf16_tflops_sustained"],
                "frac_of_burst": tf / peaks["bf16_tflops"], "frac_of_nominal_2250": tf / 2250.0,
                "pack_ms": pack_ms, "pack_gbs": pack_gbs, "pack_frac_of_hbm": pack_gbs / peaks["hbm_gbs"],
                "gpu_launches": job.launches_per_step * steps})
    if job.T < 10000:
        out["host_enqueue_us_per_step"] = host_enqueue_us(job)
        if not w.token_budget and not w.backward:
            out["graph_replay_us_per_scoring_step"] = graph_replay_us(job)
        out["note"] = ("launch- and epilogue-bound: the device work of a step is tens of microseconds, the host's "
                       "calls take longer; tokens/s here measures call overhead, not the kernels")
    if w.backward:
        bwd_ms = float(np.sum([a.elapsed_time(b) for a, b in job.bwd_events])) / steps
        out["three_calls"] = {"ms_per_step": ms, "backward_ms": bwd_ms,
                              "backward_tflops_6TdV": 6.0 * job.T * w.d * w.V / (bwd_ms * 1e-3) / 1e12,
                              "step_tflops_8TdV": 8.0 * job.T * w.d * w.V / (ms * 1e-3) / 1e12}
        ms_f = timed_leg(job.step_fused_update, steps, 2, 1, job.T)
        out["fused_update"] = {"ms_per_step": ms_f, "value": job.T / (ms_f * 1e-3), "unit": UNIT,
                               "tflops_6TdV_model": 6.0 * job.T * w.d * w.V / (ms_f * 1e-3) / 1e12,
                               "frac_of_sustained": 6.0 * job.T * w.d * w.V / (ms_f * 1e-3) / 1e12 / peaks["bf16_tflops_sustained"]}
    if w.token_budget:
        out.update(streaming_legs(job, args, 1, job.T, 3, 2))
    flags = job.ctx.check_device_errors()
    if flags:
        raise RuntimeError(f"{name}: device error word set: {flags}")
    out["loss"] = job.B.read_loss_out(job.loss_out)["loss"]
    job.ctx.close()
    del job
    torch.cuda.empty_cache()
    return out


def run_ours(args):
    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (there is no CPU path)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    global EXCHANGE_WITH_ONE_RANK
    EXCHANGE_WITH_ONE_RANK = bool(args.dp_single_rank) and world == 1
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    elif EXCHANGE_WITH_ONE_RANK:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        with socket.socket() as sk:
            sk.bind(("127.0.0.1", 0))
            os.environ.setdefault("MASTER_PORT", str(sk.getsockname()[1]))
        dist.init_process_group("nccl", rank=0, world_size=1, device_id=dev)
    variant = {"default": 0, "single": 1, "pair": 2, "die": 3}[args.gemm]
    base = wl.make_workload(args.workload)
    # data parallel: the global batch (one draw of the workload per rank) is dealt to the ranks by
    # token count; a streaming store stays whole on its rank; vocabulary parallel: one batch, the
    # head split by rows
    dp = None
    if exchanging(world) and not args.vocab_parallel and not base.token_budget:
        dp = DataParallelShare(args.workload, world, rank, balance=not args.no_balance)
    w = rank_workload(args.workload, 0 if args.vocab_parallel else rank)
    job = ScoringJob(w, dev, variant, world, args.v_splits, args.vocab_parallel, rank, args.bwd_token_block, dp)
    w = job.w
    peaks = measured_peaks()
    hbm_alone = job.hbm_kernels_at_scale(peaks["hbm_gbs"], args.hbm_log2) if rank == 0 and world == 1 else {}

    for _ in range(args.warmup):
        job.step()
    torch.cuda.synchronize()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    ms_total = timed_loop(lambda: job.step(time_gemm=True), args.steps, world)
    clocks = sampler.stop() if rank == 0 else None
    steps_ms = list(timed_loop.last_steps_ms)
    # per step: summed over the step's micro-batches
    gemm_ms = float(np.sum([a.elapsed_time(b) for a, b in job.gemm_events])) / args.steps
    pack_ms = float(np.sum([a.elapsed_time(b) for a, b in job.pack_events])) / args.steps
    bwd_ms = float(np.sum([a.elapsed_time(b) for a, b in job.bwd_events])) / args.steps if job.bwd_events else None
    ms_step, tokens = reduce_over_ranks(ms_total / args.steps, job.T, world)
    if args.vocab_parallel:
        tokens = job.T           # the ranks score the same tokens together
    flags = job.ctx.check_device_errors()
    if flags:
        raise RuntimeError(f"device error word set: {flags}")
    loss = job.B.read_loss_out(job.loss_out)["loss"]

    # end to end from pinned host memory
    job.make_host_store()
    for _ in range(max(1, min(args.warmup, 2))):
        job.step_e2e()
    ms_e2e_total = timed_loop(job.step_e2e, args.steps, world)
    ms_e2e, _ = reduce_over_ranks(ms_e2e_total / args.steps, job.T, world)
    e2e_steps_ms = list(timed_loop.last_steps_ms)
    logp_back = job.e2e_logp_host[:job.T]
    if not bool(torch.isfinite(logp_back).all()):
        raise RuntimeError("end-to-end step: log-probs read back to the host are not finite")
    job.e2e_logp_host = None

    fused = None
    if w.backward and not args.vocab_parallel:
        ms_f = timed_leg(job.step_fused_update, args.steps, 2, world, job.T)
        loss_f = job.B.read_loss_out(job.loss_out)["loss"]
        fused = {"value": tokens / (ms_f * 1e-3), "unit": UNIT, "ms_per_step": ms_f, "loss": loss_f,
                 "tflops_6TdV_model": 6.0 * job.T * w.d * w.V / (ms_f * 1e-3) / 1e12,
                 "what": "the same step through af_policy_update: forward, loss and backward in one call, the "
                         "logits evaluated once per token (6 T d V products instead of 8)"}

    streaming = {}
    if w.token_budget and world == 1 and (args.live_controller or args.weight_refresh or args.closed_loop):
        streaming = streaming_legs(job, args, world, tokens, args.steps, 2)

    flops = 2.0 * job.T * w.d * (job.v_hi - job.v_lo)       # this rank's rows of the head
    achieved = flops / (gemm_ms * 1e-3) / 1e12
    peak = peaks["bf16_tflops_sustained"]
    line = {
        "metric": METRIC, "value": tokens / (ms_step * 1e-3), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step,
        "step_ms_rank0": {"median": float(np.median(steps_ms)), "min": float(np.min(steps_ms)),
                          "max": float(np.max(steps_ms))},
        "higher_is_better": True,
        "scaling": "strong" if args.vocab_parallel else "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": describe(w, job, args.workload),
                   "l2": "inputs (hidden states >> 126 MB L2) exceed L2; no flush needed",
                   "gemm": "one CTA per 128x256 tile" if args.gemm == "single" else
                           "CTA pairs (cta_group::2), 256x256 tiles" + (", dealt without regard to dies" if args.gemm == "pair"
                                                                        else ", row tiles dealt by die"),
                   "die_split_sms": list(job.ctx.die_split()),
                   "l2_bytes": int(torch.cuda.get_device_properties(dev).L2_cache_size),
                   "parallelism": ("vocabulary-parallel head" if args.vocab_parallel else
                                   f"dp{world}: global batch dealt by token count (Karmarkar-Karp, equal counts)" if dp
                                   else f"dp{world}: a store per rank" if world > 1 else "single GPU"),
                   "loss": {"clip_eps": w.clip_eps, "kl_coef": w.kl_coef, "agg": "seq-mean-token-mean"}},
        "roofline": {"bound": "tensor", "kernel": "fused LM-head GEMM + online log-softmax (af_token_logprob)",
                     "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                     "peak_source": f"bf16_tflops_sustained, {peaks['source']}",
                     "frac_of_burst": achieved / peaks["bf16_tflops"], "frac_of_nominal_2250": achieved / 2250.0,
                     "kernel_ms": gemm_ms,
                     "traffic": (GEMM_DRAM_BYTES_PER_TOKEN_7B * job.T
                                 if GEMM_DRAM_BYTES_PER_TOKEN_7B and (w.d, w.V) == (3584, 152064)
                                 and args.gemm in ("default", "die") and args.v_splits == 0 and not w.token_budget
                                 and job.ctx.die_split()[0] > 0 else None)},
        "e2e": {"value": tokens / (ms_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": job.h2d_bytes,
                "d2h_bytes_per_step": int(job.d2h_bytes), "ms_per_step": ms_e2e,
                "d2h": "per-token log-probs in packed order (4 B per token) and the loss record",
                # the first timed step cannot hide its own copy behind a previous step's kernels
                "step_ms_rank0": {"first": e2e_steps_ms[0], "median": float(np.median(e2e_steps_ms)),
                                  "min": float(np.min(e2e_steps_ms))}},
        "gpu_launches": job.launches_per_step * args.steps,
        "clocks": clocks, "loss": loss,
    }
    pack_bytes = 2.0 * job.T * (2 * w.d + 12) + 8.0 * w.N
    pack_gbs = pack_bytes / (pack_ms * 1e-3) / 1e9
    line["hbm_kernels"] = {"peak_gbs": peaks["hbm_gbs"], "peak_source": f"hbm_gbs, {peaks['source']}",
                           "pack_microbatch_in_step": {"tokens": job.T, "bytes_per_token": 2 * (2 * w.d + 12),
                                                       "ms": pack_ms, "gbs": pack_gbs, "frac": pack_gbs / peaks["hbm_gbs"],
                                                       "where": "inside the timed steps (all micro-batches of a step), "
                                                                "each right after a GEMM (part at its power cap)"}}
    line["hbm_kernels"].update(hbm_alone)
    if fused is not None:
        line["fused_update"] = fused
    line.update(streaming)
    if dp is not None:
        line["data_parallel"] = dp.report()
    if rank == 0:
        line["balance"] = job.balance_report()
    if bwd_ms is not None:
        bflops = 6.0 * job.T * w.d * w.V
        line["backward"] = {"ms": bwd_ms, "tflops": bflops / (bwd_ms * 1e-3) / 1e12, "flop_model": "6*T*d*V",
                            "frac_of_sustained": bflops / (bwd_ms * 1e-3) / 1e12 / peak}
    if rank == 0 and world == 1:
        n = args.cpu_sample
        rows = job.packed["hidden"][:n].cpu()
        W_bits = wl.bf16_bits(job.W)
        secs = cpu_oracle_sample(w, rows, W_bits, job.packed["target"][:n].cpu().numpy(), job.reward.cpu().numpy())
        line["cpu_baseline"] = {"value": n / secs, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                                "sample": f"first {n} packed tokens as one sequence through pack/log-prob/loss "
                                          f"oracles at full V={w.V}, advantage oracle over all {w.N} responses; "
                                          f"{secs:.1f} s"}
    # the other workloads, one short leg each (single GPU, default workload only)
    if rank == 0 and world == 1 and args.workload == "cfg2" and not args.no_configs:
        job.ctx.close()
        del job, rows, W_bits
        torch.cuda.empty_cache()
        line["configs"] = {}
        for name in ("cfg1", "cfg3", "cfg4", "cfg5"):
            try:
                line["configs"][name] = side_leg(name, args, dev, peaks)
            except Exception as exc:          # a failed leg is reported as such; the headline stands
                line["configs"][name] = {"error": f"{type(exc).__name__}: {exc}"}
                try:
                    torch.cuda.empty_cache()
                except Exception:
                    pass
        c = line["configs"]

        def fig(name, *path):
            v = c.get(name, {})
            for k in path:
                v = v.get(k) if isinstance(v, dict) else None
            return v

        # the same figures as flat scalars beside the headline kernel's
        line["roofline"].update({
            "cfg1_tokens_per_s": fig("cfg1", "value"), "cfg1_host_enqueue_us_per_step": fig("cfg1", "host_enqueue_us_per_step"),
            "cfg1_graph_replay_us_per_scoring_step": fig("cfg1", "graph_replay_us_per_scoring_step"),
            "cfg3_tokens_per_s": fig("cfg3", "value"), "cfg3_logprob_tflops": fig("cfg3", "logprob_tflops"),
            "cfg3_frac_of_sustained": fig("cfg3", "frac_of_sustained"),
            "cfg4_three_calls_ms": fig("cfg4", "three_calls", "ms_per_step"),
            "cfg4_three_calls_tflops_8TdV": fig("cfg4", "three_calls", "step_tflops_8TdV"),
            "cfg4_backward_ms": fig("cfg4", "three_calls", "backward_ms"),
            "cfg4_fused_update_ms": fig("cfg4", "fused_update", "ms_per_step"),
            "cfg4_fused_update_tflops_6TdV": fig("cfg4", "fused_update", "tflops_6TdV_model"),
            "cfg5_tokens_per_s_incl_pack": fig("cfg5", "value"),
            "cfg5_live_controller_tokens_per_s": fig("cfg5", "live_controller", "value"),
            "cfg5_weight_refresh_tokens_per_s": fig("cfg5", "weight_refresh", "value"),
            "cfg5_closed_loop_scored_tokens_per_s": fig("cfg5", "closed_loop", "scored_tokens_per_s"),
            "cfg5_pack_frac_of_hbm": fig("cfg5", "pack_frac_of_hbm")})
    if rank == 0:
        print(json.dumps(line), flush=True)
    if exchanging(world):
        import torch.distributed as dist
        dist.destroy_process_group()


# ------------------------------------------------------------------------------------------
# the reference arm: the CPU oracle on bounded samples
# ------------------------------------------------------------------------------------------
def run_reference(args):
    rank, _, world = dist_env()
    ranks_reported = 1
    if world > 1:
        # every rank reports in (gloo, CPU); rank 0 alone does the work
        import torch.distributed as dist
        dist.init_process_group("gloo")
        seen = [torch.zeros(1, dtype=torch.int64) for _ in range(world)]
        dist.all_gather(seen, torch.tensor([rank + 1], dtype=torch.int64))
        ranks_reported = int(sum(int(t.item()) > 0 for t in seen))
        dist.barrier()
        dist.destroy_process_group()
    if rank != 0:
        return
    # a launcher may have pinned the math libraries to one thread per rank (torchrun exports
    # OMP_NUM_THREADS=1); the oracle runs alone here and gets the host's cores back
    try:
        from threadpoolctl import threadpool_limits
        threadpool_limits(limits=os.cpu_count() or 1, user_api="blas")
    except Exception:
        pass
    w = wl.make_workload(args.workload)
    n = args.cpu_sample
    W_bits = wl.bf16_bits(wl.gen_weight(w, "cpu"))
    reward = wl.gen_reward(w).numpy()
    target = wl.gen_target(w).numpy()
    times = []
    for s in range(args.warmup + args.steps):
        rows = wl.gen_hidden(w, "cpu", row_start=s * n, rows=n)
        secs = cpu_oracle_sample(w, rows, W_bits, target[s * n:(s + 1) * n], reward)
        if s >= args.warmup:
            times.append(secs)
    ms = 1e3 * float(np.mean(times))
    value = n / (ms * 1e-3)
    sample = f"{n} tokens per step as one sequence at full V={w.V} (pack/log-prob/loss oracles), advantage over {w.N} responses"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{args.workload}: {head_name(w)} head d={w.d} V={w.V}; bounded sample: {sample}"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0, "ranks_reported": ranks_reported,
    }
    print(json.dumps(line), flush=True)


def launch_ranks(n: int) -> int:
    """`python bench.py --gpus N` with no launcher around it: start N ranks of this script, one per
    GPU, through torch.distributed.run on this node, and pass their output through (rank 0 prints
    the JSON line).  Returns the launcher's exit code."""
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__), *sys.argv[1:]]
    env = dict(os.environ)
    env.setdefault("OMP_NUM_THREADS", str(max(1, (os.cpu_count() or 1) // n)))
    return subprocess.run(cmd, env=env).returncode


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2")
    ap.add_argument("--cpu-sample", type=int, default=1536, help="tokens in the CPU-oracle sample")
    ap.add_argument("--vocab-parallel", action="store_true",
                    help="split the LM head by vocabulary rows over the ranks (one batch for all; shard statistics "
                         "all-gathered and merged) instead of giving every rank its own batch")
    ap.add_argument("--no-balance", action="store_true",
                    help="data parallel: deal the global batch to the ranks by prompt index instead of by token "
                         "count (af_balance_partitions)")
    ap.add_argument("--dp-single-rank", action="store_true",
                    help="one GPU: run the data-parallel code path (split, reward all-gather, advantages by group "
                         "id, dW all-reduce started by the backward's event on a second stream) through a process "
                         "group of one rank")
    ap.add_argument("--no-configs", action="store_true",
                    help="skip the short legs of the other four workloads that follow the default cfg2 run")
    ap.add_argument("--v-splits", type=int, default=0,
                    help="vocabulary ranges per row tile of the fused GEMM (af_set_tuning v_splits); 0 = the library's choice")
    ap.add_argument("--hbm-log2", type=int, default=28, choices=range(20, 30),
                    help="the memory-bound kernels are also timed alone on 2^N tokens / responses / samples")
    ap.add_argument("--bwd-token-block", type=int, default=0,
                    help="token rows per block of the backward and fused-update calls (af_set_tuning "
                         "bwd_token_block, a multiple of 128); 0 = the library's choice")
    ap.add_argument("--live-controller", action="store_true",
                    help="streaming workloads: also time the steps with the controller in the loop, with the "
                         "weight refresh, and as the two-task closed loop")
    ap.add_argument("--weight-refresh", action="store_true", help="same as --live-controller")
    ap.add_argument("--closed-loop", action="store_true", help="same as --live-controller")
    ap.add_argument("--gemm", default="default", choices=["default", "single", "pair", "die"],
                    help="main loop of the tensor-core GEMMs (af_set_tuning gemm_variant): CTA pairs (the default) "
                         "or one CTA per tile")
    args = ap.parse_args()
    if args.gpus > 1 and "RANK" not in os.environ:
        sys.exit(launch_ranks(args.gpus))
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
