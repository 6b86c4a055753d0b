"""World-size-2 checks of the data-parallel host logic on CPU (gloo): prompts are split into
whole groups, rank results concatenate to the single-rank result, and bench.py's reduction takes
the max step time and the token sum over ranks."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import grpo_oracle as O
from paper_2507_01663_b200 import workloads as wl


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    w = wl.make_workload("cfg5_mini")
    prompts = wl.shard_prompts(w.n_prompts, world, rank)
    mine = np.concatenate([np.arange(p * w.group_size, (p + 1) * w.group_size) for p in prompts])
    r = wl.gen_reward(w).numpy()
    # group statistics need no exchange: every group is whole on its rank
    local_gid = w.group_id[mine] - prompts.start
    adv_local = O.grpo_advantage_ref(r[mine], local_gid, len(prompts))
    tokens_local = int(w.lengths[mine].sum())
    ms, tokens = bench.reduce_over_ranks(10.0 + 5.0 * rank, tokens_local, world)
    gathered = [None] * world
    dist.all_gather_object(gathered, (mine, adv_local))
    if rank == 0:
        idx = np.concatenate([g[0] for g in gathered])
        adv = np.concatenate([g[1] for g in gathered])
        full = O.grpo_advantage_ref(r, w.group_id, w.n_prompts)
        ok = (np.array_equal(np.sort(idx), np.arange(w.N)) and np.allclose(adv, full[idx], atol=1e-14)
              and ms == 10.0 + 5.0 * (world - 1) and tokens == w.total_tokens)
        with open(os.path.join(out_dir, "ok"), "w") as f:
            f.write("1" if ok else "0")
    # per-rank workloads of the weak-scaling bench differ by seed but not by shape
    a, b = bench.rank_workload("cfg2_mini", 0), bench.rank_workload("cfg2_mini", 1)
    assert (a.d, a.V, a.N) == (b.d, b.V, b.N) and not np.array_equal(a.lengths, b.lengths)
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_sharding(tmp_path):
    port = _free_port()
    mp.start_processes(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True, start_method="spawn")
    assert open(tmp_path / "ok").read() == "1"
