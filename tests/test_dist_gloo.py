"""World-size-2 checks of the data-parallel host logic on CPU (gloo): prompts are split into
whole groups, rank results concatenate to the single-rank result, bench.py's reduction takes the
max step time and the token sum over ranks, and the weight gradients of the ranks' batches, each
scored with loss_scale = B_rank / B_global, sum to the gradient of the global batch; the
statistics of vocabulary shards, gathered over the ranks, merge to the full-vocabulary result; a
global batch dealt to the ranks by token count (Karmarkar-Karp, equal sample counts) with gathered
rewards reproduces the single-rank advantages, loss and weight gradient."""
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


def _grad_worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    w = wl.make_workload("cfg1")
    H, W, y = wl.bf16_bits(wl.gen_hidden(w)), wl.bf16_bits(wl.gen_weight(w)), wl.gen_target(w).numpy()
    r = wl.gen_reward(w).numpy()
    adv = O.grpo_advantage_ref(r, w.group_id, w.n_prompts)
    off = w.tok_offset

    def actor_update(samples, scale):
        """Oracle forward + loss + backward over the given samples (packed in that order)."""
        packed = O.pack_microbatch_ref(off, samples, {"hidden": H, "target": y}, adv)
        lp, _, lse = O.token_logprob_ref(packed["hidden"], W, packed["target"])
        T = lp.shape[0]
        old = lp + 0.1 * np.sin(np.arange(T))            # any fixed perturbation, the same on every path
        ref = lp - 0.05 * np.cos(np.arange(T))
        res = O.policy_loss_ref(lp, old, ref, packed["adv_seq"], packed["cu_seqlens"], loss_scale=scale)
        _, dW = O.policy_loss_backward_ref(packed["hidden"], W, packed["target"], lse, res["dlogp"])
        return res["loss"], dW

    prompts = wl.shard_prompts(w.n_prompts, world, rank)
    mine = np.concatenate([np.arange(p * w.group_size, (p + 1) * w.group_size) for p in prompts])
    loss_local, dW_local = actor_update(mine, len(mine) / w.N)
    dW_sum = bench.allreduce_sum_(torch.from_numpy(dW_local.copy()), world).numpy()
    loss_sum = bench.allreduce_sum_(torch.tensor([loss_local], dtype=torch.float64), world).item()
    if rank == 0:
        # old / ref perturbations depend on the position inside the rank's batch: replay both
        # ranks' batches on one process and add them, which is what the global batch means here
        total_loss, total_dW = 0.0, 0.0
        for rk in range(world):
            pr = wl.shard_prompts(w.n_prompts, world, rk)
            idx = np.concatenate([np.arange(p * w.group_size, (p + 1) * w.group_size) for p in pr])
            l, g = actor_update(idx, len(idx) / w.N)
            total_loss, total_dW = total_loss + l, total_dW + g
        ok = np.allclose(dW_sum, total_dW, rtol=0, atol=1e-12 * np.abs(total_dW).max()) and abs(loss_sum - total_loss) < 1e-14
        # and the scaled per-rank losses add up to the global-batch loss when the inputs agree:
        # with old = ref = logp every token's loss is -A, so L = -(1/B) sum_i A_i on any split
        packed = O.pack_microbatch_ref(off, np.arange(w.N), {"hidden": H, "target": y}, adv)
        lp, _, _ = O.token_logprob_ref(packed["hidden"], W, packed["target"])
        full = O.policy_loss_ref(lp, lp, lp, packed["adv_seq"], packed["cu_seqlens"])["loss"]
        parts = 0.0
        for rk in range(world):
            pr = wl.shard_prompts(w.n_prompts, world, rk)
            idx = np.concatenate([np.arange(p * w.group_size, (p + 1) * w.group_size) for p in pr])
            pk = O.pack_microbatch_ref(off, idx, {"hidden": H, "target": y}, adv)
            lpr, _, _ = O.token_logprob_ref(pk["hidden"], W, pk["target"])
            parts += O.policy_loss_ref(lpr, lpr, lpr, pk["adv_seq"], pk["cu_seqlens"], loss_scale=len(idx) / w.N)["loss"]
        ok = ok and abs(parts - full) < 1e-12
        with open(os.path.join(out_dir, "ok_grad"), "w") as f:
            f.write("1" if ok else "0")
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_gradient_sum(tmp_path):
    port = _free_port()
    mp.start_processes(_grad_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True, start_method="spawn")
    assert open(tmp_path / "ok_grad").read() == "1"


def _vocab_worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    w = wl.make_workload("cfg1")
    H, W, y = wl.bf16_bits(wl.gen_hidden(w)), wl.bf16_bits(wl.gen_weight(w)), wl.gen_target(w).numpy()
    lo, hi = bench.vocab_shard(w.V, world, rank)
    mine = torch.from_numpy(O.token_logprob_shard_ref(H, W[lo:hi], y, lo))
    gathered = bench.allgather_partials(mine, world)                     # [R, T, 4]
    logp, ent, lse = O.merge_logprob_shards_ref(gathered.numpy())
    ref = O.token_logprob_ref(H, W, y)
    ok = all(np.allclose(a, b, atol=1e-12) for a, b in zip((logp, ent, lse), ref))
    ok = ok and gathered.shape == (world, H.shape[0], 4)
    # backward of the sharded head: the ranks' dH contributions are summed, dW rows stay local
    g = np.random.default_rng(3).standard_normal(H.shape[0]) / H.shape[0]
    dH_part, dW_rows = O.policy_loss_backward_shard_ref(H, W[lo:hi], y, lse, g, lo)
    dH = bench.allreduce_sum_(torch.from_numpy(dH_part.copy()), world).numpy()
    dH_ref, dW_ref = O.policy_loss_backward_ref(H, W, y, ref[2], g)
    ok = ok and np.allclose(dH, dH_ref, atol=1e-12) and np.allclose(dW_rows, dW_ref[lo:hi], atol=1e-12)
    los = [bench.vocab_shard(w.V, world, r) for r in range(world)]
    ok = ok and los[0][0] == 0 and los[-1][1] == w.V and all(a[1] == b[0] for a, b in zip(los[:-1], los[1:]))
    with open(os.path.join(out_dir, f"ok_vocab_{rank}"), "w") as f:
        f.write("1" if ok else "0")
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_vocabulary_parallel_exchange(tmp_path):
    port = _free_port()
    mp.start_processes(_vocab_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True, start_method="spawn")
    assert open(tmp_path / "ok_vocab_0").read() == "1" and open(tmp_path / "ok_vocab_1").read() == "1"


def _balanced_worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    dp = bench.DataParallelShare("cfg4_mini", world, rank)
    w0 = dp.sources[0]
    W = wl.bf16_bits(wl.gen_weight(w0))
    goff = np.concatenate([[0], np.cumsum(dp.lengths)])                  # global token index of a response's first row

    def perturbation(samples):
        """old / ref offsets as a function of the token's global identity, so that they do not
        depend on which rank scores the token or where it sits in the rank's batch."""
        t = np.concatenate([np.arange(goff[g], goff[g + 1]) for g in samples]).astype(np.float64)
        return 0.1 * np.sin(t), -0.05 * np.cos(t)

    def actor_update(H_bits, y, lengths, adv, samples, scale):
        cu = np.concatenate([[0], np.cumsum(lengths)])
        lp, _, lse = O.token_logprob_ref(H_bits, W, y)
        d_old, d_ref = perturbation(samples)
        res = O.policy_loss_ref(lp, lp + d_old, lp + d_ref, adv, cu, loss_scale=scale)
        _, dW = O.policy_loss_backward_ref(H_bits, W, y, lse, res["dlogp"])
        return res["loss"], dW

    # this rank: its own rows and rewards only; the rewards of the others arrive by the all-gather
    H, y, r_mine = dp.build_columns("cpu")
    gathered = dp.gather_rewards(r_mine).numpy()
    adv_all = O.grpo_advantage_ref(gathered, dp.gathered_group_id, dp.n_groups)
    adv_mine = adv_all[rank * dp.n_mine:(rank + 1) * dp.n_mine]
    loss_local, dW_local = actor_update(wl.bf16_bits(H), y.numpy(), dp.lengths[dp.mine], adv_mine, dp.mine, dp.loss_scale)
    dW_sum = bench.allreduce_sum_(torch.from_numpy(dW_local.copy()), world).numpy()
    loss_sum = bench.allreduce_sum_(torch.tensor([loss_local], dtype=torch.float64), world).item()
    if rank == 0:
        # the global batch on one process, in global index order
        Hs = [wl.bf16_bits(wl.gen_hidden(w)) for w in dp.sources]
        ys = [wl.gen_target(w).numpy() for w in dp.sources]
        r_all = np.concatenate([wl.gen_reward(w).numpy() for w in dp.sources])
        adv_global = O.grpo_advantage_ref(r_all, dp.group_id, dp.n_groups)
        loss_g, dW_g = actor_update(np.concatenate(Hs), np.concatenate(ys), dp.lengths, adv_global,
                                    np.arange(dp.N_global), 1.0)
        rep = dp.report()
        counts = np.bincount(dp.part, minlength=world)
        ok = (np.array_equal(gathered, r_all[dp.gathered_order])
              and np.allclose(adv_all, adv_global[dp.gathered_order], rtol=0, atol=1e-14)
              and abs(loss_sum - loss_g) <= 1e-12 * max(1.0, abs(loss_g))
              and np.allclose(dW_sum, dW_g, rtol=0, atol=1e-11 * np.abs(dW_g).max())
              and counts.min() == counts.max() == w0.N
              and rep["token_spread_balanced"] <= rep["token_spread_by_prompt_index"]
              and sum(rep["tokens_per_rank"]) == int(dp.lengths.sum())
              and len(set(dp.group_id[dp.mine])) > w0.n_prompts // 2)       # groups really are spread over ranks
        with open(os.path.join(out_dir, "ok_balanced"), "w") as f:
            f.write("1" if ok else "0")
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_token_balanced_actor_update(tmp_path):
    from paper_2507_01663_b200 import build as b
    b.build()                                    # af_balance_partitions is a host call of the library
    port = _free_port()
    mp.start_processes(_balanced_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True, start_method="spawn")
    assert open(tmp_path / "ok_balanced").read() == "1"
