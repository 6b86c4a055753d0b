"""The data-parallel step of the benchmark on one GPU: the ranks' shares of a token-balanced global
batch are run one after the other (nothing here waits on another rank), with the reward all-gather
replaced by the concatenation it would deliver.  The shares' advantages, losses and weight gradients
must add up to the oracle's result for the global batch."""
import numpy as np
import pytest
import torch

import bench
from oracle import grpo_oracle as O
from paper_2507_01663_b200 import workloads as wl
from gpu_util import ADV_TOL, GRAD_RTOL, LOGP_TOL, LOSS_RTOL, device, f32, np_of, off_the_clip_bounds

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("fused", [False, True], ids=["three_calls", "update"])
def test_rank_shares_add_up_to_the_global_batch(fused):
    dev = device()
    world = 2
    shares = [bench.DataParallelShare("cfg4_mini", world, r) for r in range(world)]
    ref = shares[0]
    assert len(set(ref.group_id[ref.mine])) > ref.sources[0].n_prompts // 2      # groups are spread over the ranks
    own_rewards = [s.build_columns("cpu")[2] for s in shares]
    gathered = torch.cat(own_rewards).to(dev)                                    # what the all-gather delivers
    adv_global = O.grpo_advantage_ref(np_of(gathered), ref.gathered_group_id, ref.n_groups)
    W_bits = wl.bf16_bits(wl.gen_weight(ref.sources[0]))
    loss_sum, dW_sum, loss_ref, dW_ref = 0.0, None, 0.0, 0.0
    for r, dp in enumerate(shares):
        dp.gather_rewards = lambda mine: gathered
        job = bench.ScoringJob(None, dev, world=1, rank=r, dp=dp)
        try:
            w = job.w
            # keep every token's ratio off the clip bounds (the two chains decide in different precisions)
            lp_store, _, _ = O.token_logprob_ref(wl.bf16_bits(job.store["hidden"]), W_bits, np_of(job.store["target"]))
            job.store["old_logp"].copy_(f32(off_the_clip_bounds(lp_store, np_of(job.store["old_logp"]), w.clip_eps, w.clip_eps)))
            (job.step_fused_update if fused else job.step)()
            torch.cuda.synchronize()
            assert job.ctx.check_device_errors() == 0
            # advantages: the whole batch by group id on every rank, its own slice kept
            assert np.abs(np_of(job.adv_all) - adv_global).max() <= ADV_TOL
            assert np.array_equal(np_of(job.adv), np_of(job.adv_all)[r * dp.n_mine:(r + 1) * dp.n_mine])
            got = job.B.read_loss_out(job.loss_out)
            loss_sum += got["loss"]
            dW_sum = job.d_W.double().cpu() if dW_sum is None else dW_sum + job.d_W.double().cpu()
            # the oracle on the same share: its own log-probs, the share's old / ref columns, its weight
            idx = job.mbs[0]
            cols = {"hidden": wl.bf16_bits(job.store["hidden"]), "target": np_of(job.store["target"]),
                    "old_logp": np_of(job.store["old_logp"]), "ref_logp": np_of(job.store["ref_logp"])}
            adv_mine = adv_global[r * dp.n_mine:(r + 1) * dp.n_mine]
            p = O.pack_microbatch_ref(w.tok_offset, idx, cols, adv_mine)
            lp, _, lse = O.token_logprob_ref(p["hidden"], W_bits, p["target"])
            assert np.abs(np_of(job.logp[:len(lp)]) - lp).max() <= LOGP_TOL
            res = O.policy_loss_ref(lp, p["old_logp"], p["ref_logp"], p["adv_seq"], p["cu_seqlens"], w.clip_eps, w.clip_eps,
                                    w.kl_coef, 0, dp.loss_scale)
            _, dW = O.policy_loss_backward_ref(p["hidden"], W_bits, p["target"], lse, res["dlogp"])
            slack = LOGP_TOL * float(np.abs(res["dlogp"]).sum())
            assert abs(got["loss"] - res["loss"]) <= LOSS_RTOL * abs(res["loss"]) + slack
            loss_ref += res["loss"]
            dW_ref = dW_ref + dW
        finally:
            job.ctx.close()
    n = np.linalg.norm(dW_ref)
    assert np.linalg.norm(dW_sum.numpy() - dW_ref) <= GRAD_RTOL * n and abs(np.linalg.norm(dW_sum.numpy()) - n) <= GRAD_RTOL * n
    assert abs(loss_sum - loss_ref) <= LOSS_RTOL * abs(loss_ref) + 2 * LOGP_TOL
