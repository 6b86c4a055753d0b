"""The streaming pieces as one path (Section 4.2: controller get -> worker fetch -> compute -> write-back
-> status update -> the next task's get; Section 5.2: new weights swapped in between micro-batches),
run through the benchmark's own step function and checked against the oracle."""
import numpy as np
import pytest
import torch

import bench
from oracle import controller_oracle as CO
from oracle import grpo_oracle as O
from paper_2507_01663_b200 import workloads as wl
from gpu_util import LOGP_TOL, LOSS_RTOL, device, np_of

pytestmark = pytest.mark.gpu


def test_two_tasks_through_one_store_and_status_table():
    w = wl.make_workload("cfg5_mini")
    dev = device()
    job = bench.ScoringJob(w, dev)
    try:
        job.make_closed_loop(wave=24)
        lp, _, _ = O.token_logprob_ref(wl.bf16_bits(job.store["hidden"]), wl.bf16_bits(job.W), np_of(job.store["target"]))
        adv_ref = O.grpo_advantage_ref(np_of(job.reward), w.group_id, w.n_prompts)
        ref_col = np_of(job.store["ref_logp"]).astype(np.float64)
        off = w.tok_offset
        for rep in range(2):                       # the second pass starts from a cleared table
            scored = job.step_closed_loop(refresh_weights=True)
            torch.cuda.synchronize()
            assert scored == 2 * w.total_tokens and job.ctx.check_device_errors() == 0
            # actor inference stored every token's log-prob in the store column, by index list
            col = np_of(job.cl_old_col)
            assert np.isfinite(col).all() and np.abs(col - lp).max() <= LOGP_TOL
            # status: both columns written, both tasks served, every sample exactly once per task
            both = job.COL_RESPONSE | job.COL_OLD_LOGP
            assert (np_of(job.cl_tab["ready"]) == both).all()
            assert (np_of(job.cl_tab["consumed"]) == (job.TASK_INFER | job.TASK_UPDATE)).all()
            for task in (job.TASK_INFER, job.TASK_UPDATE):
                seen = np.concatenate([mb for t, mb in job.cl_history if t == task])
                assert np.array_equal(np.sort(seen), np.arange(w.N))
            # a sample reached the loss task only after actor inference had written it
            first_seen = {}
            for pos, (t, mb) in enumerate(job.cl_history):
                for i in mb:
                    first_seen.setdefault((t, int(i)), pos)
            assert all(first_seen[(job.TASK_INFER, i)] < first_seen[(job.TASK_UPDATE, i)] for i in range(w.N))
            # every micro-batch respects the token budget (a longer single response goes alone)
            for _, mb in job.cl_history:
                assert int(w.lengths[mb].sum()) <= w.token_budget or len(mb) == 1
            # the loss records: the oracle chain on each micro-batch the loss task was handed, with the
            # oracle's own log-probs as the stored old_logp column
            loss_mbs = [mb for t, mb in job.cl_history if t == job.TASK_UPDATE]
            assert len(loss_mbs) == job.cl_loss_count
            for mb, lo in zip(loss_mbs, job.cl_loss_outs):
                got = job.B.read_loss_out(lo)
                rows = np.concatenate([np.arange(off[i], off[i + 1]) for i in mb])
                cu = np.concatenate([[0], np.cumsum(w.lengths[mb])])
                want = O.policy_loss_ref(lp[rows], lp[rows], ref_col[rows], adv_ref[mb], cu, w.clip_eps, w.clip_eps, w.kl_coef)
                slack = LOGP_TOL * float(np.abs(want["dlogp"]).sum())
                assert got["n_tokens"] == len(rows) and got["clip_frac"] == 0.0
                assert abs(got["loss"] - want["loss"]) <= LOSS_RTOL * abs(want["loss"]) + slack
        assert job.w_swaps == 2                    # one weight swap per pass, at an iteration boundary
    finally:
        job.ctx.close()


def test_first_request_matches_the_controller_oracle():
    """The first answers of the loop against the controller oracle: after the first wave of puts the
    inference task gets the longest in-budget prefix of the written samples, the loss task nothing."""
    w = wl.make_workload("cfg5_mini")
    job = bench.ScoringJob(w, device())
    try:
        job.make_closed_loop(wave=24)
        job.step_closed_loop(refresh_weights=False)
        order = wl.arrival_order(w)
        ready, consumed = np.zeros(w.N, np.uint32), np.zeros(w.N, np.uint32)
        CO.controller_put_ref(ready, order[:24], job.COL_RESPONSE)
        want, _, _ = CO.controller_get_ref(ready, consumed, w.lengths.astype(np.int32), job.COL_RESPONSE, job.TASK_INFER,
                                           w.N, w.token_budget)
        task, first = job.cl_history[0]
        assert task == job.TASK_INFER and np.array_equal(first, np.asarray(want, dtype=np.int32))
        tasks = [t for t, _ in job.cl_history]
        assert tasks.index(job.TASK_UPDATE) > tasks.index(job.TASK_INFER)
    finally:
        job.ctx.close()
