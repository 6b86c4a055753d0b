"""af_unpack_microbatch (results written back to the store by index list) against the oracle, bit
for bit, and the three RL tasks of the paper's workflow run through one store and one status table:
reference inference and actor inference score micro-batches and write their log-probs back, the
actor update consumes samples once both columns are there."""
import numpy as np
import pytest
import torch

from oracle import controller_oracle as C
from oracle import grpo_oracle as O
from paper_2507_01663_b200 import workloads as wl
from gpu_util import GRAD_RTOL, LOGP_TOL, LOSS_RTOL, device, f32, i32, np_of, packed_buffers, rel

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2507_01663_b200 import binding as B
    c = B.Context(0)
    yield c
    c.close()


def make_store(seed, N, max_len):
    rng = np.random.default_rng(seed)
    lengths = rng.integers(0, max_len + 1, size=N)
    off = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int64)
    tot = int(off[-1])
    cols = {"a": rng.standard_normal(tot).astype(np.float32), "b": rng.integers(-5, 1 << 30, size=tot).astype(np.int32)}
    return rng, off, cols


@pytest.mark.parametrize("N,B,max_len", [(1, 1, 5), (9, 4, 7), (300, 300, 40), (2000, 1234, 300), (50, 0, 9), (64, 64, 0)])
def test_unpack_matches_oracle(ctx, N, B, max_len):
    rng, off, cols = make_store(N + B, N, max_len)
    idx = rng.permutation(N)[:B].astype(np.int32)
    T = int(sum(off[i + 1] - off[i] for i in idx))
    res = {"a": rng.standard_normal(T).astype(np.float32), "b": rng.integers(0, 99, size=T).astype(np.int32)}
    want = {k: v.copy() for k, v in cols.items()}
    assert O.unpack_microbatch_ref(off, idx, res, want) == T
    dev_store = {"a": f32(cols["a"]), "b": i32(cols["b"])}
    got_T = ctx.unpack_microbatch(off, idx, [f32(res["a"]), i32(res["b"])], [dev_store["a"], dev_store["b"]])
    assert got_T == T
    assert np_of(dev_store["a"]).tobytes() == want["a"].tobytes()
    assert np_of(dev_store["b"]).tobytes() == want["b"].tobytes()
    assert ctx.check_device_errors() == 0


def test_unpack_undoes_pack_and_sets_status_bits(ctx):
    rng, off, cols = make_store(5, 400, 60)
    N = 400
    idx = rng.permutation(N)[:150].astype(np.int32)
    dev = device()
    src = f32(cols["a"])
    out = packed_buffers(int(off[-1]), 150, 8)
    store = {"tok_offset_host": off, "d": 8, "old_logp": src}
    T = ctx.pack_microbatch(store, idx, {"cu_seqlens": out["cu_seqlens"], "old_logp": out["old_logp"]})
    dst = torch.zeros_like(src)
    tab = {"ready": torch.full((N,), 0b100, dtype=torch.int32, device=dev),
           "consumed": torch.zeros(N, dtype=torch.int32, device=dev)}
    assert ctx.unpack_microbatch(off, idx, [out["old_logp"]], [dst], table=tab, column_bits=0b011) == T
    want = np.zeros_like(cols["a"])
    rdy = np.full(N, 0b100, np.uint32)
    for i in idx:
        want[off[i]:off[i + 1]] = cols["a"][off[i]:off[i + 1]]
    C.controller_put_ref(rdy, idx, 0b011)
    assert np_of(dst).tobytes() == want.tobytes()
    assert np.array_equal(np_of(tab["ready"]).view(np.uint32), rdy)
    assert ctx.check_device_errors() == 0


def test_unpack_argument_errors(ctx):
    from paper_2507_01663_b200 import binding as B
    off = np.array([0, 3, 5, 9], np.int64)
    col, res = torch.zeros(9, device=device()), torch.ones(9, device=device())
    for bad in ([0, 3], [-1], [1, 1], [0, 2, 0]):
        with pytest.raises(B.AfError):
            ctx.unpack_microbatch(off, np.array(bad, np.int32), [res], [col])
    with pytest.raises(B.AfError):                                # five columns
        ctx.unpack_microbatch(off, np.array([0], np.int32), [res] * 5, [col] * 5)
    tab = {"ready": torch.zeros(2, dtype=torch.int32, device=device()),
           "consumed": torch.zeros(2, dtype=torch.int32, device=device())}
    with pytest.raises(B.AfError):                                # status table of another store
        ctx.unpack_microbatch(off, np.array([0], np.int32), [res], [col], table=tab, column_bits=1)
    assert float(col.abs().max()) == 0.0                          # nothing was written by the refused calls
    assert ctx.unpack_microbatch(off, np.array([2, 0], np.int32), [res], [col]) == 7
    assert np_of(col).tolist() == [1, 1, 1, 0, 0, 1, 1, 1, 1]
    assert ctx.check_device_errors() == 0


COL_RESP, COL_REF, COL_OLD = 1, 2, 4
TASK_REF, TASK_ACTOR_INF, TASK_UPDATE = 1, 2, 4


def test_three_tasks_through_one_store(ctx):
    """Responses arrive in waves.  Reference inference and actor inference each ask the controller
    for ready responses they have not seen, gather them, score them and write the log-probs back
    with the status bit of their column; the actor update asks for responses whose two log-prob
    columns are both there and runs the fused update.  Every request, every written column and
    the accumulated gradient are checked against the oracles."""
    from paper_2507_01663_b200 import binding as Bn
    dev = device()
    w = wl.make_workload("cfg5_mini")
    N, d, V = w.N, w.d, w.V
    off, lengths = w.tok_offset, w.lengths.astype(np.int32)
    H, W, y = wl.gen_hidden(w), wl.gen_weight(w), wl.gen_target(w)
    W_ref = wl._normal_matrix(w.seed + 77, wl.S_W, V, d, 0.02, "cpu")          # the frozen reference policy
    reward = wl.gen_reward(w)
    adv_ref = O.grpo_advantage_ref(np_of(reward), w.group_id, w.n_prompts).astype(np.float32)
    Ttot = int(off[-1])
    store = {"tok_offset_host": off, "d": d, "hidden": H.to(dev), "target": y.to(dev),
             "old_logp": torch.zeros(Ttot, device=dev), "ref_logp": torch.zeros(Ttot, device=dev),
             "adv": torch.empty(N, device=dev)}
    ctx.grpo_advantage(reward.to(dev), None, w.n_prompts, store["adv"])
    tab = {"ready": torch.zeros(N, dtype=torch.int32, device=dev), "consumed": torch.zeros(N, dtype=torch.int32, device=dev),
           "length": torch.as_tensor(lengths, device=dev)}
    rdy, con = np.zeros(N, np.uint32), np.zeros(N, np.uint32)
    host_old, host_ref = np.zeros(Ttot, np.float32), np.zeros(Ttot, np.float32)
    Wd, Wrd = W.to(dev), W_ref.to(dev)
    packed = packed_buffers(Ttot, N, d)
    logp, ent, lse = (torch.empty(Ttot, device=dev) for _ in range(3))
    out_idx, res = torch.empty(N, dtype=torch.int32, device=dev), Bn.new_get_result(dev)
    dH = torch.empty(Ttot, d, dtype=torch.bfloat16, device=dev)
    dW = torch.zeros(V, d, device=dev)
    dW_ref = np.zeros((V, d))
    loss_out = Bn.new_loss_out(dev)
    budget = 1024
    arrival = wl.arrival_order(w)
    waves = np.array_split(arrival, 5)
    updated = 0

    def request(task, mask):
        ctx.controller_get(tab, mask, task, N, budget, out_idx, res)
        r = Bn.read_get_result(res)
        want, tokens, eligible = C.controller_get_ref(rdy, con, lengths, mask, task, N, budget)
        got = np_of(out_idx)[: r["count"]]
        assert r["count"] == len(want) and r["tokens"] == tokens and r["eligible"] == eligible
        assert np.array_equal(got, np.asarray(want, dtype=np.int32))
        return got

    def score_and_write_back(task, weights_dev, weights_cpu, column, bit, host_col):
        while True:
            mb = request(task, COL_RESP)
            if len(mb) == 0:
                return
            T = ctx.pack_microbatch(store, mb, packed)
            ctx.token_logprob(packed["hidden"], weights_dev, packed["target"], logp, ent, lse, T=T)
            assert ctx.unpack_microbatch(off, mb, [logp], [store[column]], table=tab, column_bits=bit) == T
            p = O.pack_microbatch_ref(off, mb, {"hidden": wl.bf16_bits(H), "target": y.numpy()})
            lp, _, _ = O.token_logprob_ref(p["hidden"], wl.bf16_bits(weights_cpu), p["target"])
            got = np_of(logp)[:T]
            assert np.abs(got - lp).max() <= LOGP_TOL
            # the store column now holds, bit for bit, what the device computed for these samples
            O.unpack_microbatch_ref(off, mb, {"c": got}, {"c": host_col})
            C.controller_put_ref(rdy, mb, bit)
            assert np_of(store[column]).tobytes() == host_col.tobytes()

    for wave in waves:
        ctx.controller_put(tab, torch.as_tensor(wave.astype(np.int32), device=dev), COL_RESP)   # rollouts land
        C.controller_put_ref(rdy, wave, COL_RESP)
        score_and_write_back(TASK_REF, Wrd, W_ref, "ref_logp", COL_REF, host_ref)
        score_and_write_back(TASK_ACTOR_INF, Wd, W, "old_logp", COL_OLD, host_old)
        while True:                                                   # the actor update
            mb = request(TASK_UPDATE, COL_RESP | COL_REF | COL_OLD)
            if len(mb) == 0:
                break
            T = ctx.pack_microbatch(store, mb, packed)
            ctx.policy_update(packed["hidden"], Wd, packed["target"], packed["old_logp"], packed["ref_logp"],
                              packed["adv_seq"], packed["cu_seqlens"], loss_out, logp, lse, dH, dW, entropy=ent,
                              accumulate_dW=True, clip_lo=w.clip_eps, clip_hi=w.clip_eps, kl_coef=w.kl_coef,
                              B=len(mb), T=T)
            p = O.pack_microbatch_ref(off, mb, {"hidden": wl.bf16_bits(H), "target": y.numpy(), "old": host_old,
                                                "ref": host_ref}, adv_ref)
            oref = O.policy_loss_ref(np_of(logp)[:T], p["old"], p["ref"], p["adv_seq"], p["cu_seqlens"], w.clip_eps,
                                     w.clip_eps, w.kl_coef)
            got = Bn.read_loss_out(loss_out)
            scale = max(abs(oref["pg_loss"]), abs(oref["kl_mean"]), 1e-3)
            assert abs(got["loss"] - oref["loss"]) <= LOSS_RTOL * max(abs(oref["loss"]), scale)
            _, dW_mb = O.policy_loss_backward_ref(p["hidden"], wl.bf16_bits(W), p["target"], np_of(lse)[:T], oref["dlogp"])
            dW_ref += dW_mb
            updated += len(mb)
    assert updated == N                                               # every response trained on exactly once
    assert np.all(con == (TASK_REF | TASK_ACTOR_INF | TASK_UPDATE))
    assert np.array_equal(np_of(tab["consumed"]).view(np.uint32), con)
    assert np.array_equal(np_of(tab["ready"]).view(np.uint32), rdy)
    assert np.linalg.norm(np_of(dW) - dW_ref) <= GRAD_RTOL * np.linalg.norm(dW_ref)
    assert ctx.check_device_errors() == 0
