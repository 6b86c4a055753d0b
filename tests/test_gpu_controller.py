"""af_controller_put / get / clear against the oracle: integer work, compared bit for bit
(returned indices, the result record and the whole status table after every request)."""
import numpy as np
import pytest
import torch

from oracle import controller_oracle as C
from paper_2507_01663_b200 import workloads as wl
from gpu_util import device, np_of

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2507_01663_b200 import binding as B
    c = B.Context(0)
    yield c
    c.close()


def u32_table(seed, n, p_ready=0.8, n_cols=4, n_tasks=3, max_len=300):
    """Seeded status table: each column bit on with probability p_ready, a few consumption bits."""
    bits = wl.counter_bits(seed, wl.S_MISC, 0, max(n, 1))[:n]
    u = wl.uniform01(seed, wl.S_MISC, 1 << 20, max(n * n_cols, 1))[: n * n_cols].view(n, n_cols) if n else torch.zeros(0, n_cols)
    ready = torch.zeros(n, dtype=torch.int64)
    for c in range(n_cols):
        ready |= (u[:, c] < p_ready).to(torch.int64) << c
    consumed = (bits >> 7) & ((1 << n_tasks) - 1) & ((bits >> 20) & ((1 << n_tasks) - 1))
    length = wl.randint(seed, wl.S_LEN, 0, max(n, 1), max_len)[:n] + 1
    return (ready.numpy().astype(np.uint32), consumed.numpy().astype(np.uint32), length.numpy().astype(np.int32))


def dev_table(ready, consumed, length, offset=0):
    """Device copies (as int32 bit patterns); ``offset`` shifts the base pointers off 16 bytes."""
    dev = device()
    def up(a):
        t = torch.zeros(a.shape[0] + offset, dtype=torch.int32, device=dev)
        t[offset:] = torch.as_tensor(a.view(np.int32), device=dev)
        return t[offset:]
    return {"ready": up(ready), "consumed": up(consumed), "length": up(length)}


def one_get(ctx, tab, host, mask, task, max_s, budget):
    from paper_2507_01663_b200 import binding as B
    dev = device()
    ready, consumed, length = host
    out_idx = torch.full((max(max_s, 1),), -7, dtype=torch.int32, device=dev)
    out = B.new_get_result(dev)
    ctx.controller_get(tab, mask, task, max_s, budget, out_idx, out)
    res = B.read_get_result(out)
    idx_ref, tok_ref, elig_ref = C.controller_get_ref(ready, consumed, length, mask, task, max_s, budget)
    assert res["count"] == len(idx_ref) and res["eligible"] == elig_ref
    assert res["tokens"] == tok_ref
    got = np_of(out_idx)
    assert np.array_equal(got[:res["count"]], idx_ref)
    assert np.all(got[res["count"]:] == -7)                          # nothing written past the result
    assert np.array_equal(np_of(tab["consumed"]).view(np.uint32), consumed)   # table state, every entry
    assert np.array_equal(np_of(tab["ready"]).view(np.uint32), ready)
    return idx_ref


@pytest.mark.parametrize("n", [0, 1, 3, 4, 5, 1023, 1024, 1025, 4096, 16384, 16385, 100003, 1 << 20])
def test_get_matches_oracle_across_table_sizes(ctx, n):
    host = u32_table(n + 1, n)
    tab = dev_table(*host)
    host = (host[0], host[1], host[2].copy())
    # repeated requests of two tasks with different needs and limits drain the table in order
    for rnd, (mask, task, max_s, budget) in enumerate([(0b0011, 1, 64, 5000), (0b0110, 2, 1000, 0),
                                                       (0b0011, 1, 7, 100000), (0b1111, 4, 100000, 0),
                                                       (0b0011, 1, 300, 20000), (0b0001, 2, 50, 1)]):
        one_get(ctx, tab, (host[0], host[1], host[2]), mask, task, max_s, budget)
    assert ctx.check_device_errors() == 0


@pytest.mark.parametrize("offset", [1, 2, 3])
def test_get_with_unaligned_tables(ctx, offset):
    host = u32_table(77, 20001)
    tab = dev_table(*host, offset=offset)
    one_get(ctx, tab, host, 0b0101, 2, 5000, 300000)
    one_get(ctx, tab, host, 0b0101, 2, 5000, 300000)


@pytest.mark.parametrize("n", [300000, 5000003])
def test_selection_ends_deep_inside_a_large_table(ctx, n):
    """The prefix ends in a late block of the two-pass path: count limit, then token limit.  At the
    larger size a block's segment spans several tiles and the first eligible sample sits in the
    middle of one, after tiles the second pass does not visit."""
    ready = np.full(n, 1, np.uint32)
    ready[: n - 5000] = 0                                            # only the last 5000 samples are ready
    consumed = np.zeros(n, np.uint32)
    length = np.full(n, 10, np.int32)
    tab = dev_table(ready, consumed, length)
    host = (ready, consumed, length)
    a = one_get(ctx, tab, host, 1, 1, 1200, 0)
    b = one_get(ctx, tab, host, 1, 1, 100000, 10 * 777)
    assert a[0] == n - 5000 and len(a) == 1200 and len(b) == 777 and b[0] == a[-1] + 1


def test_budget_smaller_than_first_sample(ctx):
    ready = np.full(6, 1, np.uint32)
    consumed = np.zeros(6, np.uint32)
    length = np.array([50, 7, 7, 7, 0, 3], np.int32)
    tab = dev_table(ready, consumed, length)
    host = (ready, consumed, length)
    assert list(one_get(ctx, tab, host, 1, 1, 10, 20)) == [0]
    assert list(one_get(ctx, tab, host, 1, 1, 10, 20)) == [1, 2]
    assert list(one_get(ctx, tab, host, 1, 1, 10, 20)) == [3, 4, 5]
    assert list(one_get(ctx, tab, host, 1, 1, 10, 20)) == []
    assert list(one_get(ctx, tab, host, 1, 1, 0, 0)) == []          # zero samples requested


def test_streaming_production_and_consumption(ctx):
    """The streaming store workload through the controller: responses arrive in waves (put), the
    scoring task polls with a 32768-token budget (get) and reports its result column (put); a
    second task waits for that column.  Both see every sample exactly once, every batch within
    the budget, and the device follows the oracle request for request."""
    from paper_2507_01663_b200 import binding as B
    dev = device()
    w = wl.make_workload("cfg5")
    n = w.N
    ready, consumed = np.zeros(n, np.uint32), np.zeros(n, np.uint32)
    length = w.lengths.astype(np.int32)
    tab = dev_table(ready, consumed, length)
    host = (ready, consumed, length)
    COL_RESP, COL_LOGP, SCORER, TRAINER = 1, 2, 1, 2
    arrival = wl.arrival_order(w)
    scored, trained = [], []
    for s in range(0, n, 512):
        wave = arrival[s:s + 512]
        ctx.controller_put(tab, torch.as_tensor(wave, device=dev), COL_RESP)
        C.controller_put_ref(ready, wave, COL_RESP)
        for _ in range(4):
            idx = one_get(ctx, tab, host, COL_RESP, SCORER, 4096, w.token_budget)
            if len(idx) == 0:
                break
            assert int(length[idx].sum()) <= w.token_budget or len(idx) == 1
            scored.extend(idx.tolist())
            ctx.controller_put(tab, torch.as_tensor(idx, device=dev), COL_LOGP)     # result written back
            C.controller_put_ref(ready, idx, COL_LOGP)
        idx = one_get(ctx, tab, host, COL_RESP | COL_LOGP, TRAINER, 256, 0)
        assert set(idx.tolist()) <= set(scored)
        trained.extend(idx.tolist())
    while True:
        idx = one_get(ctx, tab, host, COL_RESP, SCORER, 4096, w.token_budget)
        if len(idx) == 0:
            break
        scored.extend(idx.tolist())
        ctx.controller_put(tab, torch.as_tensor(idx, device=dev), COL_LOGP)
        C.controller_put_ref(ready, idx, COL_LOGP)
    while True:
        idx = one_get(ctx, tab, host, COL_RESP | COL_LOGP, TRAINER, 256, 0)
        if len(idx) == 0:
            break
        trained.extend(idx.tolist())
    assert sorted(scored) == list(range(n)) and sorted(trained) == list(range(n))
    # next iteration: the table is cleared and fills again
    ctx.controller_clear(tab, COL_RESP | COL_LOGP, SCORER | TRAINER)
    assert not np_of(tab["ready"]).any() and not np_of(tab["consumed"]).any()
    assert ctx.check_device_errors() == 0


def test_put_flags_bad_indices_and_skips_them(ctx):
    from paper_2507_01663_b200 import binding as B
    dev = device()
    tab = dev_table(np.zeros(8, np.uint32), np.zeros(8, np.uint32), np.ones(8, np.int32))
    ctx.controller_put(tab, torch.tensor([1, 9, -1, 3, 3], dtype=torch.int32, device=dev), 0b10)
    assert ctx.check_device_errors() == B.DEVERR_SAMPLE_INDEX
    assert np_of(tab["ready"]).tolist() == [0, 2, 0, 2, 0, 0, 0, 0]
    assert ctx.check_device_errors() == 0


@pytest.mark.parametrize("n,offset", [(1, 0), (3, 0), (5000, 0), (5003, 0), (4099, 1), (1 << 20, 0), ((1 << 20) + 2, 3)])
def test_clear_is_selective(ctx, n, offset):
    ready, consumed, length = u32_table(n, n)
    tab = dev_table(ready | 0b010, consumed | 0b01, length, offset=offset)
    ctx.controller_clear(tab, 0b010, 0b01)
    assert np.array_equal(np_of(tab["ready"]).view(np.uint32), ready & ~np.uint32(0b010))
    assert np.array_equal(np_of(tab["consumed"]).view(np.uint32), consumed & ~np.uint32(0b01))
    ctx.controller_clear(tab, 0, 0b10)                              # one column only
    assert np.array_equal(np_of(tab["ready"]).view(np.uint32), ready & ~np.uint32(0b010))
    assert np.array_equal(np_of(tab["consumed"]).view(np.uint32), consumed & ~np.uint32(0b11))
    ctx.controller_clear(tab, 0, 0)                                 # nothing asked: nothing changes
    assert np.array_equal(np_of(tab["consumed"]).view(np.uint32), consumed & ~np.uint32(0b11))


def test_host_argument_errors(ctx):
    from paper_2507_01663_b200 import binding as B
    dev = device()
    tab = dev_table(np.zeros(8, np.uint32), np.zeros(8, np.uint32), np.ones(8, np.int32))
    out_idx, out = torch.zeros(4, dtype=torch.int32, device=dev), B.new_get_result(dev)
    for bad_task in (0, 3, 6):
        with pytest.raises(B.AfError):
            ctx.controller_get(tab, 1, bad_task, 4, 0, out_idx, out)
    with pytest.raises(B.AfError):
        ctx.controller_get(tab, 1, 1, -1, 0, out_idx, out)
    with pytest.raises(B.AfError):                                   # a token budget needs lengths
        ctx.controller_get({"ready": tab["ready"], "consumed": tab["consumed"]}, 1, 1, 4, 100, out_idx, out)
    with pytest.raises(B.AfError):
        ctx.controller_put(tab, out_idx, 1, n=-2)
    assert ctx.check_device_errors() == 0
