"""Pins for the controller oracle (status-table put/get, Karmarkar-Karp balancing): what the
definitions and the published behaviour of the differencing method fix, independently of the
oracle's own loops."""
import itertools

import numpy as np
import pytest

from oracle import controller_oracle as C


def rng_table(seed, n, n_cols=5, n_tasks=3):
    r = np.random.default_rng(seed)
    ready = r.integers(0, 1 << n_cols, n).astype(np.uint32)
    consumed = r.integers(0, 1 << n_tasks, n).astype(np.uint32)
    length = r.integers(1, 200, n).astype(np.int32)
    return ready, consumed, length


# ---------------------------------------------------------------- get: eligibility and prefix
@pytest.mark.parametrize("seed", range(6))
def test_get_matches_set_definitions(seed):
    n = 300
    ready, consumed, length = rng_table(seed, n)
    mask, task, max_s, budget = 0b00101, 0b010, 17, 900 + 100 * seed
    before = consumed.copy()
    idx, tokens, n_elig = C.controller_get_ref(ready, consumed, length, mask, task, max_s, budget)
    # eligibility written as sets: every requested column ready, never handed to this task
    elig = [i for i in range(n) if all((ready[i] >> c) & 1 for c in (0, 2)) and not (before[i] >> 1) & 1]
    assert n_elig == len(elig)
    # the answer is a prefix of the eligible sequence ...
    assert list(idx) == elig[:len(idx)]
    # ... within both limits, and the longest one: the next eligible sample would break a limit
    assert len(idx) <= max_s and tokens == int(length[idx].sum())
    assert tokens <= budget or len(idx) == 1
    if len(idx) < len(elig):
        nxt = elig[len(idx)]
        assert len(idx) == max_s or tokens + int(length[nxt]) > budget
    # consumption record: exactly the returned samples gained exactly this task's bit
    changed = np.nonzero(consumed != before)[0]
    assert list(changed) == list(idx)
    assert np.all((consumed[idx] ^ before[idx]) == task)


def test_get_sample_longer_than_budget_goes_alone():
    ready = np.full(4, 1, np.uint32)
    consumed = np.zeros(4, np.uint32)
    length = np.array([50, 7, 7, 7], np.int32)
    idx, tokens, _ = C.controller_get_ref(ready, consumed, length, 1, 1, 10, 20)
    assert list(idx) == [0] and tokens == 50
    idx, tokens, _ = C.controller_get_ref(ready, consumed, length, 1, 1, 10, 20)
    assert list(idx) == [1, 2] and tokens == 14          # 7 + 7 + 7 > 20


def test_get_without_budget_counts_samples_only():
    ready = np.full(10, 3, np.uint32)
    consumed = np.zeros(10, np.uint32)
    idx, tokens, n_elig = C.controller_get_ref(ready, consumed, None, 3, 4, 4, 0)
    assert list(idx) == [0, 1, 2, 3] and tokens == 0 and n_elig == 10


@pytest.mark.parametrize("seed", range(4))
def test_every_sample_reaches_every_task_exactly_once(seed):
    """Production and consumption interleaved: columns arrive in random order, two tasks with
    different column needs poll; each task ends up with every sample exactly once."""
    r = np.random.default_rng(seed)
    n = 200
    ready = np.zeros(n, np.uint32)
    consumed = np.zeros(n, np.uint32)
    length = r.integers(1, 100, n).astype(np.int32)
    needs = {1: 0b011, 2: 0b110}                       # task bit -> columns
    got = {1: [], 2: []}
    events = [(i, c) for i in range(n) for c in range(3)]
    r.shuffle(events)
    for step, (i, c) in enumerate(events):
        C.controller_put_ref(ready, [i], 1 << c)
        if step % 7 == 0:
            for t, m in needs.items():
                idx, _, _ = C.controller_get_ref(ready, consumed, length, m, t, 16, 500)
                assert all((int(ready[j]) & m) == m for j in idx)     # never before its columns exist
                got[t].extend(idx.tolist())
    for t, m in needs.items():
        while True:
            idx, _, _ = C.controller_get_ref(ready, consumed, length, m, t, 16, 500)
            if len(idx) == 0:
                break
            got[t].extend(idx.tolist())
        assert sorted(got[t]) == list(range(n))


def test_put_is_idempotent_and_additive():
    ready = np.zeros(5, np.uint32)
    C.controller_put_ref(ready, [1, 3, 3], 0b01)
    C.controller_put_ref(ready, [3], 0b10)
    assert ready.tolist() == [0, 1, 0, 3, 0]


# ---------------------------------------------------------------- Karmarkar-Karp
def numbers_only_differencing(values):
    """Two-way differencing in its original form: replace the two largest numbers by their
    difference until one number is left; that number is the difference of the two sums."""
    v = sorted(values)
    while len(v) > 1:
        a, b = v.pop(), v.pop()
        v.append(a - b)
        v.sort()
    return v[0] if v else 0


def test_kk_textbook_example():
    # the standard illustration of the method: {8,7,6,5,4} ends with a difference of 2
    # (8-7=1, 6-5=1, 4-1=3, 3-1=2), although {8,7} | {6,5,4} would be perfect
    L = [8, 7, 6, 5, 4]
    part = C.kk_partition_ref(L, 2, equal_size=False)
    s = C.group_sums(L, part, 2)
    assert abs(int(s[0]) - int(s[1])) == 2 and s.sum() == 30


@pytest.mark.parametrize("seed", range(8))
def test_kk_two_way_equals_numbers_only_form(seed):
    r = np.random.default_rng(seed)
    L = r.integers(1, 1000, int(r.integers(2, 40))).tolist()
    part = C.kk_partition_ref(L, 2, equal_size=False)
    s = C.group_sums(L, part, 2)
    assert abs(int(s[0]) - int(s[1])) == numbers_only_differencing(L)
    assert abs(int(s[0]) - int(s[1])) <= max(L)            # the method's classical guarantee


def brute_force_best_spread(L, k, equal_size):
    best = None
    n = len(L)
    for assign in itertools.product(range(k), repeat=n):
        if equal_size and len(set(np.bincount(assign, minlength=k).tolist())) != 1:
            continue
        s = np.bincount(assign, weights=L, minlength=k)
        spread = s.max() - s.min()
        best = spread if best is None else min(best, spread)
    return best


@pytest.mark.parametrize("k,n,equal", [(2, 8, False), (3, 7, False), (2, 8, True), (3, 6, True), (4, 8, True)])
def test_kk_valid_and_no_better_than_the_optimum(k, n, equal):
    for seed in range(5):
        r = np.random.default_rng(100 * k + seed)
        L = r.integers(1, 60, n).tolist()
        part = C.kk_partition_ref(L, k, equal)
        assert part.shape == (n,) and part.min() >= 0 and part.max() < k
        s = C.group_sums(L, part, k)
        assert s.sum() == sum(L)                                           # exact cover
        if equal:
            assert set(np.bincount(part, minlength=k).tolist()) == {n // k}  # equal sample counts
        opt = brute_force_best_spread(L, k, equal)
        assert s.max() - s.min() >= opt
        # a heuristic, but a good one: never worse than the largest item off the optimum
        assert s.max() - s.min() <= opt + max(L)


def test_kk_equal_items_and_scaling():
    part = C.kk_partition_ref([5] * 12, 4, equal_size=True)
    assert C.group_sums([5] * 12, part, 4).tolist() == [15, 15, 15, 15]
    L = [13, 9, 40, 22, 7, 31, 18, 3]
    p1 = C.kk_partition_ref(L, 3, False)
    p2 = C.kk_partition_ref([7 * x for x in L], 3, False)
    assert np.array_equal(p1, p2)                                          # scale-free decisions


def test_kk_equal_size_with_ragged_tail_and_groups_sorted():
    L = [10, 9, 8, 7, 6, 5, 4]                                             # 7 items, 3 groups
    part = C.kk_partition_ref(L, 3, equal_size=True)
    counts = np.bincount(part, minlength=3)
    assert counts.max() - counts.min() <= 1
    s = C.group_sums(L, part, 3)
    assert list(s) == sorted(s, reverse=True)                              # group g = g-th largest sum


def test_kk_beats_arrival_order_on_long_tailed_lengths():
    """On long-tailed length mixes (the case the paper's load balancing is for) the token spread
    across 8 groups collapses against dealing samples out round-robin.  With equal sample counts
    the method starts from runs of 8 consecutive sorted items, so a run holding one giant item
    bounds what it can repair: on a Pareto tail the equal-count variant is only somewhat better
    than round-robin, while the free variant is near-perfect; on a lognormal mix both are."""
    r = np.random.default_rng(7)
    pareto = np.minimum(np.floor(128 * (1 - r.random(512)) ** (-1 / 1.5)), 16384).astype(np.int64)
    lognormal = np.clip(np.rint(np.exp(np.log(1024) + r.standard_normal(512))), 64, 8192).astype(np.int64)
    for L, dp_factor in ((pareto, 0.7), (lognormal, 0.001)):
        rr = C.group_sums(L, np.arange(512) % 8, 8)
        rr_spread = rr.max() - rr.min()
        dp = C.kk_partition_ref(L, 8, equal_size=True)
        s = C.group_sums(L, dp, 8)
        assert set(np.bincount(dp, minlength=8).tolist()) == {64}
        assert s.max() - s.min() < dp_factor * rr_spread
        pp = C.kk_partition_ref(L, 8, equal_size=False)
        s = C.group_sums(L, pp, 8)
        assert s.max() - s.min() < 0.001 * rr_spread
