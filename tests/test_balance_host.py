"""af_balance_partitions (a host call of the C ABI: needs no GPU) against the oracle: the stated
tie-breaks make the partition unique, so it is compared index by index."""
import numpy as np
import pytest

from oracle import controller_oracle as C
from paper_2507_01663_b200 import workloads as wl


@pytest.fixture(scope="module")
def balance():
    from paper_2507_01663_b200 import build as b
    b.build()
    from paper_2507_01663_b200 import binding
    return binding.balance_partitions


@pytest.mark.parametrize("equal", [True, False])
@pytest.mark.parametrize("name,k", [("cfg1", 4), ("cfg2", 8), ("cfg3", 8), ("cfg5", 16), ("cfg5_mini", 3), ("cfg3_mini", 7)])
def test_partition_of_workload_lengths_matches_oracle(balance, name, k, equal):
    L = wl.make_workload(name).lengths
    part, sums = balance(L, k, equal)
    ref = C.kk_partition_ref(L, k, equal)
    assert np.array_equal(part, ref)
    assert np.array_equal(sums, C.group_sums(L, ref, k))
    assert list(sums) == sorted(sums, reverse=True)
    if equal:
        counts = np.bincount(part, minlength=k)
        assert counts.max() - counts.min() <= 1


@pytest.mark.parametrize("seed", range(20))
def test_random_small_cases_with_many_ties(balance, seed):
    r = np.random.default_rng(seed)
    n, k = int(r.integers(0, 40)), int(r.integers(1, 7))
    L = r.integers(0, 6, n)                        # few distinct values: ties everywhere
    for equal in (True, False):
        part, sums = balance(L, k, equal)
        assert np.array_equal(part, C.kk_partition_ref(L, k, equal))
        assert sums.sum() == L.sum()


def test_micro_batch_of_the_streaming_store(balance):
    """The use the paper describes: a batch handed out by the controller is split over the
    data-parallel groups of the task with equal sample counts and near-equal token totals."""
    w = wl.make_workload("cfg5")
    mb = wl.microbatches(w)[3]
    mb = mb[: len(mb) // 4 * 4]
    L = w.lengths[mb]
    part, sums = balance(L, 4, True)
    assert set(np.bincount(part, minlength=4).tolist()) == {len(mb) // 4}
    assert np.array_equal(part, C.kk_partition_ref(L, 4, True))


def test_argument_errors(balance):
    from paper_2507_01663_b200 import binding as B
    lib = B.load_library()
    assert lib.af_balance_partitions(None, 3, 2, 0, None, None) == -1
    assert lib.af_balance_partitions(None, -1, 2, 0, None, None) == -1
    assert lib.af_balance_partitions(None, 0, 0, 0, None, None) == -1
    assert lib.af_balance_partitions(None, 0, 2, 0, None, None) == 0        # empty batch is valid
    with pytest.raises(B.AfError):
        balance(np.array([3, -1, 2]), 2, False)
