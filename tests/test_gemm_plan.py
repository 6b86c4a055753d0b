"""Work decomposition of the fused LM-head kernel, checked on the host (no GPU).

af_plan_token_logprob / af_plan_units expose how a scoring call is cut into units (row tile x
vocabulary range) and which units each persistent worker processes, plainly or by die.  What must
hold whatever the shape: every unit is processed exactly once; dealing by die never costs a round
of units; a row tile's units stay on one die."""
import numpy as np
import pytest

from paper_2507_01663_b200 import binding as B

HEADS = [(3584, 152064), (5120, 152064), (256, 4096), (512, 8200)]
DIE_SPLITS = [0, 74, 72, 76, 70, 78, 68, 80, 40, 108]


def units_of_all(plan):
    return [list(B.plan_units(plan, r)) for r in range(plan.workers)]


@pytest.mark.parametrize("d,V", HEADS)
def test_every_unit_exactly_once(d, V):
    rng = np.random.default_rng(d)
    sizes = [1, 127, 128, 129, 255, 256, 257, 1195, 9472, 18944, 32768, 62989, 65536, 1106674]
    sizes += [int(x) for x in rng.integers(1, 300000, size=12)]
    for T in sizes:
        for die0 in DIE_SPLITS:
            for variant in (0, 1, 2):
                plan = B.plan_token_logprob(T, d, V, 148, die0, 0, variant)
                total = plan.m_tiles * plan.v_splits
                tile_rows = 128 if variant == 1 else 256
                assert plan.m_tiles == -(-T // tile_rows) and plan.n_tiles == -(-V // 256)
                assert 1 <= plan.v_splits <= plan.n_tiles
                assert plan.workers == min(total, 148 if variant == 1 else 74)
                seen = np.zeros(total, dtype=np.int32)
                for us in units_of_all(plan):
                    for u in us:
                        assert 0 <= u < total
                        seen[u] += 1
                assert np.all(seen == 1), (T, die0, variant)
                if variant != 0 or die0 == 0:
                    assert plan.die0_workers == 0 or variant == 0


def test_dealing_by_die_keeps_rounds_and_row_tiles_on_one_die():
    for d, V in HEADS[:2]:
        for T in (9472, 32768, 62989, 65536, 200000, 1106674):
            for die0 in DIE_SPLITS[1:]:
                plan = B.plan_token_logprob(T, d, V, 148, die0)
                plain = B.plan_token_logprob(T, d, V, 148, 0, plan.v_splits)
                if plan.die0_workers == 0:
                    continue
                assert plan.die0_workers == die0 // 2 and 0 < plan.die0_row_tiles < plan.m_tiles
                rounds = max(len(us) for us in units_of_all(plan))
                assert rounds <= max(len(us) for us in units_of_all(plain)), (T, d, die0)
                # a row tile's units are all on the first die's workers, or all on the other's
                S, n0 = plan.v_splits, plan.die0_workers
                for r, us in enumerate(units_of_all(plan)):
                    for u in us:
                        assert (u // S < plan.die0_row_tiles) == (r < n0)


def test_requested_ranges_and_the_bench_shape():
    # a caller's number of ranges is taken as given (capped by the number of vocabulary tiles)
    assert B.plan_token_logprob(5000, 3584, 152064, 148, 72, 5).v_splits == 5
    assert B.plan_token_logprob(5000, 256, 4096, 148, 72, 99).v_splits == 16
    # the 7B head at the benchmark's batch: by die two ranges keep the hidden-state panels of a wave
    # within one die's share of L2; dealt plainly it takes three
    by_die = B.plan_token_logprob(1106674, 3584, 152064, 148, 72)
    plain = B.plan_token_logprob(1106674, 3584, 152064, 148, 0)
    assert (by_die.v_splits, plain.v_splits) == (2, 3)
    alive = -(-(by_die.workers - by_die.die0_workers) // by_die.v_splits)      # row tiles of the larger die in flight
    assert alive * 256 * 3584 * 2 <= 36 << 20
    assert B.plan_token_logprob(1106674, 5120, 152064, 148, 72).v_splits == 3


def test_plan_argument_errors():
    for bad in [(0, 64, 64, 148, 0), (5, 0, 64, 148, 0), (5, 64, 0, 148, 0), (5, 64, 64, 0, 0), (5, 64, 64, 148, 149),
                (5, 64, 64, 148, -1)]:
        with pytest.raises(B.AfError) as e:
            B.plan_token_logprob(*bad)
        assert e.value.status == -1
    with pytest.raises(B.AfError) as e:
        B.plan_token_logprob(1 << 31, 64, 64, 148)
    assert e.value.status == -2
    plan = B.plan_token_logprob(5000, 3584, 152064, 148, 72)
    for rank in (-1, plan.workers):
        with pytest.raises(B.AfError):
            B.plan_units(plan, rank)
