"""af_token_logprob against the fp64 oracle, element by element."""
import math

import numpy as np
import pytest
import torch

from oracle import grpo_oracle as O
from paper_2507_01663_b200 import workloads as wl
from gpu_util import LOGP_TOL, device, np_of

pytestmark = pytest.mark.gpu


VARIANT = 0    # which GEMM variant the helpers below select (0 = library default)


@pytest.fixture(autouse=True, params=[1, 2], ids=["cta", "pair"])
def gemm_variant(request):
    """Every test of this module runs on both tensor-core main loops: one CTA per 128 x 256
    tile and a CTA pair per 256 x 256 tile (the default)."""
    global VARIANT
    VARIANT = request.param
    yield
    VARIANT = 0


@pytest.fixture(scope="module")
def ctx():
    from paper_2507_01663_b200 import binding as B
    c = B.Context(0)
    yield c
    c.close()


def run_case(ctx, H, W, y, splits=0):
    dev = device()
    T = H.shape[0]
    Hd, Wd, yd = H.to(dev), W.to(dev), y.to(dev)
    logp, ent, lse = (torch.full((T,), 9.0, device=dev) for _ in range(3))
    ctx.set_tuning(splits, 0, VARIANT)
    ctx.token_logprob(Hd, Wd, yd, logp, ent, lse)
    flags = ctx.check_device_errors()
    ctx.set_tuning(0, 0)
    return np_of(logp), np_of(ent), np_of(lse), flags


def random_case(T, d, V, seed, w_scale=None):
    H = wl._normal_matrix(seed, wl.S_HIDDEN, T, d, 1.0, "cpu")
    W = wl._normal_matrix(seed, wl.S_W, V, d, w_scale if w_scale else 1.0 / math.sqrt(d), "cpu")
    y = wl.randint(seed, wl.S_TARGET, 0, T, V).to(torch.int32)
    return H, W, y


def check(ctx, H, W, y, splits=0):
    logp, ent, lse, flags = run_case(ctx, H, W, y, splits)
    r_logp, r_ent, r_lse = O.token_logprob_ref(wl.bf16_bits(H), wl.bf16_bits(W), y.numpy())
    assert flags == 0
    assert np.abs(logp - r_logp).max() <= LOGP_TOL
    assert np.abs(ent - r_ent).max() <= LOGP_TOL
    assert np.abs(lse - r_lse).max() <= LOGP_TOL


def test_cfg1_full(ctx):
    w = wl.make_workload("cfg1")
    check(ctx, wl.gen_hidden(w), wl.gen_weight(w), wl.gen_target(w))


@pytest.mark.parametrize("name", ["cfg2_mini", "cfg3_mini", "cfg5_mini"])
def test_mini_workloads(ctx, name):
    w = wl.make_workload(name)
    check(ctx, wl.gen_hidden(w), wl.gen_weight(w), wl.gen_target(w))


# T spans one row, a ragged tile, several tiles; V below / across / ragged past the 256-wide tile;
# d below, equal to and ragged past the 64-wide K block (d % 8 == 0 is the ABI's requirement)
@pytest.mark.parametrize("T,d,V", [(1, 8, 2), (5, 8, 10), (127, 64, 255), (128, 64, 256), (129, 72, 257),
                                   (300, 200, 1000), (777, 512, 8200), (1025, 1096, 3001), (2100, 3584, 2304)])
def test_shapes(ctx, T, d, V):
    check(ctx, *random_case(T, d, V, seed=T + d + V))


@pytest.mark.parametrize("splits", [1, 2, 3, 7, 16])
def test_vocabulary_split_counts_agree(ctx, splits):
    H, W, y = random_case(600, 256, 5000, seed=42)
    check(ctx, H, W, y, splits)


def test_targets_at_tile_and_split_edges(ctx):
    T, d, V = 512, 128, 2050
    H, W, _ = random_case(T, d, V, seed=7)
    edges = [0, 31, 32, 255, 256, 257, 511, 512, 1023, 1024, 1025, 2047, 2048, 2049]
    y = torch.tensor([edges[i % len(edges)] for i in range(T)], dtype=torch.int32)
    for splits in (1, 4, 9):
        check(ctx, H, W, y, splits)


def test_degenerate_distributions(ctx):
    T, d, V = 130, 64, 700
    H, _, y = random_case(T, d, V, seed=3)
    # zero weights: uniform distribution, logp = -ln V, entropy = ln V
    logp, ent, lse, flags = run_case(ctx, H, torch.zeros(V, d, dtype=torch.bfloat16), y)
    assert flags == 0 and np.abs(logp + math.log(V)).max() < 1e-5 and np.abs(ent - math.log(V)).max() < 1e-5
    # one dominant logit (|z| ~ 500): logp -> 0 at the winner, very negative elsewhere, entropy -> 0
    Hd = torch.full((T, d), 1.0, dtype=torch.bfloat16)
    Wd = torch.zeros(V, d, dtype=torch.bfloat16)
    Wd[5] = 8.0
    yd = torch.full((T,), 5, dtype=torch.int32)
    yd[1::2] = 6
    check(ctx, Hd, Wd, yd)
    # large negative and positive logits together, identical rows give identical results
    Wm = wl._normal_matrix(5, wl.S_W, V, d, 1.5, "cpu")
    Hs = H[:1].repeat(T, 1).contiguous()
    logp, ent, lse, _ = run_case(ctx, Hs, Wm, torch.full((T,), 9, dtype=torch.int32))
    assert np.all(logp == logp[0]) and np.all(ent == ent[0])
    check(ctx, Hs, Wm, torch.full((T,), 9, dtype=torch.int32))


def test_target_out_of_range_is_flagged_not_faulted(ctx):
    from paper_2507_01663_b200 import binding as B
    H, W, y = random_case(200, 64, 300, seed=11)
    y[3] = 300
    y[150] = -1
    logp, ent, lse, flags = run_case(ctx, H, W, y)
    assert flags & B.DEVERR_TARGET_RANGE
    assert np.isnan(logp[3]) and np.isnan(logp[150]) and np.isfinite(np.delete(logp, [3, 150])).all()
    y[3], y[150] = 0, 1
    r = O.token_logprob_ref(wl.bf16_bits(H), wl.bf16_bits(W), y.numpy())
    assert np.abs(np.delete(logp, [3, 150]) - np.delete(r[0], [3, 150])).max() <= LOGP_TOL
    assert np.abs(ent - r[1]).max() <= LOGP_TOL           # entropy does not depend on the target
    assert ctx.check_device_errors() == 0                 # the word is cleared by the read


def test_host_argument_errors(ctx):
    from paper_2507_01663_b200.binding import AfError
    dev = device()
    H = torch.zeros(4, 12, dtype=torch.bfloat16, device=dev)     # d % 8 != 0
    W = torch.zeros(16, 12, dtype=torch.bfloat16, device=dev)
    y = torch.zeros(4, dtype=torch.int32, device=dev)
    out = torch.zeros(4, device=dev)
    with pytest.raises(AfError) as e:
        ctx.token_logprob(H, W, y, out)
    assert e.value.status == -3
    H8 = torch.zeros(4, 16, dtype=torch.bfloat16, device=dev)
    W8 = torch.zeros(16, 16, dtype=torch.bfloat16, device=dev)
    buf = torch.zeros(4 * 16 + 8, dtype=torch.bfloat16, device=dev)
    with pytest.raises(AfError) as e:
        ctx.token_logprob(buf[4:4 + 64].view(4, 16), W8, y, out)   # base pointer 8 bytes off
    assert e.value.status == -3
    ctx.token_logprob(H8, W8, y, out, T=0)                        # empty batch is a no-op
    assert ctx.check_device_errors() == 0


def test_bitwise_reproducible(ctx):
    H, W, y = random_case(900, 256, 4096, seed=21)
    a = run_case(ctx, H, W, y)
    b = run_case(ctx, H, W, y)
    for x, z in zip(a[:3], b[:3]):
        assert x.tobytes() == z.tobytes()


def test_weights_swapped_between_microbatches(ctx):
    """Delayed parameter update: while micro-batches are scored with the old LM-head weight, the
    new one is loaded into a standby buffer on a second stream; after the swap at a micro-batch
    boundary the results are those of the new weight, before it those of the old one, bit for bit
    (the load does not disturb the scoring in flight)."""
    dev = device()
    H, W0, y = random_case(640, 256, 4104, seed=21)
    _, W1, _ = random_case(640, 256, 4104, seed=22)
    Hd, yd = H.to(dev), y.to(dev)
    ctx.set_tuning(0, 0, VARIANT)

    def score(Wd, rows):
        out = torch.empty(rows.stop - rows.start, device=dev)
        ctx.token_logprob(Hd[rows], Wd, yd[rows], out)
        return out

    ref0 = [score(W0.to(dev), r) for r in (slice(0, 300), slice(300, 640))]
    ref1 = [score(W1.to(dev), r) for r in (slice(0, 300), slice(300, 640))]
    torch.cuda.synchronize()
    active, standby = W0.to(dev), torch.empty_like(W0, device=dev)
    W1_host = W1.pin_memory()
    side, loaded = torch.cuda.Stream(), torch.cuda.Event()
    with torch.cuda.stream(side):
        standby.copy_(W1_host, non_blocking=True)          # arrives while micro-batch 0 is scored
        loaded.record(side)
    got0 = score(active, slice(0, 300))
    torch.cuda.current_stream().wait_event(loaded)
    active, standby = standby, active                      # swap at the micro-batch boundary
    got1 = score(active, slice(300, 640))
    torch.cuda.synchronize()
    ctx.set_tuning(0, 0)
    assert torch.equal(got0, ref0[0]) and torch.equal(got1, ref1[1])
    assert not torch.equal(got1, ref0[1])
    lp_ref, _, _ = O.token_logprob_ref(wl.bf16_bits(H[300:]), wl.bf16_bits(W1), y[300:].numpy())
    assert np.abs(np_of(got1) - lp_ref).max() <= LOGP_TOL
    assert ctx.check_device_errors() == 0


def test_two_contexts_on_two_streams_do_not_disturb_each_other(ctx):
    """Two scoring calls of full-grid size in flight at once (two contexts, two streams): the
    CTAs of the second cannot all be resident while the first runs, which is the situation the
    pacing of the CTA pairs has to give way in.  Results equal those of the calls made one
    after the other, bit for bit."""
    from paper_2507_01663_b200 import binding as B
    dev = device()
    other = B.Context(0)
    try:
        cases = [random_case(19000, 256, 4104, seed=31), random_case(18000, 320, 4104, seed=32)]
        dev_in = [(H.to(dev), W.to(dev), y.to(dev)) for H, W, y in cases]
        ctxs, streams = [ctx, other], [torch.cuda.Stream(), torch.cuda.Stream()]
        for c in ctxs:
            c.set_tuning(0, 0, VARIANT)
        ref = []
        for c, (H, W, y) in zip(ctxs, dev_in):
            out = [torch.empty(H.shape[0], device=dev) for _ in range(3)]
            c.token_logprob(H, W, y, *out)
            ref.append(out)
        torch.cuda.synchronize()
        for rep in range(3):
            got = []
            for c, s, (H, W, y) in zip(ctxs, streams, dev_in):
                out = [torch.empty(H.shape[0], device=dev) for _ in range(3)]
                with torch.cuda.stream(s):
                    c.token_logprob(H, W, y, *out, stream=s)
                got.append(out)
            torch.cuda.synchronize()
            for g, r in zip(got, ref):
                assert all(torch.equal(a, b) for a, b in zip(g, r))
        assert ctx.check_device_errors() == 0 and other.check_device_errors() == 0
    finally:
        ctx.set_tuning(0, 0)
        other.close()


def test_reserved_workspace_does_not_grow(ctx):
    """After af_reserve for the largest batch, scoring calls of that size and smaller ones (which
    pick other numbers of vocabulary ranges) allocate nothing more."""
    dev = device()
    T, d, V = 6000, 128, 8200
    ctx.set_tuning(0, 0, VARIANT)
    ctx.reserve(T, 64, d, V)
    held = ctx.workspace_bytes()
    H, W, y = random_case(T, d, V, seed=41)
    Hd, Wd, yd = H.to(dev), W.to(dev), y.to(dev)
    out = torch.empty(T, device=dev)
    for t in (T, T // 2, 700, 129, 1):
        ctx.token_logprob(Hd, Wd, yd, out, T=t)
    torch.cuda.synchronize()
    ctx.set_tuning(0, 0)
    assert ctx.workspace_bytes() == held
    assert ctx.check_device_errors() == 0


@pytest.mark.parametrize("cuts", [[0, 8200], [0, 3000, 8200], [0, 1, 257, 4100, 8199, 8200]])
def test_vocabulary_shards_merge_to_the_full_result(ctx, cuts):
    """The head split by vocabulary rows: every shard's statistics against the oracle's, and the
    merged result against the full-vocabulary oracle and the unsharded call."""
    dev = device()
    w = wl.make_workload("cfg2_mini")                       # V = 8200, not a multiple of the tile
    H, W, y = wl.gen_hidden(w), wl.gen_weight(w), wl.gen_target(w)
    T = H.shape[0]
    Hd, Wd, yd = H.to(dev), W.to(dev), y.to(dev)
    ctx.set_tuning(0, 0, VARIANT)
    R = len(cuts) - 1
    partials = torch.full((R, T, 4), 9.0, device=dev)
    for r, (a, b) in enumerate(zip(cuts[:-1], cuts[1:])):
        ctx.token_logprob_shard(Hd, Wd[a:b].contiguous(), yd, a, partials[r])
        ref = O.token_logprob_shard_ref(wl.bf16_bits(H), wl.bf16_bits(W[a:b]), y.numpy(), a)
        got = np_of(partials[r]).astype(np.float64)
        assert np.abs(got[:, 0] - ref[:, 0]).max() <= LOGP_TOL                                   # max logit
        assert np.abs(np.log(got[:, 1]) - np.log(ref[:, 1])).max() <= LOGP_TOL                   # shard normaliser
        assert np.abs(got[:, 2] / got[:, 1] - ref[:, 2] / ref[:, 1]).max() <= LOGP_TOL          # mean logit
        inside = np.isfinite(ref[:, 3])
        assert np.array_equal(np.isfinite(got[:, 3]), inside)
        assert np.abs(got[inside, 3] - ref[inside, 3]).max(initial=0.0) <= LOGP_TOL
        assert np.all(got[~inside, 3] == -np.inf)
    logp, ent, lse = (torch.empty(T, device=dev) for _ in range(3))
    ctx.merge_logprob_shards(partials, yd, w.V, logp, ent, lse)
    full = [torch.empty(T, device=dev) for _ in range(3)]
    ctx.token_logprob(Hd, Wd, yd, *full)
    flags = ctx.check_device_errors()
    ctx.set_tuning(0, 0)
    assert flags == 0
    r_logp, r_ent, r_lse = O.token_logprob_ref(wl.bf16_bits(H), wl.bf16_bits(W), y.numpy())
    for got, ref, one in ((logp, r_logp, full[0]), (ent, r_ent, full[1]), (lse, r_lse, full[2])):
        assert np.abs(np_of(got) - ref).max() <= LOGP_TOL
        assert np.abs(np_of(got) - np_of(one)).max() <= 1e-4
    # the merge of the oracle's own shard statistics, fed through the device merge
    o_parts = np.stack([O.token_logprob_shard_ref(wl.bf16_bits(H), wl.bf16_bits(W[a:b]), y.numpy(), a)
                        for a, b in zip(cuts[:-1], cuts[1:])]).astype(np.float32)
    ctx.merge_logprob_shards(torch.as_tensor(o_parts, device=dev), yd, w.V, logp, ent, lse)
    assert np.abs(np_of(logp) - r_logp).max() <= 1e-4 and np.abs(np_of(ent) - r_ent).max() <= 1e-4


def test_shard_argument_errors(ctx):
    from paper_2507_01663_b200 import binding as B
    dev = device()
    H = torch.zeros(4, 16, dtype=torch.bfloat16, device=dev)
    W = torch.zeros(8, 16, dtype=torch.bfloat16, device=dev)
    y = torch.zeros(4, dtype=torch.int32, device=dev)
    part = torch.zeros(1, 4, 4, device=dev)
    with pytest.raises(B.AfError):
        ctx.token_logprob_shard(H, W, y, -1, part[0])
    with pytest.raises(B.AfError):
        ctx.token_logprob_shard(H, W, y, 0, None)
    with pytest.raises(B.AfError):
        ctx.merge_logprob_shards(part, y, 0, torch.zeros(4, device=dev))
    ctx.merge_logprob_shards(part, y, 8, torch.zeros(4, device=dev), T=0)      # empty batch is a no-op
    y[1] = 99                                                                  # a global id outside [0, V_total)
    ctx.token_logprob_shard(H, W, y, 0, part[0])
    out = torch.zeros(4, device=dev)
    ctx.merge_logprob_shards(part, y, 8, out)
    assert ctx.check_device_errors() == B.DEVERR_TARGET_RANGE
    assert torch.isnan(out[1]) and not torch.isnan(out[0])


def test_die_aware_dealing_of_row_tiles(ctx):
    """gemm_variant 3: the pairs claim ranks by the SM they run on and each half of the chip shares its
    own row tiles.  Every unit must still be processed exactly once: all rows against the oracle,
    at sizes with several units per pair (the mode switches itself off below that), on ragged shapes."""
    for T, d, V, splits in [(40000, 64, 1024, 0), (50001, 72, 1500, 2), (38400, 128, 520, 0)]:
        H, W, y = random_case(T, d, V, seed=T)
        dev = device()
        logp, ent, lse = (torch.full((T,), 9.0, device=dev) for _ in range(3))
        ctx.set_tuning(splits, 0, 3)
        ctx.token_logprob(H.to(dev), W.to(dev), y.to(dev), logp, ent, lse)
        again = torch.full((T,), 9.0, device=dev)
        ctx.token_logprob(H.to(dev), W.to(dev), y.to(dev), again)
        flags = ctx.check_device_errors()
        ctx.set_tuning(0, 0)
        assert flags == 0
        want = O.token_logprob_ref(wl.bf16_bits(H), wl.bf16_bits(W), y.numpy())
        for got, ref in zip((logp, ent, lse), want):
            assert np.abs(np_of(got) - ref).max() <= LOGP_TOL
        assert torch.equal(again, logp)              # the claimed ranks may differ between launches, the bits may not


def test_the_plan_is_what_the_call_does(ctx):
    """af_plan_token_logprob, fed with this part's SM count and measured die split, names the number
    of vocabulary ranges the call itself picks: asking for exactly that number gives the same bits
    (the ranges' partial statistics are merged in range order, so another number gives others),
    and the workspace holds one partial per range and token."""
    from paper_2507_01663_b200 import binding as B
    dev = device()
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    die0 = max(ctx.die_split()[0], 0)
    for T, d, V in [(40000, 64, 4096), (9000, 512, 8200)]:
        H, W, y = random_case(T, d, V, seed=T + 1)
        Hd, Wd, yd = H.to(dev), W.to(dev), y.to(dev)
        plan = B.plan_token_logprob(T, d, V, sms, die0)
        own, asked, other = (torch.empty(T, device=dev) for _ in range(3))
        ctx.token_logprob(Hd, Wd, yd, own)
        ctx.set_tuning(plan.v_splits, 0)
        ctx.token_logprob(Hd, Wd, yd, asked)
        ctx.set_tuning(plan.v_splits + 1, 0)
        ctx.token_logprob(Hd, Wd, yd, other)
        ctx.set_tuning(0, 0)
        assert ctx.check_device_errors() == 0
        assert torch.equal(own, asked)
        assert not torch.equal(own, other)
        assert (other - own).abs().max().item() <= LOGP_TOL


def test_die_split_measured_at_creation(ctx):
    """The latency probe behind die-aware dealing: either a clean split of the SMs into two dies (even
    counts that add up to the SM count, neither die tiny) or a stated reason for having none."""
    a, b = ctx.die_split()
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    if a > 0:
        assert a + b == sms and a % 2 == 0 and b % 2 == 0 and min(a, b) >= sms // 4
    else:
        assert a == 0 and -5 <= b <= -1


def test_a_wait_that_nothing_satisfies_ends_by_itself(ctx):
    """Failure detection on the device: the bounded wait every kernel uses gives up after its limit
    (one millisecond here), raises the watchdog flag and returns; the context then works as before."""
    from paper_2507_01663_b200 import binding as B
    assert ctx.check_device_errors() == 0
    waited = ctx.selftest_bounded_wait()
    assert 900 <= waited <= 50000                    # the limit, plus at most a scheduling hiccup
    assert ctx.check_device_errors() == B.DEVERR_WATCHDOG
    assert ctx.check_device_errors() == 0            # read clears it
    check(ctx, *random_case(300, 64, 520, seed=3))   # and scoring still matches the oracle
