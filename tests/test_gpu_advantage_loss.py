"""af_grpo_advantage and af_policy_loss against the oracle."""
import numpy as np
import pytest
import torch

from oracle import grpo_oracle as O
from paper_2507_01663_b200 import workloads as wl
from gpu_util import ADV_TOL, LOSS_RTOL, device, f32, i32, np_of, rel

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2507_01663_b200 import binding as B
    c = B.Context(0)
    yield c
    c.close()


# ---------------------------------------------------------------- advantage
@pytest.mark.parametrize("name", ["cfg1", "cfg2", "cfg3", "cfg4", "cfg5"])
@pytest.mark.parametrize("ddof", [0, 1])
def test_advantage_workload_rewards(ctx, name, ddof):
    w = wl.make_workload(name)
    dev = device()
    r = wl.gen_reward(w, dev)
    ref = O.grpo_advantage_ref(np_of(r), w.group_id, w.n_prompts, 1e-6, ddof)
    adv = torch.full((w.N,), 9.0, device=dev)
    ctx.grpo_advantage(r, None, w.n_prompts, adv, 1e-6, ddof)                 # contiguous groups
    assert np.abs(np_of(adv) - ref).max() <= ADV_TOL
    adv2 = torch.full((w.N,), 9.0, device=dev)
    ctx.grpo_advantage(r, i32(w.group_id), w.n_prompts, adv2, 1e-6, ddof)     # explicit ids
    assert np.abs(np_of(adv2) - ref).max() <= ADV_TOL
    # ids in arbitrary order
    perm = wl.arrival_order(w)
    adv3 = torch.full((w.N,), 9.0, device=dev)
    ctx.grpo_advantage(r[torch.as_tensor(perm.astype(np.int64), device=dev)].contiguous(),
                       i32(w.group_id[perm]), w.n_prompts, adv3, 1e-6, ddof)
    assert np.abs(np_of(adv3) - ref[perm]).max() <= ADV_TOL
    assert ctx.check_device_errors() == 0


@pytest.mark.parametrize("G", [1, 2, 3, 4, 5, 6, 7, 8, 9, 10, 11, 12, 13, 14, 15, 16, 17, 24, 31, 32, 33, 48, 64, 100, 128, 256, 300, 511, 512, 513, 1000, 1024, 5000])
def test_advantage_group_sizes(ctx, G):
    # a handful of groups (a ragged run only) and a few thousand (full runs of every kernel plus a tail)
    for n_groups in ((37, 4099) if G < 1000 else (3,)):
        N = G * n_groups
        r = wl.uniform01(G, wl.S_REWARD, 0, N, device())
        ref = O.grpo_advantage_ref(np_of(r), np.arange(N) // G, n_groups, 1e-6, 0)
        adv = torch.full((N + 8,), 9.0, device=device())
        ctx.grpo_advantage(r, None, n_groups, adv[:N], N=N)
        assert np.abs(np_of(adv[:N]) - ref).max() <= ADV_TOL
        assert np.all(np_of(adv[N:]) == 9.0)                      # nothing written past the end


@pytest.mark.parametrize("G", [4, 8, 16, 32, 64, 128, 512, 3, 6, 7, 12, 15, 24, 200, 500])
def test_advantage_of_nearly_equal_rewards(ctx, G):
    """Rewards of a group a few units in the last place apart: the deviations (~1e-8..1e-6) are of the
    size of eps, so the mean must be right to far below an fp32 ulp for the advantages to be."""
    n_groups = 9
    base = np.float32(0.3)
    steps = np.random.default_rng(G).integers(0, 40, size=G * n_groups)
    r = base + steps.astype(np.float32) * np.spacing(base)            # exact in fp32
    assert np.all(r.astype(np.float32) == r)
    ref = O.grpo_advantage_ref(r.astype(np.float32), np.arange(G * n_groups) // G, n_groups, 1e-6, 0)
    adv = torch.full((G * n_groups,), 9.0, device=device())
    ctx.grpo_advantage(f32(r), None, n_groups, adv)
    assert np.abs(ref).max() > 0.05                                   # the case is not trivially zero
    assert np.abs(np_of(adv) - ref).max() <= ADV_TOL


def groups_ref(r, gid, groups, eps=1e-6, ddof=0):
    """The oracle on the given groups only (it visits every group in turn, which at 2^17 groups
    would take hours): each group's members form a batch of one group."""
    order = np.argsort(gid, kind="stable")
    bounds = np.searchsorted(gid[order], np.arange(gid.max() + 2))
    out = {}
    for g in groups:
        members = order[bounds[g]:bounds[g + 1]]
        out[g] = (members, O.grpo_advantage_ref(r[members], np.zeros(len(members), np.int64), 1, eps, ddof))
    return out


@pytest.mark.parametrize("law", ["uniform", "bernoulli", "last_bits", "outliers"])
def test_advantage_by_group_id_at_scale(ctx, law):
    """2^20 responses in 2^17 shuffled groups of unequal size (some empty): O(N) work, checked
    against the oracle on sampled groups, and the same bits on every run although the members of a
    group meet in no fixed order."""
    dev = device()
    N, n_groups = 1 << 20, 1 << 17
    # group sizes from 0 to a few dozen: ids drawn with a skew, then shuffled by construction
    u = np_of(wl.uniform01(41, wl.S_MISC, 0, N))
    gid = np.minimum((u ** 1.7 * n_groups).astype(np.int64), n_groups - 1)
    if law == "uniform":
        r = np_of(wl.uniform01(42, wl.S_REWARD, 0, N))
    elif law == "bernoulli":
        r = (np_of(wl.uniform01(42, wl.S_REWARD, 0, N)) < 0.3).astype(np.float32)
    elif law == "last_bits":          # rewards that differ only in the last bits of an fp32
        steps = np_of(wl.randint(42, wl.S_REWARD, 0, N, 40)).astype(np.float32)
        r = (np.float32(0.3) + steps * np.spacing(np.float32(0.3))).astype(np.float32)
    else:                             # a few huge rewards among tiny ones, both signs
        big = np_of(wl.uniform01(43, wl.S_REWARD, 0, N)) < 0.02
        r = np.where(big, 1.0e6, 1.0e-3 * np_of(wl.normal01(44, wl.S_REWARD, 0, N))).astype(np.float32)
    counts = np.bincount(gid, minlength=n_groups)
    assert counts.min() == 0 and counts.max() > 30
    for ddof in (0, 1):
        adv = torch.full((N,), 9.0, device=dev)
        ctx.grpo_advantage(f32(r), i32(gid), n_groups, adv, 1e-6, ddof)
        a = np_of(adv)
        again = torch.full((N,), 9.0, device=dev)
        ctx.grpo_advantage(f32(r), i32(gid), n_groups, again, 1e-6, ddof)
        assert a.tobytes() == np_of(again).tobytes()
        pick = sorted({int(np.argmax(counts)), int(np.argmax(counts == 1)), int(np.argmax(counts == 2)), 0, n_groups - 1}
                      | set(np.random.default_rng(5).integers(0, n_groups, 1500).tolist()))
        for g, (members, want) in groups_ref(r, gid, pick, 1e-6, ddof).items():
            assert np.abs(a[members] - want).max(initial=0.0) <= ADV_TOL, (law, ddof, g)
        assert np.isfinite(a).all()
    assert ctx.check_device_errors() == 0


def test_advantage_by_group_id_few_huge_groups_and_bad_ids(ctx):
    from paper_2507_01663_b200 import binding as B
    dev = device()
    N = 1 << 18
    r = np_of(wl.uniform01(45, wl.S_REWARD, 0, N))
    gid = np_of(wl.randint(46, wl.S_MISC, 0, N, 3)).astype(np.int64)          # three groups of ~87 k members
    adv = torch.full((N,), 9.0, device=dev)
    ctx.grpo_advantage(f32(r), i32(gid), 3, adv)
    ref = O.grpo_advantage_ref(r, gid, 3)
    assert np.abs(np_of(adv) - ref).max() <= ADV_TOL
    # one group holding everything, in one warp's worth of lanes each time
    ctx.grpo_advantage(f32(r), i32(np.zeros(N)), 1, adv)
    assert np.abs(np_of(adv) - O.grpo_advantage_ref(r, np.zeros(N, np.int64), 1)).max() <= ADV_TOL
    assert ctx.check_device_errors() == 0
    # ids outside [0, n_groups): NaN for those samples, the flag is raised, the rest is unaffected
    bad = gid.copy()
    bad[[5, 70000]] = [3, -1]
    ctx.grpo_advantage(f32(r), i32(bad), 3, adv)
    a = np_of(adv)
    assert ctx.check_device_errors() & B.DEVERR_GROUP_ID
    assert np.isnan(a[[5, 70000]]).all() and np.isnan(a).sum() == 2
    keep = np.ones(N, bool)
    keep[[5, 70000]] = False
    ref_bad = O.grpo_advantage_ref(r[keep], gid[keep], 3)
    assert np.abs(a[keep] - ref_bad).max() <= ADV_TOL


def test_advantage_degenerate_groups(ctx):
    # equal rewards inside a group (also non-dyadic values) give exactly-zero-sized advantages
    r = f32([0.3] * 8 + [1.0] * 8 + [0.0] * 8 + [0.1, 0.7, 0.1, 0.7, 0.1, 0.7, 0.1, 0.7])
    adv = torch.full((32,), 9.0, device=device())
    ctx.grpo_advantage(r, None, 4, adv)
    ref = O.grpo_advantage_ref(np_of(r), np.arange(32) // 8, 4, 1e-6, 0)
    a = np_of(adv)
    assert np.abs(a - ref).max() <= ADV_TOL and np.abs(a[:24]).max() <= ADV_TOL
    assert np.allclose(np.abs(a[24:]), 1.0, atol=1e-4)
    # many groups (bandwidth shape): still element-exact against the oracle on a sample
    N, G = 1 << 20, 8
    rr = (wl.uniform01(3, wl.S_REWARD, 0, N, device()) < 0.3).float()
    out = torch.empty(N, device=device())
    ctx.grpo_advantage(rr, None, N // G, out)
    sl = slice(1000 * G, 1200 * G)
    ref2 = O.grpo_advantage_ref(np_of(rr[sl]), np.arange(200 * G) // G, 200, 1e-6, 0)
    assert np.abs(np_of(out[sl]) - ref2).max() <= ADV_TOL
    # empty input is a no-op; N not divisible by the group count is refused
    from paper_2507_01663_b200.binding import AfError
    ctx.grpo_advantage(r, None, 4, adv, N=0)
    with pytest.raises(AfError) as e:
        ctx.grpo_advantage(r, None, 5, adv)
    assert e.value.status == -2
    # eps_adv = 0 would turn a group of equal rewards into 0 / 0: refused
    with pytest.raises(AfError) as e:
        ctx.grpo_advantage(r, None, 4, adv, eps_adv=0.0)
    assert e.value.status == -1


# ---------------------------------------------------------------- loss
def loss_inputs(w, T, lens, seed_shift=0):
    """logp around a random head's magnitude; old / ref = logp + N(0, 0.1) as in the workloads."""
    logp = wl.gen_surrogate_logp(w, T)
    old = logp + wl.gen_noise(w, wl.S_OLD, T, start=seed_shift)
    ref = logp + wl.gen_noise(w, wl.S_REF, T, start=seed_shift)
    ent = torch.abs(wl.normal01(w.seed, wl.S_MISC, 0, T)) + 5.0
    return logp, old, ref, ent


def run_loss(ctx, logp, old, ref, ent, adv_seq, cu, **kw):
    from paper_2507_01663_b200 import binding as B
    dev = device()
    T = logp.shape[0]
    out = B.new_loss_out(dev)
    g = torch.full((max(T, 1),), 9.0, device=dev)
    ctx.policy_loss(logp.to(dev), old.to(dev), ref.to(dev), f32(adv_seq), i32(cu), out, g,
                    None if ent is None else ent.to(dev), T=T, **kw)
    res = B.read_loss_out(out)
    return res, np_of(g)[:T]


def compare_loss(res, g, ref, T, clip_lo=0.2, clip_hi=0.2):
    for k in ("loss", "pg_loss", "kl_mean", "entropy_mean"):
        assert rel(res[k], ref[k]) <= LOSS_RTOL or abs(res[k] - ref[k]) < 1e-9, (k, res[k], ref[k])
    assert res["n_tokens"] == T
    # tokens whose ratio sits on a clip bound to within fp32 rounding may fall on either side
    rho = ref["rho"]
    near = (np.abs(rho - (1 - clip_lo)) < 1e-5) | (np.abs(rho - (1 + clip_hi)) < 1e-5)
    assert abs(res["clip_frac"] - ref["clip_frac"]) <= (near.sum() + 0.5) / max(T, 1) + 1e-7
    ok = ~near
    scale = np.abs(ref["dlogp"]).max() if T else 1.0
    assert np.abs(g[ok] - ref["dlogp"][ok]).max(initial=0.0) <= 1e-5 * scale + 1e-12


@pytest.mark.parametrize("name", ["cfg1", "cfg2_mini", "cfg3_mini", "cfg5_mini"])
@pytest.mark.parametrize("agg_mode", [0, 1])
def test_loss_on_workload_batches(ctx, name, agg_mode):
    w = wl.make_workload(name)
    r = np_of(wl.gen_reward(w))
    adv = O.grpo_advantage_ref(r, w.group_id, w.n_prompts)
    for mb in wl.microbatches(w)[:4]:
        lens = w.lengths[mb]
        cu = np.concatenate([[0], np.cumsum(lens)])
        T = int(cu[-1])
        logp, old, ref, ent = loss_inputs(w, T, lens)
        kw = dict(clip_lo=w.clip_eps, clip_hi=w.clip_eps, kl_coef=w.kl_coef, agg_mode=agg_mode, loss_scale=1.0)
        res, g = run_loss(ctx, logp, old, ref, ent, adv[mb], cu, **kw)
        oref = O.policy_loss_ref(logp.numpy(), old.numpy(), ref.numpy(), adv[mb].astype(np.float32), cu,
                                 entropy=ent.numpy(), **kw)
        compare_loss(res, g, oref, T)
        assert 0.0 < oref["clip_frac"] < 0.9 or name == "cfg1"
    assert ctx.check_device_errors() == 0


@pytest.mark.parametrize("lens", [[1], [4], [1, 1, 1], [1023, 1, 1024, 2, 1025], [5, 0, 7, 0, 0, 3], [4097], [3] * 700])
def test_loss_ragged_and_tiny_sequences(ctx, lens):
    w = wl.make_workload("cfg1")
    cu = np.concatenate([[0], np.cumsum(lens)])
    T = int(cu[-1])
    logp, old, ref, ent = loss_inputs(w, T, lens, seed_shift=17)
    A = np_of(wl.normal01(5, wl.S_MISC, 0, len(lens)))
    for agg_mode in (0, 1):
        kw = dict(clip_lo=0.2, clip_hi=0.28, kl_coef=0.04, agg_mode=agg_mode, loss_scale=0.5)
        res, g = run_loss(ctx, logp, old, ref, None, A, cu, **kw)
        oref = O.policy_loss_ref(logp.numpy(), old.numpy(), ref.numpy(), A, cu, **kw)
        compare_loss(res, g, oref, T, 0.2, 0.28)
        assert res["entropy_mean"] == 0.0


def test_loss_identities_on_device(ctx):
    w = wl.make_workload("cfg2_mini")
    lens = w.lengths[:16]
    cu = np.concatenate([[0], np.cumsum(lens)])
    T = int(cu[-1])
    logp, old, ref, ent = loss_inputs(w, T, lens)
    A = np_of(wl.normal01(6, wl.S_MISC, 0, 16))
    # old == current: ratio 1, nothing clipped, pg loss = -mean advantage; ref == current: no KL
    res, g = run_loss(ctx, logp, logp, logp, ent, A, cu, kl_coef=0.04)
    assert res["clip_frac"] == 0.0 and res["kl_mean"] == 0.0
    assert rel(res["pg_loss"], -float(np.mean(A.astype(np.float64)))) <= 1e-5
    # empty batch
    res0, _ = run_loss(ctx, logp[:0], old[:0], ref[:0], None, A[:0], [0])
    assert res0["loss"] == 0.0 and res0["n_tokens"] == 0
    # run-to-run bitwise reproducibility
    r1, g1 = run_loss(ctx, logp, old, ref, ent, A, cu)
    r2, g2 = run_loss(ctx, logp, old, ref, ent, A, cu)
    assert r1 == r2 and g1.tobytes() == g2.tobytes()


def test_loss_bad_cu_seqlens_is_flagged(ctx):
    from paper_2507_01663_b200 import binding as B
    w = wl.make_workload("cfg1")
    logp, old, ref, ent = loss_inputs(w, 64, [64])
    run_loss(ctx, logp, old, ref, None, [1.0, 1.0], [0, 32, 60])      # cu[B] != T
    assert ctx.check_device_errors() & B.DEVERR_CU_SEQLENS
    assert ctx.check_device_errors() == 0
    run_loss(ctx, logp, old, ref, None, [1.0, 1.0], [4, 32, 64])      # cu[0] != 0
    assert ctx.check_device_errors() & B.DEVERR_CU_SEQLENS
    run_loss(ctx, logp, old, ref, None, [1.0, 1.0, 1.0], [0, 40, 32, 64])   # decreasing in the middle, ends right
    assert ctx.check_device_errors() & B.DEVERR_CU_SEQLENS
    res, _ = run_loss(ctx, logp, old, ref, None, [1.0, 1.0, 1.0], [0, 32, 32, 64])  # an empty sequence is fine
    assert ctx.check_device_errors() == 0 and res["n_tokens"] == 64


def test_kl_term_close_to_the_reference_policy(ctx):
    """Late in training the policy sits close to the reference: delta = ref - logp ~ N(0, 0.01), k3 ~
    5e-5 per token.  kl_mean and the KL part of the gradient must still meet the loss tolerance."""
    w = wl.make_workload("cfg2_mini")
    lens = w.lengths[:24]
    cu = np.concatenate([[0], np.cumsum(lens)])
    T = int(cu[-1])
    logp, old, _, ent = loss_inputs(w, T, lens)
    A = np_of(wl.normal01(8, wl.S_MISC, 0, 24))
    for std in (1e-2, 1e-3, 0.3):
        ref = logp + std * wl.normal01(w.seed, wl.S_REF, 0, T)
        for agg_mode in (0, 1):
            kw = dict(clip_lo=0.2, clip_hi=0.2, kl_coef=0.04, agg_mode=agg_mode, loss_scale=1.0)
            res, g = run_loss(ctx, logp, old, ref, ent, A, cu, **kw)
            oref = O.policy_loss_ref(logp.numpy(), old.numpy(), ref.numpy(), A, cu, entropy=ent.numpy(), **kw)
            assert rel(res["kl_mean"], oref["kl_mean"]) <= LOSS_RTOL, (std, res["kl_mean"], oref["kl_mean"])
            compare_loss(res, g, oref, T)
            # the KL part of dL/dlogp alone (advantages of zero leave nothing else): exp(delta) - 1 carries
            # the approximate exp2's 2.4e-7 absolute error, a few 1e-4 of its size at delta ~ 1e-3
            res0, g0 = run_loss(ctx, logp, old, ref, ent, np.zeros(24, np.float32), cu, **kw)
            o0 = O.policy_loss_ref(logp.numpy(), old.numpy(), ref.numpy(), np.zeros(24), cu, entropy=ent.numpy(), **kw)
            assert np.abs(g0 - o0["dlogp"]).max() <= 1e-3 * np.abs(o0["dlogp"]).max()
    assert ctx.check_device_errors() == 0
