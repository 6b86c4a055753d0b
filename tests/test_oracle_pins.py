"""Pins for the CPU oracle: what mathematics fixes independently of the oracle's own code.

Each test is chosen so that a plausible slip (a dropped term, a wrong sign or index, a
transposed operand, a wrong divisor) fails at least one of them.
"""
import math
import os

import numpy as np
import pytest
import torch

from oracle import grpo_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def to_bits(x):
    """float array -> bf16 bit patterns (round to nearest even through torch)."""
    t = torch.as_tensor(np.asarray(x, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16)


def bits_val(b):
    return O.bf16_bits_to_f64(b)


# ---------------------------------------------------------------- bf16 widening
def test_bf16_widening_exact():
    vals = np.array([0.0, -0.0, 1.0, -2.5, 0.0078125, 3.0e38, 1e-30], dtype=np.float32)
    bits = to_bits(vals)
    back = O.bf16_bits_to_f64(bits)
    ref = torch.as_tensor(vals).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(back, ref)
    assert np.signbit(back[1])
    # the four patterns that decode by hand: sign|exp|mantissa
    assert O.bf16_bits_to_f64(np.array([0x3F80, 0xC000, 0x3FC0, 0x0000], np.uint16)).tolist() == [1.0, -2.0, 1.5, 0.0]


# ---------------------------------------------------------------- O1 pack
def _store(rng, N=9, d=6):
    lengths = rng.integers(1, 7, size=N)
    off = np.zeros(N + 1, np.int64)
    off[1:] = np.cumsum(lengths)
    tot = int(off[-1])
    cols = {
        "hidden": rng.integers(0, 65536, size=(tot, d)).astype(np.uint16),
        "target": rng.integers(0, 1000, size=tot).astype(np.int32),
        "old_logp": rng.standard_normal(tot).astype(np.float32),
    }
    adv = rng.standard_normal(N).astype(np.float32)
    return off, cols, adv


def test_pack_identity_and_roundtrip():
    rng = np.random.default_rng(0)
    off, cols, adv = _store(rng)
    N = off.shape[0] - 1
    ident = O.pack_microbatch_ref(off, np.arange(N), cols, adv)
    assert ident["cu_seqlens"][0] == 0
    assert np.array_equal(ident["cu_seqlens"].astype(np.int64), off)
    for k in cols:
        assert ident[k].tobytes() == cols[k].tobytes()
    assert np.array_equal(ident["adv_seq"], adv)
    # permutation, then the inverse permutation applied to the packed result, restores the store
    perm = rng.permutation(N)
    p = O.pack_microbatch_ref(off, perm, cols, adv)
    cu = p["cu_seqlens"].astype(np.int64)
    assert np.all(np.diff(cu) == (off[1:] - off[:-1])[perm])
    assert cu[-1] == off[-1]
    inv = np.argsort(perm)
    back = O.pack_microbatch_ref(cu, inv, {k: p[k] for k in cols}, p["adv_seq"])
    for k in cols:
        assert back[k].tobytes() == cols[k].tobytes()
    assert np.array_equal(back["adv_seq"], adv)


def test_pack_subset_duplicates_and_seq_id():
    rng = np.random.default_rng(1)
    off, cols, adv = _store(rng)
    idx = np.array([4, 4, 0, 7])
    p = O.pack_microbatch_ref(off, idx, cols, adv)
    cu = p["cu_seqlens"]
    L4 = off[5] - off[4]
    assert cu[1] - cu[0] == L4 and cu[2] - cu[1] == L4
    assert np.array_equal(p["target"][cu[0]:cu[1]], p["target"][cu[1]:cu[2]])
    assert np.array_equal(p["target"][cu[2]:cu[3]], cols["target"][off[0]:off[1]])
    assert np.array_equal(p["hidden"][cu[3]:cu[4]], cols["hidden"][off[7]:off[8]])
    # seq_id is constant on each segment and equals the list position
    for j in range(4):
        assert np.all(p["seq_id"][cu[j]:cu[j + 1]] == j)
    assert np.array_equal(p["adv_seq"], adv[idx])
    # element-by-element definition on one token
    t = cu[3] + 1 if cu[4] - cu[3] > 1 else cu[3]
    assert p["old_logp"][t] == cols["old_logp"][off[7] + (t - cu[3])]


def test_pack_empty():
    off, cols, adv = _store(np.random.default_rng(2))
    p = O.pack_microbatch_ref(off, np.zeros(0, np.int64), cols, adv)
    assert p["cu_seqlens"].tolist() == [0] and p["hidden"].shape[0] == 0


def test_unpack_is_the_inverse_of_pack():
    rng = np.random.default_rng(21)
    off, cols, adv = _store(rng, N=11)
    N = off.shape[0] - 1
    idx = rng.permutation(N)[:7]
    p = O.pack_microbatch_ref(off, idx, cols, adv)
    # results in packed order, written back: the listed samples' rows take them, the rest stay
    res = {"old_logp": rng.standard_normal(p["old_logp"].shape[0]).astype(np.float32),
           "target": rng.integers(0, 1000, size=p["target"].shape[0]).astype(np.int32)}
    store = {"old_logp": cols["old_logp"].copy(), "target": cols["target"].copy()}
    T = O.unpack_microbatch_ref(off, idx, res, store)
    assert T == p["cu_seqlens"][-1]
    # (a) gathering the written columns again returns the results bit for bit
    again = O.pack_microbatch_ref(off, idx, store)
    assert again["old_logp"].tobytes() == res["old_logp"].tobytes()
    assert again["target"].tobytes() == res["target"].tobytes()
    # (b) rows of samples outside the list are untouched
    others = np.setdiff1d(np.arange(N), idx)
    for i in others:
        assert np.array_equal(store["old_logp"][off[i]:off[i + 1]], cols["old_logp"][off[i]:off[i + 1]])
        assert np.array_equal(store["target"][off[i]:off[i + 1]], cols["target"][off[i]:off[i + 1]])
    # (c) the scatter written as one fancy-index assignment through the gather's own row map
    rows = O.pack_microbatch_ref(off, idx, {"row": np.arange(off[-1])})["row"]
    direct = cols["old_logp"].copy()
    direct[rows] = res["old_logp"]
    assert direct.tobytes() == store["old_logp"].tobytes()
    # (d) writing back what was gathered changes nothing
    same = {"old_logp": cols["old_logp"].copy()}
    O.unpack_microbatch_ref(off, idx, {"old_logp": p["old_logp"]}, same)
    assert same["old_logp"].tobytes() == cols["old_logp"].tobytes()


def test_unpack_empty_list_and_duplicates():
    off, cols, _ = _store(np.random.default_rng(22))
    store = {"old_logp": cols["old_logp"].copy()}
    assert O.unpack_microbatch_ref(off, np.zeros(0, np.int64), {"old_logp": np.zeros(0, np.float32)}, store) == 0
    assert store["old_logp"].tobytes() == cols["old_logp"].tobytes()
    with pytest.raises(ValueError):
        O.unpack_microbatch_ref(off, np.array([2, 5, 2]), {"old_logp": np.zeros(64, np.float32)}, store)


# ---------------------------------------------------------------- O2 log-prob / entropy
def _rand_hw(rng, T, d, V, hs=1.0, ws=0.3):
    return to_bits(rng.standard_normal((T, d)) * hs), to_bits(rng.standard_normal((V, d)) * ws)


def test_logprob_rows_sum_to_one():
    rng = np.random.default_rng(3)
    Hb, Wb = _rand_hw(rng, 12, 24, 301)
    y = rng.integers(0, 301, 12)
    logp, ent, lse, rows = O.token_logprob_ref(Hb, Wb, y, return_rows=True)
    assert np.allclose(np.exp(rows).sum(1), 1.0, rtol=0, atol=1e-12)
    assert np.array_equal(logp, rows[np.arange(12), y])
    assert np.all(logp <= 0) and np.all(ent >= 0) and np.all(ent <= math.log(301) + 1e-12)


@pytest.mark.parametrize("V", [2, 3, 5, 16])
def test_logprob_bruteforce_tiny_vocab(V):
    """Enumerate the vocabulary with Python floats, no max-shift, no matrix product."""
    rng = np.random.default_rng(10 + V)
    T, d = 5, 4
    Hb, Wb = _rand_hw(rng, T, d, V, ws=0.7)
    y = rng.integers(0, V, T)
    logp, ent, lse = O.token_logprob_ref(Hb, Wb, y)
    H, W = bits_val(Hb), bits_val(Wb)
    for t in range(T):
        z = [sum(float(H[t, k]) * float(W[v, k]) for k in range(d)) for v in range(V)]
        Zs = sum(math.exp(zv) for zv in z)
        p = [math.exp(zv) / Zs for zv in z]
        assert abs(logp[t] - math.log(p[int(y[t])])) < 1e-12
        assert abs(ent[t] - (-sum(pv * math.log(pv) for pv in p))) < 1e-12
        assert abs(lse[t] - math.log(Zs)) < 1e-12


def test_logprob_closed_forms():
    rng = np.random.default_rng(4)
    T, d, V = 6, 8, 37
    Hb, _ = _rand_hw(rng, T, d, V)
    y = rng.integers(0, V, T)
    # zero weights: uniform distribution
    logp, ent, lse = O.token_logprob_ref(Hb, np.zeros((V, d), np.uint16), y)
    assert np.allclose(logp, -math.log(V), atol=1e-14) and np.allclose(ent, math.log(V), atol=1e-13)
    assert np.allclose(lse, math.log(V), atol=1e-14)
    # V = 2: logistic closed form and binary entropy
    Hb2, Wb2 = _rand_hw(rng, T, d, 2, ws=0.5)
    y2 = rng.integers(0, 2, T)
    logp, ent, _ = O.token_logprob_ref(Hb2, Wb2, y2)
    z = bits_val(Hb2) @ bits_val(Wb2).T
    zy, zo = z[np.arange(T), y2], z[np.arange(T), 1 - y2]
    assert np.allclose(logp, -np.log1p(np.exp(zo - zy)), atol=1e-13)
    q = 1.0 / (1.0 + np.exp(zo - zy))
    assert np.allclose(ent, -(q * np.log(q) + (1 - q) * np.log1p(-q)), atol=1e-13)
    # one dominant logit: logp -> 0, entropy -> 0
    Hd = to_bits(np.ones((1, 4)) * 8.0)
    Wd = to_bits(np.vstack([np.ones((1, 4)) * 8.0, np.zeros((9, 4))]))
    logp, ent, _ = O.token_logprob_ref(Hd, Wd, np.array([0]))
    assert abs(logp[0]) < 1e-12
    assert 0 <= ent[0] < 1e-12


def test_logprob_invariances():
    rng = np.random.default_rng(5)
    T, d, V = 7, 16, 50
    Hb, Wb = _rand_hw(rng, T, d, V)
    y = rng.integers(0, V, T)
    base = O.token_logprob_ref(Hb, Wb, y)
    # a constant extra feature adds the same c to every logit of a row: nothing but lse moves
    Hc = np.concatenate([Hb, to_bits(np.full((T, 1), 2.0))], 1)
    Wc = np.concatenate([Wb, to_bits(np.full((V, 1), 1.5))], 1)
    sh = O.token_logprob_ref(Hc, Wc, y)
    assert np.allclose(sh[0], base[0], atol=1e-12) and np.allclose(sh[1], base[1], atol=1e-12)
    assert np.allclose(sh[2], base[2] + 3.0, atol=1e-12)
    # permuting the vocabulary (and the targets with it) changes nothing
    perm = rng.permutation(V)
    inv = np.argsort(perm)
    pm = O.token_logprob_ref(Hb, Wb[perm], inv[y])
    for a, b in zip(pm, base):
        assert np.allclose(a, b, atol=1e-12)
    # H and W are not interchangeable: a transposed operand would not even have this shape,
    # and each row depends only on its own hidden state
    one = O.token_logprob_ref(Hb[3:4], Wb, y[3:4])
    assert np.allclose(one[0], base[0][3], atol=1e-13)


def test_logprob_against_torch_float64():
    rng = np.random.default_rng(6)
    T, d, V = 9, 32, 200
    Hb, Wb = _rand_hw(rng, T, d, V)
    y = rng.integers(0, V, T)
    logp, ent, lse = O.token_logprob_ref(Hb, Wb, y)
    z = torch.from_numpy(bits_val(Hb)) @ torch.from_numpy(bits_val(Wb)).T
    ls = torch.log_softmax(z, dim=1)
    assert np.allclose(logp, ls[torch.arange(T), torch.from_numpy(y)].numpy(), atol=1e-12)
    assert np.allclose(ent, torch.distributions.Categorical(logits=z).entropy().numpy(), atol=1e-12)
    assert np.allclose(lse, torch.logsumexp(z, 1).numpy(), atol=1e-12)


# ---------------------------------------------------------------- O3 advantage
def _golden_rows(name):
    rows = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append([float(x) for x in line.split()])
    return rows


def test_advantage_bernoulli_golden():
    for G, k, a1, a0 in _golden_rows("grpo_bernoulli_groups.txt"):
        G, k = int(G), int(k)
        r = np.array([1.0] * k + [0.0] * (G - k))
        adv = O.grpo_advantage_ref(r, np.zeros(G, int), 1, eps_adv=0.0, ddof=0)
        assert np.allclose(adv[:k], a1, atol=1e-13) and np.allclose(adv[k:], a0, atol=1e-13)


def test_advantage_moments_and_invariances():
    rng = np.random.default_rng(7)
    n_groups, G, eps = 5, 8, 1e-6
    r = rng.random(n_groups * G)
    gid = np.repeat(np.arange(n_groups), G)
    for ddof in (0, 1):
        adv = O.grpo_advantage_ref(r, gid, n_groups, eps, ddof)
        for g in range(n_groups):
            a, rr = adv[gid == g], r[gid == g]
            sigma = rr.std(ddof=ddof)
            assert abs(a.mean()) < 1e-12
            assert abs(a.std(ddof=ddof) - sigma / (sigma + eps)) < 1e-12
    base = O.grpo_advantage_ref(r, gid, n_groups, 0.0, 0)
    assert np.allclose(O.grpo_advantage_ref(3.5 * r - 2.0, gid, n_groups, 0.0, 0), base, atol=1e-12)
    # sign: a larger reward gets a larger advantage
    g0 = np.nonzero(gid == 0)[0]
    assert np.array_equal(np.argsort(base[g0]), np.argsort(r[g0]))
    # membership given in any order
    perm = rng.permutation(r.size)
    shuffled = O.grpo_advantage_ref(r[perm], gid[perm], n_groups, 0.0, 0)
    assert np.allclose(shuffled, base[perm], atol=1e-14)


def test_advantage_special_cases():
    # two distinct rewards: +-1 (population) and +-1/sqrt 2 (sample)
    a0 = O.grpo_advantage_ref([0.2, 0.9], [0, 0], 1, 0.0, 0)
    a1 = O.grpo_advantage_ref([0.2, 0.9], [0, 0], 1, 0.0, 1)
    assert np.allclose(a0, [-1, 1], atol=1e-14) and np.allclose(a1, [-1 / math.sqrt(2), 1 / math.sqrt(2)], atol=1e-14)
    # a group with equal rewards has zero advantage (0 / (0 + eps)), never NaN
    z = O.grpo_advantage_ref([1, 1, 1, 0, 1], [0, 0, 0, 1, 1], 2, 1e-6, 0)
    assert np.all(z[:3] == 0) and np.all(np.isfinite(z))
    # eps sits outside the root: A = dev / (sigma + eps)
    a = O.grpo_advantage_ref([0.0, 2.0], [0, 0], 1, 0.5, 0)
    assert np.allclose(a, [-1 / 1.5, 1 / 1.5], atol=1e-14)
    # a singleton group with ddof = 1 must not divide by zero
    s = O.grpo_advantage_ref([3.0], [0], 1, 1e-6, 1)
    assert s[0] == 0.0


# ---------------------------------------------------------------- O4 loss
def _loss_inputs(rng, lens):
    cu = np.concatenate([[0], np.cumsum(lens)])
    T = int(cu[-1])
    logp = -np.abs(rng.standard_normal(T)) - 0.1
    old = logp + 0.3 * rng.standard_normal(T)
    ref = logp + 0.3 * rng.standard_normal(T)
    A = rng.standard_normal(len(lens))
    return logp, old, ref, A, cu


def test_loss_golden_quadrants():
    for A, rho, pg, clipped, grad in _golden_rows("ppo_clip_quadrants.txt"):
        logp = np.array([-1.0])
        old = logp - math.log(rho)
        out = O.policy_loss_ref(logp, old, logp, [A], [0, 1], 0.2, 0.2, kl_coef=0.0)
        assert abs(out["pg_loss"] - pg) < 1e-12 and abs(out["loss"] - pg) < 1e-12
        assert bool(out["clipped"][0]) == bool(clipped)
        assert abs(out["dlogp"][0] - grad) < 1e-12
        assert abs(out["clip_frac"] - clipped) < 1e-15


def test_loss_on_policy_and_reference_identities():
    rng = np.random.default_rng(8)
    lens = [3, 7, 1, 5]
    logp, old, ref, A, cu = _loss_inputs(rng, lens)
    # old == current: rho = 1, nothing clipped, pg = -mean of advantages (per aggregation)
    out = O.policy_loss_ref(logp, logp, ref, A, cu, kl_coef=0.0, agg_mode=0)
    assert out["clip_frac"] == 0 and np.all(out["rho"] == 1.0)
    assert abs(out["pg_loss"] - (-A.mean())) < 1e-13
    out1 = O.policy_loss_ref(logp, logp, ref, A, cu, kl_coef=0.0, agg_mode=1)
    assert abs(out1["pg_loss"] - (-(A * lens).sum() / sum(lens))) < 1e-13
    # ref == current: k3 = 0 and carries no gradient
    o2 = O.policy_loss_ref(logp, old, logp, A, cu, kl_coef=0.7)
    assert o2["kl_mean"] == 0 and abs(o2["loss"] - o2["pg_loss"]) < 1e-15
    # k3 >= 0, and ~ delta^2 / 2 for small delta
    o3 = O.policy_loss_ref(logp, old, ref, A, cu, kl_coef=1.0)
    assert o3["kl_mean"] >= 0
    small = O.policy_loss_ref(logp, old, logp + 1e-4, A, cu, kl_coef=1.0, agg_mode=1)
    assert abs(small["kl_mean"] - 0.5e-8) < 1e-11
    # loss = pg + coef * kl, and loss_scale is a plain factor
    assert abs(o3["loss"] - (o3["pg_loss"] + 1.0 * o3["kl_mean"])) < 1e-13
    o4 = O.policy_loss_ref(logp, old, ref, A, cu, kl_coef=1.0, loss_scale=0.25)
    assert abs(o4["loss"] - 0.25 * o3["loss"]) < 1e-14 and np.allclose(o4["dlogp"], 0.25 * o3["dlogp"])


def test_loss_aggregation_modes():
    rng = np.random.default_rng(9)
    # one sequence, or equal lengths: both aggregations coincide
    for lens in ([11], [4, 4, 4]):
        logp, old, ref, A, cu = _loss_inputs(rng, lens)
        a = O.policy_loss_ref(logp, old, ref, A, cu, agg_mode=0)
        b = O.policy_loss_ref(logp, old, ref, A, cu, agg_mode=1)
        assert abs(a["loss"] - b["loss"]) < 1e-13 and np.allclose(a["dlogp"], b["dlogp"], atol=1e-15)
    # unequal lengths: mode 0 weights each sequence equally -- check by hand on 2 sequences
    lens = [1, 3]
    logp, old, ref, A, cu = _loss_inputs(rng, lens)
    a = O.policy_loss_ref(logp, old, ref, A, cu, agg_mode=0, kl_coef=0.3)
    parts = []
    for i in range(2):
        seg = slice(cu[i], cu[i + 1])
        s = O.policy_loss_ref(logp[seg], old[seg], ref[seg], A[i:i + 1], [0, lens[i]], agg_mode=1, kl_coef=0.3)
        parts.append(s["loss"])
    assert abs(a["loss"] - 0.5 * (parts[0] + parts[1])) < 1e-13
    # entropy is only averaged, never part of the loss
    ent = rng.random(4)
    e = O.policy_loss_ref(logp, old, ref, A, cu, entropy=ent)
    assert abs(e["entropy_mean"] - ent.mean()) < 1e-15
    assert e["loss"] == O.policy_loss_ref(logp, old, ref, A, cu)["loss"]


@pytest.mark.parametrize("agg_mode", [0, 1])
def test_loss_gradient_finite_difference(agg_mode):
    rng = np.random.default_rng(20 + agg_mode)
    lens = [6, 11, 7, 8]
    logp, old, ref, A, cu = _loss_inputs(rng, lens)
    kw = dict(clip_lo=0.2, clip_hi=0.28, kl_coef=0.04, agg_mode=agg_mode, loss_scale=1.7)
    out = O.policy_loss_ref(logp, old, ref, A, cu, **kw)
    h = 1e-6
    checked = 0
    for t in range(logp.size):
        rho = out["rho"][t]
        if min(abs(rho - 0.8), abs(rho - 1.28)) < 1e-3:
            continue                                     # kink of the clip
        lp, lm = logp.copy(), logp.copy()
        lp[t] += h
        lm[t] -= h
        fd = (O.policy_loss_ref(lp, old, ref, A, cu, **kw)["loss"]
              - O.policy_loss_ref(lm, old, ref, A, cu, **kw)["loss"]) / (2 * h)
        assert abs(fd - out["dlogp"][t]) < 1e-8
        checked += 1
    assert checked >= 8 and out["clipped"].any() and not out["clipped"].all()


# ---------------------------------------------------------------- O5 backward
def _chain_loss(H, W, y, old, ref, A, cu, kw):
    """The whole fp64 chain H, W -> loss written independently with torch-free numpy."""
    z = H @ W.T
    lse = np.log(np.exp(z).sum(1))
    logp = z[np.arange(z.shape[0]), y] - lse
    return O.policy_loss_ref(logp, old, ref, A, cu, **kw)["loss"]


def test_backward_finite_difference_full_chain():
    rng = np.random.default_rng(30)
    lens = [3, 4]
    T, d, V = 7, 6, 11
    # the chain is evaluated in fp64 on the widened bf16 values; gradients are taken w.r.t. them
    Hb, Wb = _rand_hw(rng, T, d, V, ws=0.5)
    H, W = bits_val(Hb), bits_val(Wb)
    y = rng.integers(0, V, T)
    cu = np.array([0, 3, 7])
    A = rng.standard_normal(2)
    logp0, _, lse0 = O.token_logprob_ref(Hb, Wb, y)
    old = logp0 + 0.05 * rng.standard_normal(T)          # well inside the clip range
    ref = logp0 + 0.2 * rng.standard_normal(T)
    kw = dict(clip_lo=0.2, clip_hi=0.2, kl_coef=0.04, agg_mode=0, loss_scale=1.0)
    g = O.policy_loss_ref(logp0, old, ref, A, cu, **kw)["dlogp"]
    dH, dW = O.policy_loss_backward_ref(Hb, Wb, y, lse0, g)
    assert dH.shape == (T, d) and dW.shape == (V, d)
    h = 1e-6
    for t in range(T):
        for k in range(d):
            Hp, Hm = H.copy(), H.copy()
            Hp[t, k] += h
            Hm[t, k] -= h
            fd = (_chain_loss(Hp, W, y, old, ref, A, cu, kw) - _chain_loss(Hm, W, y, old, ref, A, cu, kw)) / (2 * h)
            assert abs(fd - dH[t, k]) < 2e-9
    for v in range(V):
        for k in range(d):
            Wp, Wm = W.copy(), W.copy()
            Wp[v, k] += h
            Wm[v, k] -= h
            fd = (_chain_loss(H, Wp, y, old, ref, A, cu, kw) - _chain_loss(H, Wm, y, old, ref, A, cu, kw)) / (2 * h)
            assert abs(fd - dW[v, k]) < 2e-9


def test_backward_structure():
    rng = np.random.default_rng(31)
    T, d, V = 10, 8, 23
    Hb, Wb = _rand_hw(rng, T, d, V)
    y = rng.integers(0, V, T)
    _, _, lse = O.token_logprob_ref(Hb, Wb, y)
    g = rng.standard_normal(T)
    dH, dW = O.policy_loss_backward_ref(Hb, Wb, y, lse, g)
    H, W = bits_val(Hb), bits_val(Wb)
    # rows of dZ sum to zero => columns of dW sum to zero ... weighted by nothing: sum_v dW[v] = 0
    assert np.allclose(dW.sum(0), 0, atol=1e-12)
    # <dW, W> = sum dZ*Z = <dH, H>
    assert abs((dW * W).sum() - (dH * H).sum()) < 1e-10
    # zero upstream gradient gives exactly zero
    z0 = O.policy_loss_backward_ref(Hb, Wb, y, lse, np.zeros(T))
    assert not z0[0].any() and not z0[1].any()
    # linear in g; row t of dH depends only on token t
    dH2, dW2 = O.policy_loss_backward_ref(Hb, Wb, y, lse, 2 * g)
    assert np.allclose(dH2, 2 * dH) and np.allclose(dW2, 2 * dW)
    one = O.policy_loss_backward_ref(Hb[4:5], Wb, y[4:5], lse[4:5], g[4:5])[0]
    assert np.allclose(one[0], dH[4], atol=1e-13)
    # selected vocabulary rows equal the rows of the dense result
    vs = [int(y[0]), 0, V - 1, 7]
    rows = O.policy_loss_backward_ref(Hb, Wb, y, lse, g, vocab_rows=vs)
    assert np.allclose(rows, dW[vs], atol=1e-12)
    # torch float64 autograd as a second opinion
    Ht = torch.tensor(H, requires_grad=True)
    Wt = torch.tensor(W, requires_grad=True)
    lp = torch.log_softmax(Ht @ Wt.T, 1)[torch.arange(T), torch.from_numpy(y)]
    (lp * torch.from_numpy(g)).sum().backward()
    assert np.allclose(Ht.grad.numpy(), dH, atol=1e-12) and np.allclose(Wt.grad.numpy(), dW, atol=1e-12)


# ---------------------------------------------------------------- O2b vocabulary shards
@pytest.mark.parametrize("cuts", [[0, 50], [0, 17, 50], [0, 1, 2, 49, 50], [0, 25, 25, 50]])
def test_sharded_scoring_merges_to_the_full_vocabulary_result(cuts):
    """Any split of the vocabulary into contiguous shards (an empty one included) merges to the
    full-row definition, which is pinned above on its own."""
    rng = np.random.default_rng(5)
    H = to_bits(rng.normal(size=(9, 12)))
    W = to_bits(rng.normal(size=(50, 12)) * 3.0)          # wide logits: the max shift matters
    y = rng.integers(0, 50, 9)
    parts = []
    for a, b in zip(cuts[:-1], cuts[1:]):
        if b > a:
            parts.append(O.token_logprob_shard_ref(H, W[a:b], y, a))
    logp, ent, lse = O.merge_logprob_shards_ref(np.stack(parts))
    r_logp, r_ent, r_lse = O.token_logprob_ref(H, W, y)
    assert np.allclose(logp, r_logp, atol=1e-12) and np.allclose(ent, r_ent, atol=1e-12)
    assert np.allclose(lse, r_lse, atol=1e-12)


@pytest.mark.parametrize("cuts", [[0, 50], [0, 17, 50], [0, 1, 2, 49, 50]])
def test_sharded_backward_adds_up_to_the_full_vocabulary_gradient(cuts):
    """The shards' contributions to dH add up to the dense dH and their dW rows stack to the dense dW
    (the dense gradient is pinned by finite differences and by autograd above); and by autograd on the
    sharded head itself: d/dH and d/dW_shard of sum_t g_t logp_t with the softmax over all shards."""
    rng = np.random.default_rng(6)
    T, d, V = 9, 12, 50
    Hb = to_bits(rng.normal(size=(T, d)))
    Wb = to_bits(rng.normal(size=(V, d)))
    y = rng.integers(0, V, T)
    y[0], y[1] = cuts[1] - 1, cuts[1] % V                       # targets on both sides of a cut
    g = rng.standard_normal(T)
    _, _, lse = O.token_logprob_ref(Hb, Wb, y)
    dH, dW = O.policy_loss_backward_ref(Hb, Wb, y, lse, g)
    dH_sum, rows = np.zeros_like(dH), []
    for a, b in zip(cuts[:-1], cuts[1:]):
        dH_s, dW_s = O.policy_loss_backward_shard_ref(Hb, Wb[a:b], y, lse, g, a)
        assert dW_s.shape == (b - a, d)
        dH_sum += dH_s
        rows.append(dW_s)
    assert np.allclose(dH_sum, dH, atol=1e-12) and np.allclose(np.concatenate(rows), dW, atol=1e-12)
    Ht = torch.tensor(bits_val(Hb), requires_grad=True)
    shards = [torch.tensor(bits_val(Wb[a:b]), requires_grad=True) for a, b in zip(cuts[:-1], cuts[1:])]
    lp = torch.log_softmax(torch.cat([Ht @ w.T for w in shards], 1), 1)[torch.arange(T), torch.from_numpy(y)]
    (lp * torch.from_numpy(g)).sum().backward()
    for w, r in zip(shards, rows):
        assert np.allclose(w.grad.numpy(), r, atol=1e-12)
    # a target outside the shard contributes only through the softmax term
    a, b = cuts[0], cuts[1]
    far = np.full(T, V - 1 if b <= V - 1 else 0)
    if not (a <= far[0] < b):
        dH_s, dW_s = O.policy_loss_backward_shard_ref(Hb, Wb[a:b], far, lse, g, a)
        z = bits_val(Hb) @ bits_val(Wb[a:b]).T
        assert np.allclose(dW_s, (-(g[:, None]) * np.exp(z - lse[:, None])).T @ bits_val(Hb), atol=1e-12)


def test_shard_statistics_by_hand():
    # one token, hidden = [1, 0], shard rows give logits (2, 0, 1); target id 11 with offset 10 -> z = 0
    H = to_bits(np.array([[1.0, 0.0]]))
    W = to_bits(np.array([[2.0, 5.0], [0.0, -1.0], [1.0, 7.0]]))
    p = O.token_logprob_shard_ref(H, W, np.array([11]), 10)[0]
    assert p[0] == 2.0
    assert abs(p[1] - (1.0 + math.exp(-2.0) + math.exp(-1.0))) < 1e-15
    assert abs(p[2] - (2.0 + 0.0 + math.exp(-1.0))) < 1e-15
    assert p[3] == 0.0
    assert O.token_logprob_shard_ref(H, W, np.array([3]), 10)[0][3] == -np.inf      # target in another shard
