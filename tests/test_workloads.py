"""Host-side checks of the synthetic workload generator (no method arithmetic involved)."""
import numpy as np
import torch

from paper_2507_01663_b200 import workloads as wl


def test_counter_generator_is_positional():
    a = wl.normal01(5, wl.S_HIDDEN, 0, 1000)
    b = wl.normal01(5, wl.S_HIDDEN, 300, 200)
    assert torch.equal(a[300:500], b)
    assert not torch.equal(a[:200], wl.normal01(6, wl.S_HIDDEN, 0, 200))
    assert not torch.equal(a[:200], wl.normal01(5, wl.S_W, 0, 200))
    u = wl.uniform01(1, 2, 0, 200000)
    assert 0 < u.min() and u.max() < 1 and abs(u.mean() - 0.5) < 5e-3
    n = wl.normal01(1, 3, 0, 200000)
    assert abs(n.mean()) < 1e-2 and abs(n.std() - 1) < 1e-2
    r = wl.randint(1, 4, 0, 100000, 7)
    assert r.min() == 0 and r.max() == 6


def test_rows_regenerate():
    w = wl.make_workload("cfg1")
    H = wl.gen_hidden(w)
    assert H.shape == (w.total_tokens, w.d) and H.dtype == torch.bfloat16
    rows = [0, 17, w.total_tokens - 1]
    assert torch.equal(wl.gen_hidden_rows(w, rows), H[rows])


def test_config_shapes():
    c1 = wl.make_workload("cfg1")
    assert (c1.d, c1.V, c1.N, c1.group_size) == (256, 4096, 32, 4)
    assert c1.lengths.min() >= 16 and c1.lengths.max() <= 64
    c2 = wl.make_workload("cfg2")
    assert (c2.d, c2.V, c2.N, c2.group_size) == (3584, 152064, 512, 8)
    assert c2.lengths.min() >= 256 and c2.lengths.max() <= 4096 and 1.0e6 < c2.total_tokens < 1.25e6
    c3 = wl.make_workload("cfg3")
    assert (c3.d, c3.N, c3.group_size) == (5120, 512, 16)
    assert c3.lengths.min() >= 64 and c3.lengths.max() <= 8192
    assert 800 < np.median(c3.lengths) < 1300
    c4 = wl.make_workload("cfg4")
    assert c4.N == 128 and c4.total_tokens == 65536
    assert c4.lengths.min() >= 64 and c4.lengths.max() <= 1024
    c5 = wl.make_workload("cfg5")
    assert c5.N == 4096 and c5.group_size == 64
    assert c5.lengths.min() >= 128 and c5.lengths.max() <= 16384
    assert c5.tok_offset[-1] == c5.total_tokens and np.all(np.diff(c5.tok_offset) == c5.lengths)


def test_microbatches_cover_every_sample_once():
    w = wl.make_workload("cfg5")
    mbs = wl.microbatches(w)
    flat = np.concatenate(mbs)
    assert np.array_equal(np.sort(flat), np.arange(w.N))
    assert np.array_equal(flat, wl.arrival_order(w))
    for mb in mbs:
        tok = int(w.lengths[mb].sum())
        assert tok <= w.token_budget or len(mb) == 1
    assert 30 <= len(mbs) <= 80


def test_rewards_follow_the_stated_law():
    w2 = wl.make_workload("cfg2")
    r = wl.gen_reward(w2)
    assert set(r.tolist()) <= {0.0, 1.0} and 0.2 < r.mean() < 0.4
    r3 = wl.gen_reward(wl.make_workload("cfg3"))
    assert 0 < r3.min() and r3.max() < 1 and len(set(r3.tolist())) > 400


def test_shard_prompts_partition():
    for W in (1, 2, 3, 8):
        owned = [p for r in range(W) for p in wl.shard_prompts(64, W, r)]
        assert owned == list(range(64))
