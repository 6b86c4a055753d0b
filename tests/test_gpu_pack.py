"""af_pack_microbatch against the oracle: bit-exact gather, every column, every edge case."""
import numpy as np
import pytest
import torch

from oracle import grpo_oracle as O
from paper_2507_01663_b200 import workloads as wl
from gpu_util import device, np_of, packed_buffers

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2507_01663_b200 import binding as B
    c = B.Context(0)
    yield c
    c.close()


def make_store(w, dev):
    T = w.total_tokens
    cols = {"hidden": wl.gen_hidden(w, dev), "target": wl.gen_target(w, dev),
            "old_logp": wl.gen_noise(w, wl.S_OLD, T, dev) - 3.0, "ref_logp": wl.gen_noise(w, wl.S_REF, T, dev) - 3.0}
    adv = wl.normal01(w.seed, wl.S_MISC, 0, w.N, dev)
    # special bit patterns must survive the copy: NaN payloads, -0.0, infinities
    cols["old_logp"][0] = float("nan")
    cols["old_logp"][1] = -0.0
    cols["ref_logp"][2] = float("-inf")
    return cols, adv


def check_against_oracle(ctx, w, cols, adv, idx, use=("hidden", "target", "old_logp", "ref_logp"), with_adv=True):
    dev = device()
    off = w.tok_offset
    T_cap = int(sum(w.lengths[i] for i in idx))
    out = packed_buffers(T_cap + 3, len(idx) + 2, w.d)
    out = {k: v for k, v in out.items() if k in ("cu_seqlens", "seq_id") + tuple(use) + (("adv_seq",) if with_adv else ())}
    store = {"tok_offset_host": off, "d": w.d}
    store.update({k: cols[k] for k in use})
    if with_adv:
        store["adv"] = adv
    T = ctx.pack_microbatch(store, np.asarray(idx, np.int32), out)
    torch.cuda.synchronize()
    host_cols = {k: (wl.bf16_bits(cols[k]) if k == "hidden" else np_of(cols[k])) for k in use}
    ref = O.pack_microbatch_ref(off, idx, host_cols, np_of(adv) if with_adv else None)
    assert T == T_cap == int(ref["cu_seqlens"][-1])
    B = len(idx)
    assert np.array_equal(np_of(out["cu_seqlens"])[:B + 1], ref["cu_seqlens"])
    assert np.array_equal(np_of(out["seq_id"])[:T], ref["seq_id"])
    for k in use:
        got = wl.bf16_bits(out[k][:T]) if k == "hidden" else np_of(out[k][:T])
        assert got.tobytes() == ref[k].tobytes(), k
    if with_adv:
        assert np_of(out["adv_seq"])[:B].tobytes() == ref["adv_seq"].astype(np.float32).tobytes()
    # nothing written past the packed rows (canary rows stay as initialised)
    if "target" in use:
        assert np.all(np_of(out["target"])[T:] == -7)
    assert np.all(np_of(out["seq_id"])[T:] == -7)
    assert ctx.check_device_errors() == 0


@pytest.mark.parametrize("name", ["cfg1", "cfg5_mini", "cfg3_mini"])
def test_pack_matches_oracle(ctx, name):
    w = wl.make_workload(name)
    cols, adv = make_store(w, device())
    order = wl.arrival_order(w)
    check_against_oracle(ctx, w, cols, adv, np.arange(w.N))            # identity
    check_against_oracle(ctx, w, cols, adv, order)                      # arrival order
    check_against_oracle(ctx, w, cols, adv, order[: max(1, w.N // 3)])  # a subset
    check_against_oracle(ctx, w, cols, adv, [5, 5, 0, 5, w.N - 1])      # duplicates
    check_against_oracle(ctx, w, cols, adv, [3])                        # single sequence
    for mb in wl.microbatches(w)[:3]:
        check_against_oracle(ctx, w, cols, adv, mb)


def test_pack_only_requested_columns(ctx):
    w = wl.make_workload("cfg1")
    cols, adv = make_store(w, device())
    idx = wl.arrival_order(w)[:7]
    check_against_oracle(ctx, w, cols, adv, idx, use=("hidden", "target"), with_adv=False)
    check_against_oracle(ctx, w, cols, adv, idx, use=("target", "ref_logp"), with_adv=True)
    check_against_oracle(ctx, w, cols, adv, idx, use=("hidden",), with_adv=False)


def test_pack_empty_batch_and_zero_length_samples(ctx):
    dev = device()
    w = wl.make_workload("cfg1")
    cols, adv = make_store(w, dev)
    out = packed_buffers(8, 4, w.d)
    store = {"tok_offset_host": w.tok_offset, "d": w.d, **cols, "adv": adv}
    T = ctx.pack_microbatch(store, np.zeros(0, np.int32), out)
    torch.cuda.synchronize()
    assert T == 0 and int(out["cu_seqlens"][0]) == 0 and int(out["cu_seqlens"][1]) == -7
    # a store with empty samples in it
    lengths = np.array([3, 0, 5, 0, 0, 2], np.int64)
    off = np.concatenate([[0], np.cumsum(lengths)])
    d = 16
    H = wl._normal_matrix(9, wl.S_HIDDEN, int(off[-1]), d, 1.0, dev)
    tgt = torch.arange(int(off[-1]), dtype=torch.int32, device=dev)
    idx = np.array([1, 0, 3, 4, 5, 2, 1], np.int32)
    o = {"cu_seqlens": torch.zeros(8, dtype=torch.int32, device=dev), "hidden": torch.zeros(16, d, dtype=torch.bfloat16, device=dev),
         "target": torch.zeros(16, dtype=torch.int32, device=dev), "seq_id": torch.zeros(16, dtype=torch.int32, device=dev)}
    T = ctx.pack_microbatch({"tok_offset_host": off, "d": d, "hidden": H, "target": tgt}, idx, o)
    torch.cuda.synchronize()
    ref = O.pack_microbatch_ref(off, idx, {"hidden": wl.bf16_bits(H), "target": np_of(tgt)})
    assert T == 10
    assert np.array_equal(np_of(o["cu_seqlens"]), ref["cu_seqlens"])
    assert np.array_equal(np_of(o["target"])[:T], ref["target"]) and np.array_equal(np_of(o["seq_id"])[:T], ref["seq_id"])
    assert np.array_equal(wl.bf16_bits(o["hidden"][:T]), ref["hidden"])


@pytest.mark.parametrize("B", [1, 127, 128, 129, 511, 512, 513, 1500])
def test_pack_around_the_inline_table_limit(ctx, B):
    """Up to 512 sequences the table travels with the launch, beyond that through the staged device
    copy: both sides of the limit, with duplicates, empty samples and every column, bit for bit."""
    dev = device()
    rng = np.random.default_rng(B)
    lengths = rng.integers(0, 10, size=700).astype(np.int64)
    off = np.concatenate([[0], np.cumsum(lengths)])
    n_tok, d = int(off[-1]), 64
    H = wl._normal_matrix(B, wl.S_HIDDEN, n_tok, d, 1.0, dev)
    tgt = torch.arange(n_tok, dtype=torch.int32, device=dev)
    old = wl.normal01(B, wl.S_OLD, 0, n_tok, dev)
    adv = wl.normal01(B, wl.S_MISC, 0, 700, dev)
    idx = rng.integers(0, 700, size=B).astype(np.int32)
    T_cap = int(lengths[idx].sum())
    o = {"cu_seqlens": torch.full((B + 2,), -7, dtype=torch.int32, device=dev),
         "hidden": torch.zeros(T_cap + 2, d, dtype=torch.bfloat16, device=dev),
         "target": torch.full((T_cap + 2,), -7, dtype=torch.int32, device=dev),
         "old_logp": torch.zeros(T_cap + 2, device=dev),
         "adv_seq": torch.zeros(B, device=dev),
         "seq_id": torch.full((T_cap + 2,), -7, dtype=torch.int32, device=dev)}
    T = ctx.pack_microbatch({"tok_offset_host": off, "d": d, "hidden": H, "target": tgt, "old_logp": old, "adv": adv},
                            idx, o)
    torch.cuda.synchronize()
    ref = O.pack_microbatch_ref(off, idx, {"hidden": wl.bf16_bits(H), "target": np_of(tgt), "old_logp": np_of(old)},
                                np_of(adv))
    assert T == T_cap
    assert np.array_equal(np_of(o["cu_seqlens"])[:B + 1], ref["cu_seqlens"]) and int(o["cu_seqlens"][B + 1]) == -7
    assert np.array_equal(np_of(o["target"])[:T], ref["target"]) and np.all(np_of(o["target"])[T:] == -7)
    assert np.array_equal(np_of(o["seq_id"])[:T], ref["seq_id"]) and np.all(np_of(o["seq_id"])[T:] == -7)
    assert np_of(o["old_logp"])[:T].tobytes() == ref["old_logp"].tobytes()
    assert np_of(o["adv_seq"]).tobytes() == ref["adv_seq"].astype(np.float32).tobytes()
    assert np.array_equal(wl.bf16_bits(o["hidden"][:T]), ref["hidden"])
    assert not bool(o["hidden"][T:].any())
    assert ctx.check_device_errors() == 0


def test_pack_of_empty_samples_only(ctx):
    """Sequences without tokens still get their cu_seqlens entries and advantages."""
    dev = device()
    off = np.array([0, 0, 4, 4, 4], np.int64)
    d = 32
    H = wl._normal_matrix(3, wl.S_HIDDEN, 4, d, 1.0, dev)
    adv = torch.tensor([1.5, -2.0, 0.25, 8.0], device=dev)
    idx = np.array([0, 2, 3, 0], np.int32)
    o = {"cu_seqlens": torch.full((6,), -7, dtype=torch.int32, device=dev),
         "hidden": torch.zeros(4, d, dtype=torch.bfloat16, device=dev), "adv_seq": torch.zeros(4, device=dev)}
    T = ctx.pack_microbatch({"tok_offset_host": off, "d": d, "hidden": H, "adv": adv}, idx, o)
    torch.cuda.synchronize()
    assert T == 0
    assert np_of(o["cu_seqlens"]).tolist() == [0, 0, 0, 0, 0, -7]
    assert np_of(o["adv_seq"]).tolist() == [1.5, 0.25, 8.0, 1.5]
    assert not bool(o["hidden"].any()) and ctx.check_device_errors() == 0


def test_pack_host_errors(ctx):
    from paper_2507_01663_b200.binding import AfError
    dev = device()
    w = wl.make_workload("cfg1")
    cols, adv = make_store(w, dev)
    store = {"tok_offset_host": w.tok_offset, "d": w.d, **cols, "adv": adv}
    out = packed_buffers(w.total_tokens, w.N, w.d)
    for bad in ([w.N], [-1], [0, 1, 99999]):
        with pytest.raises(AfError) as e:
            ctx.pack_microbatch(store, np.asarray(bad, np.int32), out)
        assert e.value.status == -5
    small = packed_buffers(10, w.N, w.d)
    with pytest.raises(AfError) as e:
        ctx.pack_microbatch(store, np.arange(w.N, dtype=np.int32), small)
    assert e.value.status == -4
    fewseq = packed_buffers(w.total_tokens, 2, w.d)
    with pytest.raises(AfError) as e:
        ctx.pack_microbatch(store, np.arange(5, dtype=np.int32), fewseq)
    assert e.value.status == -4
    # a requested column without an output buffer (and vice versa) is an argument error
    o2 = dict(out)
    o2.pop("old_logp")
    with pytest.raises(AfError) as e:
        ctx.pack_microbatch(store, np.arange(3, dtype=np.int32), o2)
    assert e.value.status == -1
    # the context is still usable afterwards
    check_against_oracle(ctx, w, cols, adv, [1, 2, 3])
