"""Thin ctypes binding of ``libasyncflow.so`` -- argument marshalling only.

Each function mirrors the C entry point of the same name in ``include/asyncflow.h``.  Tensors
are torch CUDA tensors used as plain device buffers (``data_ptr()``); streams are torch streams.
There is no CPU path: importing this module without the built library, or calling it without a
B200, raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libasyncflow.so")

AF_OK = 0
STATUS_NAMES = {0: "AF_OK", -1: "AF_ERR_INVALID_ARG", -2: "AF_ERR_SHAPE", -3: "AF_ERR_ALIGNMENT",
                -4: "AF_ERR_CAPACITY", -5: "AF_ERR_INDEX", -6: "AF_ERR_WORKSPACE", -7: "AF_ERR_CUDA",
                -8: "AF_ERR_UNSUPPORTED_DEVICE", -9: "AF_ERR_DEVICE_FLAGGED"}
DEVERR_TARGET_RANGE, DEVERR_WATCHDOG, DEVERR_CU_SEQLENS, DEVERR_SAMPLE_INDEX, DEVERR_GROUP_ID = 1, 2, 4, 8, 16

EXPORTS = ["af_create", "af_destroy", "af_status_string", "af_reserve", "af_workspace_bytes",
           "af_set_tuning", "af_check_device_errors", "af_pack_microbatch", "af_token_logprob",
           "af_grpo_advantage", "af_policy_loss", "af_policy_loss_backward", "af_token_logprob_static",
           "af_controller_put", "af_controller_get", "af_controller_clear", "af_balance_partitions",
           "af_token_logprob_shard", "af_merge_logprob_shards", "af_policy_update", "af_unpack_microbatch", "af_policy_loss_backward_shard", "af_set_dw_ready_event", "af_die_split", "af_selftest_bounded_wait",
           "af_plan_token_logprob", "af_plan_units"]
MAX_WRITE_COLS = 4


class AfError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)}")


class StoreView(C.Structure):
    _fields_ = [("n_samples", C.c_int64), ("d", C.c_int32), ("reserved", C.c_int32),
                ("tok_offset_host", C.c_void_p), ("hidden", C.c_void_p), ("target", C.c_void_p),
                ("old_logp", C.c_void_p), ("ref_logp", C.c_void_p), ("adv", C.c_void_p)]


class Packed(C.Structure):
    _fields_ = [("token_capacity", C.c_int64), ("seq_capacity", C.c_int32), ("reserved", C.c_int32),
                ("cu_seqlens", C.c_void_p), ("hidden", C.c_void_p), ("target", C.c_void_p),
                ("old_logp", C.c_void_p), ("ref_logp", C.c_void_p), ("adv_seq", C.c_void_p),
                ("seq_id", C.c_void_p)]


class LossParams(C.Structure):
    _fields_ = [("clip_lo", C.c_float), ("clip_hi", C.c_float), ("kl_coef", C.c_float),
                ("agg_mode", C.c_int32), ("loss_scale", C.c_float)]


class LossOut(C.Structure):
    _fields_ = [("loss", C.c_float), ("pg_loss", C.c_float), ("kl_mean", C.c_float),
                ("clip_frac", C.c_float), ("entropy_mean", C.c_float), ("reserved", C.c_int32),
                ("n_tokens", C.c_int64)]


class ControllerView(C.Structure):
    _fields_ = [("n_samples", C.c_int64), ("ready", C.c_void_p), ("consumed", C.c_void_p), ("length", C.c_void_p)]


class WriteCols(C.Structure):
    _fields_ = [("n_cols", C.c_int32), ("reserved", C.c_int32), ("packed", C.c_void_p * 4), ("store", C.c_void_p * 4)]


class GetResult(C.Structure):
    _fields_ = [("count", C.c_int32), ("eligible", C.c_int32), ("tokens", C.c_int64)]


_lib = None


def load_library() -> C.CDLL:
    """dlopen the in-tree library.  A missing library is compiled first when nvcc is at hand (a
    fresh checkout); otherwise this fails loudly: there is no fallback implementation."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        try:
            from . import build as _build
            _build.build()
        except Exception as exc:
            raise ImportError(f"{LIB_PATH} is missing and could not be built ({exc}): run "
                              "`python -m paper_2507_01663_b200.build` (there is no fallback implementation)")
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64, f32 = C.c_void_p, C.c_int32, C.c_int64, C.c_float
    lib.af_create.argtypes = [C.POINTER(vp), C.c_int]
    lib.af_destroy.argtypes = [vp]
    lib.af_status_string.argtypes = [C.c_int]
    lib.af_status_string.restype = C.c_char_p
    lib.af_reserve.argtypes = [vp, i64, i32, i32, i32, i32]
    lib.af_workspace_bytes.argtypes = [vp]
    lib.af_workspace_bytes.restype = i64
    lib.af_set_tuning.argtypes = [vp, i32, i32, i32]
    lib.af_check_device_errors.argtypes = [vp, C.POINTER(C.c_uint32), vp]
    lib.af_set_dw_ready_event.argtypes = [vp, vp]
    lib.af_die_split.argtypes = [vp, C.POINTER(i32), C.POINTER(i32)]
    lib.af_selftest_bounded_wait.argtypes = [vp, C.POINTER(C.c_uint32), vp]
    lib.af_pack_microbatch.argtypes = [vp, C.POINTER(StoreView), vp, i32, C.POINTER(Packed),
                                       C.POINTER(i64), vp]
    lib.af_token_logprob.argtypes = [vp, vp, vp, vp, i64, i32, i32, vp, vp, vp, vp]
    lib.af_grpo_advantage.argtypes = [vp, vp, vp, i64, i32, f32, i32, vp, vp]
    lib.af_policy_loss.argtypes = [vp, vp, vp, vp, vp, vp, vp, i32, i64, C.POINTER(LossParams), vp,
                                   vp, vp]
    lib.af_policy_loss_backward.argtypes = [vp, vp, vp, vp, vp, vp, i64, i32, i32, vp, vp, i32, vp]
    lib.af_token_logprob_static.argtypes = [vp, vp, vp, i64, i32, i32, vp, vp, vp, vp, vp]
    u32 = C.c_uint32
    lib.af_controller_put.argtypes = [vp, C.POINTER(ControllerView), vp, i64, u32, vp]
    lib.af_controller_get.argtypes = [vp, C.POINTER(ControllerView), u32, u32, i32, i64, vp, vp, vp]
    lib.af_controller_clear.argtypes = [vp, C.POINTER(ControllerView), u32, u32, vp]
    lib.af_balance_partitions.argtypes = [vp, i32, i32, i32, vp, vp]
    lib.af_token_logprob_shard.argtypes = [vp, vp, vp, vp, i64, i32, i32, i32, vp, vp]
    lib.af_merge_logprob_shards.argtypes = [vp, vp, vp, i32, i64, i32, vp, vp, vp, vp]
    lib.af_policy_update.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i32, i64, i32, i32, C.POINTER(LossParams), vp,
                                     vp, vp, vp, vp, vp, vp, i32, vp]
    lib.af_policy_loss_backward_shard.argtypes = [vp, vp, vp, vp, vp, vp, i64, i32, i32, i32, vp, vp, i32, vp]
    lib.af_unpack_microbatch.argtypes = [vp, vp, i64, vp, i32, C.POINTER(WriteCols), C.POINTER(ControllerView), u32,
                                         C.POINTER(i64), vp]
    for name in EXPORTS:
        if name not in ("af_status_string", "af_workspace_bytes"):
            getattr(lib, name).restype = C.c_int
    _lib = lib
    return lib


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("device buffers must be contiguous CUDA tensors")
    return C.c_void_p(t.data_ptr())


def _stream(stream) -> C.c_void_p:
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def _check(status: int, where: str):
    if status != AF_OK:
        raise AfError(status, where)


class Context:
    """Owner of an ``af_ctx`` (workspace + device error word) on one CUDA device."""

    def __init__(self, device: int = 0):
        self.lib = load_library()
        self.device = device
        h = C.c_void_p()
        _check(self.lib.af_create(C.byref(h), device), "af_create")
        self.handle = h

    def close(self):
        if getattr(self, "handle", None):
            self.lib.af_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- housekeeping ------------------------------------------------------------------------
    def reserve(self, max_T: int, max_B: int, d: int, V: int, with_backward=False):
        """with_backward: False / True (backward scratch) / 2 (also the fused update's)."""
        _check(self.lib.af_reserve(self.handle, max_T, max_B, d, V, int(with_backward)), "af_reserve")

    def workspace_bytes(self) -> int:
        return int(self.lib.af_workspace_bytes(self.handle))

    def set_tuning(self, v_splits: int = 0, bwd_token_block: int = 0, gemm_variant: int = 0):
        """gemm_variant: 0 = default (CTA pairs, row tiles dealt by die), 1 = one CTA per tile, 2 = CTA
        pairs dealt without regard to dies, 3 = same as 0."""
        _check(self.lib.af_set_tuning(self.handle, v_splits, bwd_token_block, gemm_variant), "af_set_tuning")

    def set_dw_ready_event(self, event: Optional[torch.cuda.Event]):
        """Register a torch CUDA event that the backward / fused-update calls record once d_W is
        complete (None clears it).  The event must have been recorded once, so that it exists."""
        _check(self.lib.af_set_dw_ready_event(self.handle, None if event is None else C.c_void_p(event.cuda_event)),
               "af_set_dw_ready_event")

    def die_split(self):
        """(SMs on the first die, SMs on the other) as measured at creation; (0, 0) if unclear."""
        a, b = C.c_int32(0), C.c_int32(0)
        _check(self.lib.af_die_split(self.handle, C.byref(a), C.byref(b)), "af_die_split")
        return int(a.value), int(b.value)

    def selftest_bounded_wait(self, stream=None) -> int:
        """Run the library's bounded wait on a barrier nobody arrives at (limit: 1 ms); returns the
        microseconds the warp waited.  Leaves DEVERR_WATCHDOG set for check_device_errors."""
        us = C.c_uint32(0)
        _check(self.lib.af_selftest_bounded_wait(self.handle, C.byref(us), _stream(stream)), "af_selftest_bounded_wait")
        return int(us.value)

    def check_device_errors(self, stream=None) -> int:
        """Synchronise the stream; return the device error bits (0 = none) and clear them."""
        flags = C.c_uint32(0)
        st = self.lib.af_check_device_errors(self.handle, C.byref(flags), _stream(stream))
        if st not in (AF_OK, -9):
            raise AfError(st, "af_check_device_errors")
        return int(flags.value)

    # -- the five entry points ---------------------------------------------------------------
    def pack_microbatch(self, store: dict, idx_host: np.ndarray, out: dict, stream=None) -> int:
        """``store``: tok_offset_host (np.int64 [N+1]), d, and device columns hidden / target /
        old_logp / ref_logp / adv (missing or None = not requested).  ``out``: device buffers
        cu_seqlens, hidden, target, old_logp, ref_logp, adv_seq, seq_id.  Returns T."""
        off = np.ascontiguousarray(store["tok_offset_host"], dtype=np.int64)
        idx = np.ascontiguousarray(idx_host, dtype=np.int32)
        sv = StoreView(n_samples=off.shape[0] - 1, d=int(store["d"]), reserved=0,
                       tok_offset_host=off.ctypes.data, hidden=_ptr(store.get("hidden")),
                       target=_ptr(store.get("target")), old_logp=_ptr(store.get("old_logp")),
                       ref_logp=_ptr(store.get("ref_logp")), adv=_ptr(store.get("adv")))
        cu = out["cu_seqlens"]
        cap_t = min([out[k].shape[0] for k in ("hidden", "target", "old_logp", "ref_logp", "seq_id")
                     if out.get(k) is not None] or [0])
        pk = Packed(token_capacity=cap_t, seq_capacity=cu.shape[0] - 1, reserved=0, cu_seqlens=_ptr(cu),
                    hidden=_ptr(out.get("hidden")), target=_ptr(out.get("target")),
                    old_logp=_ptr(out.get("old_logp")), ref_logp=_ptr(out.get("ref_logp")),
                    adv_seq=_ptr(out.get("adv_seq")), seq_id=_ptr(out.get("seq_id")))
        T = C.c_int64(0)
        st = self.lib.af_pack_microbatch(self.handle, C.byref(sv), C.c_void_p(idx.ctypes.data),
                                         idx.shape[0], C.byref(pk), C.byref(T), _stream(stream))
        _check(st, "af_pack_microbatch")
        return int(T.value)

    def unpack_microbatch(self, tok_offset_host: np.ndarray, idx_host: np.ndarray, packed: list, store: list,
                          table: Optional[dict] = None, column_bits: int = 0, stream=None) -> int:
        """Write per-token results back by index list: ``packed[k]`` (device, [T], 4-byte elements in
        packed order) goes to the rows of the listed samples in ``store[k]`` (device, [sum L]).  With
        ``table`` the ``column_bits`` of the listed samples' ready masks are set afterwards.  Returns T."""
        off = np.ascontiguousarray(tok_offset_host, dtype=np.int64)
        idx = np.ascontiguousarray(idx_host, dtype=np.int32)
        if len(packed) != len(store):
            raise ValueError("one store column per packed column")
        for a, b in zip(packed, store):
            if a.element_size() != 4 or b.element_size() != 4:
                raise ValueError("write-back columns hold 4-byte elements")
        wc = WriteCols(n_cols=len(packed), reserved=0)
        for k in range(min(len(packed), MAX_WRITE_COLS)):
            wc.packed[k] = _ptr(packed[k]).value
            wc.store[k] = _ptr(store[k]).value
        tv = self._table(table) if table is not None else None
        T = C.c_int64(0)
        st = self.lib.af_unpack_microbatch(self.handle, C.c_void_p(off.ctypes.data), off.shape[0] - 1,
                                           C.c_void_p(idx.ctypes.data), idx.shape[0], C.byref(wc),
                                           C.byref(tv) if tv is not None else None, column_bits, C.byref(T),
                                           _stream(stream))
        _check(st, "af_unpack_microbatch")
        return int(T.value)

    def token_logprob(self, hidden, W, target, logp, entropy=None, lse=None, T=None, stream=None):
        T = hidden.shape[0] if T is None else T
        d, V = W.shape[1], W.shape[0]
        _check(self.lib.af_token_logprob(self.handle, _ptr(hidden), _ptr(W), _ptr(target), T, d, V,
                                         _ptr(logp), _ptr(entropy), _ptr(lse), _stream(stream)),
               "af_token_logprob")

    def token_logprob_shard(self, hidden, W_shard, target, v_offset, partial_out, T=None, stream=None):
        """``partial_out``: device float32 [T, 4] = (m, s, u, zy) of this vocabulary shard."""
        T = hidden.shape[0] if T is None else T
        d, Vs = W_shard.shape[1], W_shard.shape[0]
        _check(self.lib.af_token_logprob_shard(self.handle, _ptr(hidden), _ptr(W_shard), _ptr(target), T, d, Vs,
                                               v_offset, _ptr(partial_out), _stream(stream)),
               "af_token_logprob_shard")

    def merge_logprob_shards(self, partials, target, V_total, logp, entropy=None, lse=None, T=None, stream=None):
        """``partials``: device float32 [R, T, 4], the shards' statistics after the exchange."""
        R = partials.shape[0]
        T = partials.shape[1] if T is None else T
        _check(self.lib.af_merge_logprob_shards(self.handle, _ptr(partials), _ptr(target), R, T, V_total,
                                                _ptr(logp), _ptr(entropy), _ptr(lse), _stream(stream)),
               "af_merge_logprob_shards")

    def grpo_advantage(self, reward, group_id, n_groups, adv, eps_adv=1e-6, ddof=0, N=None, stream=None):
        N = reward.shape[0] if N is None else N
        _check(self.lib.af_grpo_advantage(self.handle, _ptr(reward), _ptr(group_id), N, n_groups,
                                          eps_adv, ddof, _ptr(adv), _stream(stream)), "af_grpo_advantage")

    def policy_loss(self, logp, old_logp, ref_logp, adv_seq, cu_seqlens, out, dlogp=None, entropy=None,
                    clip_lo=0.2, clip_hi=0.2, kl_coef=0.04, agg_mode=0, loss_scale=1.0, B=None, T=None,
                    stream=None):
        """``out``: device uint8 tensor of ``ctypes.sizeof(LossOut)`` bytes (see read_loss_out)."""
        B = cu_seqlens.shape[0] - 1 if B is None else B
        T = logp.shape[0] if T is None else T
        prm = LossParams(clip_lo, clip_hi, kl_coef, agg_mode, loss_scale)
        _check(self.lib.af_policy_loss(self.handle, _ptr(logp), _ptr(old_logp), _ptr(ref_logp),
                                       _ptr(entropy), _ptr(adv_seq), _ptr(cu_seqlens), B, T,
                                       C.byref(prm), _ptr(out), _ptr(dlogp), _stream(stream)),
               "af_policy_loss")

    def policy_loss_backward(self, hidden, W, target, lse, dlogp, d_hidden, d_W, accumulate_dW=False,
                             T=None, stream=None):
        T = hidden.shape[0] if T is None else T
        d, V = W.shape[1], W.shape[0]
        _check(self.lib.af_policy_loss_backward(self.handle, _ptr(hidden), _ptr(W), _ptr(target),
                                                _ptr(lse), _ptr(dlogp), T, d, V, _ptr(d_hidden),
                                                _ptr(d_W), int(accumulate_dW), _stream(stream)),
               "af_policy_loss_backward")


    def policy_loss_backward_shard(self, hidden, W_shard, target, lse, dlogp, v_offset, d_hidden_partial, d_W_shard,
                                   accumulate_dW=False, T=None, stream=None):
        T = hidden.shape[0] if T is None else T
        d, Vs = W_shard.shape[1], W_shard.shape[0]
        _check(self.lib.af_policy_loss_backward_shard(self.handle, _ptr(hidden), _ptr(W_shard), _ptr(target),
                                                      _ptr(lse), _ptr(dlogp), T, d, Vs, v_offset,
                                                      _ptr(d_hidden_partial), _ptr(d_W_shard), int(accumulate_dW),
                                                      _stream(stream)),
               "af_policy_loss_backward_shard")

    def policy_update(self, hidden, W, target, old_logp, ref_logp, adv_seq, cu_seqlens, out, logp, lse, d_hidden,
                      d_W, entropy=None, dlogp=None, accumulate_dW=False, clip_lo=0.2, clip_hi=0.2, kl_coef=0.04,
                      agg_mode=0, loss_scale=1.0, B=None, T=None, stream=None):
        """``af_policy_update``: forward + loss + backward of one packed micro-batch in one call."""
        B = cu_seqlens.shape[0] - 1 if B is None else B
        T = hidden.shape[0] if T is None else T
        d, V = W.shape[1], W.shape[0]
        prm = LossParams(clip_lo, clip_hi, kl_coef, agg_mode, loss_scale)
        _check(self.lib.af_policy_update(self.handle, _ptr(hidden), _ptr(W), _ptr(target), _ptr(old_logp),
                                         _ptr(ref_logp), _ptr(adv_seq), _ptr(cu_seqlens), B, T, d, V, C.byref(prm),
                                         _ptr(out), _ptr(logp), _ptr(entropy), _ptr(lse), _ptr(dlogp), _ptr(d_hidden),
                                         _ptr(d_W), int(accumulate_dW), _stream(stream)), "af_policy_update")

    # -- controller: status table of the streaming store ----------------------------------------
    @staticmethod
    def _table(table: dict) -> ControllerView:
        """``table``: device tensors ready / consumed (int32 or uint32 bit masks, [N]) and
        optionally length (int32 [N])."""
        ready = table["ready"]
        return ControllerView(n_samples=ready.shape[0], ready=_ptr(ready), consumed=_ptr(table["consumed"]),
                              length=_ptr(table.get("length")))

    def controller_put(self, table: dict, idx: torch.Tensor, column_bits: int, n=None, stream=None):
        tv = self._table(table)
        n = idx.shape[0] if n is None else n
        _check(self.lib.af_controller_put(self.handle, C.byref(tv), _ptr(idx), n, column_bits, _stream(stream)),
               "af_controller_put")

    def controller_get(self, table: dict, column_mask: int, task_bit: int, max_samples: int, token_budget: int,
                       out_idx: torch.Tensor, out: torch.Tensor, stream=None):
        """``out_idx``: device int32 [>= max_samples]; ``out``: device uint8 buffer of
        ``ctypes.sizeof(GetResult)`` bytes (see read_get_result)."""
        tv = self._table(table)
        _check(self.lib.af_controller_get(self.handle, C.byref(tv), column_mask, task_bit, max_samples,
                                          token_budget, _ptr(out_idx), _ptr(out), _stream(stream)),
               "af_controller_get")

    def controller_clear(self, table: dict, column_bits: int, task_bits: int, stream=None):
        tv = self._table(table)
        _check(self.lib.af_controller_clear(self.handle, C.byref(tv), column_bits, task_bits, _stream(stream)),
               "af_controller_clear")


class GemmPlan(C.Structure):
    """Mirror of ``af_gemm_plan``."""
    _fields_ = [("m_tiles", C.c_int32), ("n_tiles", C.c_int32), ("v_splits", C.c_int32), ("workers", C.c_int32),
                ("die0_workers", C.c_int32), ("die0_row_tiles", C.c_int32)]


def plan_token_logprob(T: int, d: int, V: int, sm_count: int, die0_sms: int = 0, v_splits: int = 0,
                       gemm_variant: int = 0) -> GemmPlan:
    """``af_plan_token_logprob`` (host): the work decomposition of a scoring call."""
    plan = GemmPlan()
    _check(load_library().af_plan_token_logprob(C.c_int64(T), d, V, sm_count, die0_sms, v_splits, gemm_variant,
                                                C.byref(plan)), "af_plan_token_logprob")
    return plan


def plan_units(plan: GemmPlan, rank: int) -> range:
    """``af_plan_units`` (host): the units worker ``rank`` processes."""
    first, stride, end = C.c_int32(), C.c_int32(), C.c_int32()
    _check(load_library().af_plan_units(C.byref(plan), rank, C.byref(first), C.byref(stride), C.byref(end)),
           "af_plan_units")
    return range(first.value, end.value, stride.value)


def balance_partitions(length, k: int, equal_size: bool):
    """``af_balance_partitions`` (host): returns (part [n] int32, group token totals [k] int64)."""
    lib = load_library()
    L = np.ascontiguousarray(length, dtype=np.int32)
    part = np.empty(L.shape[0], dtype=np.int32)
    sums = np.zeros(k, dtype=np.int64)
    _check(lib.af_balance_partitions(C.c_void_p(L.ctypes.data) if L.size else None, L.shape[0], k, int(equal_size),
                                     C.c_void_p(part.ctypes.data) if L.size else None,
                                     C.c_void_p(sums.ctypes.data)), "af_balance_partitions")
    return part, sums


def new_get_result(device) -> torch.Tensor:
    return torch.zeros(C.sizeof(GetResult), dtype=torch.uint8, device=device)


def read_get_result(buf: torch.Tensor) -> dict:
    """Copy the device ``af_get_result`` to the host (synchronises) and return it as a dict."""
    o = GetResult.from_buffer_copy(buf.cpu().numpy().tobytes())
    return {"count": o.count, "eligible": o.eligible, "tokens": o.tokens}


def new_loss_out(device) -> torch.Tensor:
    return torch.zeros(C.sizeof(LossOut), dtype=torch.uint8, device=device)


def read_loss_out(buf: torch.Tensor) -> dict:
    """Copy the device ``af_loss_out`` to the host (synchronises) and return it as a dict."""
    raw = buf.cpu().numpy().tobytes()
    o = LossOut.from_buffer_copy(raw)
    return {k: getattr(o, k) for k, _ in LossOut._fields_ if k != "reserved"}


def token_logprob_static(hidden, W, target, logp, entropy=None, lse=None, device_flags=None, T=None,
                         stream=None):
    """``af_token_logprob_static``: the scoring call without a context and without any allocation
    (scratch is a fixed array inside the library; at most 32768 tokens per call).  Runs on the
    current CUDA device; calls sharing a device must not overlap on the GPU."""
    lib = load_library()
    T = hidden.shape[0] if T is None else T
    d, V = W.shape[1], W.shape[0]
    _check(lib.af_token_logprob_static(_ptr(hidden), _ptr(W), _ptr(target), T, d, V, _ptr(logp),
                                       _ptr(entropy), _ptr(lse), _ptr(device_flags), _stream(stream)),
           "af_token_logprob_static")
