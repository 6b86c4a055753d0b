// C ABI of the asyncflow library: argument validation, context and workspace management,
// tensor-map encoding.  All arithmetic lives in the kernels of the other translation units.
#include <algorithm>
#include <cstdint>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include <nvtx3/nvToolsExt.h>

#include "common.cuh"

namespace af {

af_status ws_grow(Buf& b, size_t bytes) {
  if (bytes <= b.cap) return AF_OK;
  if (b.p) { cudaFree(b.p); b.p = nullptr; b.cap = 0; }
  size_t want = (bytes + 255) & ~(size_t)255;
  if (cudaMalloc(&b.p, want) != cudaSuccess) { b.p = nullptr; cudaGetLastError(); return AF_ERR_WORKSPACE; }
  b.cap = want;
  return AF_OK;
}

namespace {
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// A named range around every entry point that enqueues work, for timelines of a profiler that
// understands NVTX (header-only: without such a tool attached the calls do nothing).
struct NvtxRange {
  explicit NvtxRange(const char* name) { nvtxRangePushA(name); }
  ~NvtxRange() { nvtxRangePop(); }
};

struct DeviceGuard {
  int prev = -1;
  bool ok = true;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
    if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
  }
  ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};
}  // namespace
}  // namespace af

using namespace af;

extern "C" {

const char* af_status_string(af_status s) {
  switch (s) {
    case AF_OK: return "ok";
    case AF_ERR_INVALID_ARG: return "invalid argument";
    case AF_ERR_SHAPE: return "unsupported shape";
    case AF_ERR_ALIGNMENT: return "pointer or pitch not 16-byte aligned";
    case AF_ERR_CAPACITY: return "output capacity exceeded";
    case AF_ERR_INDEX: return "sample index out of range";
    case AF_ERR_WORKSPACE: return "workspace allocation failed";
    case AF_ERR_CUDA: return "CUDA call failed";
    case AF_ERR_UNSUPPORTED_DEVICE: return "device is not compute capability 10.0";
    case AF_ERR_DEVICE_FLAGGED: return "device error word set";
  }
  return "unknown status";
}

af_status af_create(af_ctx** out, int device) {
  if (!out) return AF_ERR_INVALID_ARG;
  *out = nullptr;
  int count = 0;
  if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) {
    cudaGetLastError();
    return AF_ERR_UNSUPPORTED_DEVICE;
  }
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return AF_ERR_CUDA;
  if (prop.major != 10 || prop.minor != 0) return AF_ERR_UNSUPPORTED_DEVICE;
  DeviceGuard guard(device);
  if (!guard.ok) return AF_ERR_CUDA;
  af_ctx* c = new (std::nothrow) af_ctx();
  if (!c) return AF_ERR_WORKSPACE;
  c->device = device;
  c->sm_count = prop.multiProcessorCount;
  c->gemm_pair = c->sm_count >= 2 ? 1 : 0;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess || !fn) {
    af_destroy(c);
    return AF_ERR_CUDA;
  }
  c->encode = reinterpret_cast<EncodeTiledFn>(fn);
  if (cudaMalloc(&c->d_err, kDeviceBlockBytes) != cudaSuccess) { c->d_err = nullptr; cudaGetLastError(); af_destroy(c); return AF_ERR_WORKSPACE; }
  if (cudaMemset(c->d_err, 0, kDeviceBlockBytes) != cudaSuccess) { af_destroy(c); return AF_ERR_CUDA; }
  // which SMs share a die (for die-aware dealing of GEMM row tiles); 0 when the measurement is unclear
  if (!measure_die_map(c->sm_count, reinterpret_cast<unsigned char*>(c->d_err) + kDieTableByte, &c->die0_sms,
                       &c->die_map_reason)) c->die0_sms = 0;
  c->die_aware = 1;
  af_status st = ws_grow(c->loss_ws, loss_workspace_bytes(c->sm_count));
  if (st == AF_OK && cudaMemset(c->loss_ws.p, 0, c->loss_ws.cap) != cudaSuccess) st = AF_ERR_CUDA;
  if (st == AF_OK) st = ws_grow(c->ctrl_ws, controller_workspace_bytes(c->sm_count));
  if (st != AF_OK) { af_destroy(c); return st; }
  *out = c;
  return AF_OK;
}

af_status af_destroy(af_ctx* c) {
  if (!c) return AF_ERR_INVALID_ARG;
  DeviceGuard guard(c->device);
  cudaDeviceSynchronize();
  Buf* bufs[] = {&c->partial, &c->loss_ws, &c->pack_meta, &c->dz, &c->ctrl_ws, &c->zlog, &c->adv_ws};
  for (Buf* b : bufs) if (b->p) cudaFree(b->p);
  for (int i = 0; i < kPackRing; ++i) {
    if (c->pack_host[i]) cudaFreeHost(c->pack_host[i]);
    if (c->pack_evt_live[i]) cudaEventDestroy(c->pack_evt[i]);
  }
  if (c->d_err) cudaFree(c->d_err);
  delete c;
  return AF_OK;
}

int64_t af_workspace_bytes(const af_ctx* c) {
  if (!c) return 0;
  return (int64_t)(c->partial.cap + c->loss_ws.cap + c->pack_meta.cap + c->dz.cap + c->ctrl_ws.cap + c->zlog.cap + c->adv_ws.cap);
}

af_status af_selftest_bounded_wait(af_ctx* c, uint32_t* waited_us, void* stream) {
  if (!c) return AF_ERR_INVALID_ARG;
  DeviceGuard guard(c->device);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  unsigned int* d_us = c->d_err + 20;           // a spare word of the context's device block
  if (launch_bounded_wait_selftest(c->d_err, d_us, s) != cudaSuccess) return AF_ERR_CUDA;
  unsigned int us = 0;
  if (cudaMemcpyAsync(&us, d_us, sizeof(us), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
      cudaStreamSynchronize(s) != cudaSuccess) return AF_ERR_CUDA;
  if (waited_us) *waited_us = us;
  return AF_OK;
}

af_status af_die_split(const af_ctx* c, int32_t* die0_sms, int32_t* die1_sms) {
  if (!c || !die0_sms || !die1_sms) return AF_ERR_INVALID_ARG;
  *die0_sms = c->die0_sms;
  *die1_sms = c->die0_sms > 0 ? c->sm_count - c->die0_sms : -c->die_map_reason;
  return AF_OK;
}

af_status af_set_tuning(af_ctx* c, int32_t v_splits, int32_t bwd_token_block, int32_t gemm_variant) {
  if (!c || v_splits < 0 || bwd_token_block < 0 || gemm_variant < 0 || gemm_variant > 3) return AF_ERR_INVALID_ARG;
  if (bwd_token_block % 128 != 0) return AF_ERR_SHAPE;
  c->v_splits = v_splits;
  c->bwd_token_block = bwd_token_block;
  c->gemm_pair = gemm_variant == 1 ? 0 : (c->sm_count >= 2 ? 1 : 0);
  c->die_aware = gemm_variant == 2 ? 0 : 1;      // 0 and 3: by die where the die map was measured; 2: plain dealing
  return AF_OK;
}

af_status af_plan_token_logprob(int64_t T, int32_t d, int32_t V, int32_t sm_count, int32_t die0_sms,
                                int32_t v_splits, int32_t gemm_variant, af_gemm_plan* plan) {
  if (!plan || T < 1 || d < 1 || V < 1 || sm_count < 1 || die0_sms < 0 || die0_sms > sm_count || v_splits < 0 ||
      gemm_variant < 0 || gemm_variant > 3)
    return AF_ERR_INVALID_ARG;
  if (T >= ((int64_t)1 << 31)) return AF_ERR_SHAPE;
  const bool pair = gemm_variant != 1 && sm_count >= 2;          // as af_set_tuning reads the variant
  plan_token_logprob(T, d, V, sm_count, die0_sms, v_splits, pair, gemm_variant != 2, plan);
  return AF_OK;
}

af_status af_plan_units(const af_gemm_plan* plan, int32_t rank, int32_t* first, int32_t* stride, int32_t* end) {
  if (!plan || !first || !stride || !end || plan->workers < 1 || rank < 0 || rank >= plan->workers ||
      plan->m_tiles < 1 || plan->v_splits < 1 || plan->die0_workers < 0 || (plan->die0_workers > 0 && plan->die0_workers >= plan->workers) ||
      plan->die0_row_tiles < 0 || plan->die0_row_tiles > plan->m_tiles)
    return AF_ERR_INVALID_ARG;
  int f = 0, st = 1, e = 0;
  plan_units(*plan, rank, &f, &st, &e);
  *first = f; *stride = st; *end = e;
  return AF_OK;
}

af_status af_set_dw_ready_event(af_ctx* c, void* event) {
  if (!c) return AF_ERR_INVALID_ARG;
  c->dw_ready = static_cast<cudaEvent_t>(event);
  return AF_OK;
}

af_status af_check_device_errors(af_ctx* c, uint32_t* flags, void* stream) {
  NvtxRange range("af_check_device_errors");
  if (!c) return AF_ERR_INVALID_ARG;
  DeviceGuard guard(c->device);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  unsigned int h = 0;
  if (cudaMemcpyAsync(&h, c->d_err, sizeof(h), cudaMemcpyDeviceToHost, s) != cudaSuccess) return AF_ERR_CUDA;
  if (cudaMemsetAsync(c->d_err, 0, sizeof(h), s) != cudaSuccess) return AF_ERR_CUDA;
  if (cudaStreamSynchronize(s) != cudaSuccess) return AF_ERR_CUDA;
  if (flags) *flags = h;
  return h == 0 ? AF_OK : AF_ERR_DEVICE_FLAGGED;
}

static size_t pack_meta_bytes(int32_t B) {
  // [src_row int64 x B][cu int32 x (B+1)][idx int32 x B][chunk_cu int32 x (B+1)], each part
  // 16-byte aligned
  size_t a = ((size_t)B * 8 + 15) & ~(size_t)15;
  size_t b = ((size_t)(B + 1) * 4 + 15) & ~(size_t)15;
  size_t c = ((size_t)B * 4 + 15) & ~(size_t)15;
  return a + b + c + b + 16;
}

af_status af_reserve(af_ctx* c, int64_t max_T, int32_t max_B, int32_t d, int32_t V,
                     int32_t with_backward) {
  NvtxRange range("af_reserve");
  if (!c || max_T < 0 || max_B < 0 || d < 1 || V < 1) return AF_ERR_INVALID_ARG;
  if (max_T >= ((int64_t)1 << 31)) return AF_ERR_SHAPE;
  DeviceGuard guard(c->device);
  af_status st = AF_OK;
  if (max_T > 0) {
    const int S = logprob_pick_splits(max_T, d, V, c->sm_count, c->gemm_pair != 0, c->v_splits,
                                      c->gemm_pair && c->die_aware ? c->die0_sms / 2 : 0);
    // smaller batches may pick up to 8 ranges whatever their size, and more than 8 only while
    // there are at most 8 units per worker
    size_t need = (size_t)(S > 8 ? S : 8) * (size_t)max_T;
    size_t small = (size_t)c->sm_count * 8 * 128;
    if (need < small) need = small;
    st = ws_grow(c->partial, need * 16);
    if (st != AF_OK) return st;
  }
  st = ws_grow(c->pack_meta, pack_meta_bytes(max_B));
  if (st != AF_OK) return st;
  // af_grpo_advantage by group id: one accumulator per group, and a batch has at most one group per response
  st = ws_grow(c->adv_ws, advantage_ids_workspace_bytes(max_B));
  if (st != AF_OK) return st;
  if (with_backward) {
    // sizes are recomputed (and grown if needed) by the backward call itself
    st = launch_backward(c, nullptr, nullptr, nullptr, nullptr, nullptr, max_T, d, V, nullptr, nullptr,
                         -1 /* reserve only */, nullptr);
  }
  if (st == AF_OK && with_backward == 2) {
    af_loss_params none{};
    st = launch_policy_update(c, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, 0, max_T, d, V, none,
                              nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, -1 /* reserve only */,
                              nullptr);
  }
  return st;
}

// Fills the per-call sequence table from the host's offsets and index list: first store row, packed
// offset, sample index and first bulk-copy chunk of every sequence.  *T receives the token count as
// soon as it is known (also when the capacity check fails).
static af_status fill_sequence_table(const int64_t* tok_offset_host, int64_t n_samples, const int32_t* idx_host,
                                     int32_t B, int64_t rows_per_chunk, int64_t token_capacity, int64_t* h_src,
                                     int32_t* h_cu, int32_t* h_idx, int32_t* h_chunk, int64_t* T_out,
                                     int64_t* chunks_out) {
  const int64_t rpc = rows_per_chunk;
  int64_t T = 0, chunks = 0;
  h_cu[0] = 0;
  h_chunk[0] = 0;
  for (int32_t j = 0; j < B; ++j) {
    const int64_t i = idx_host[j];
    if (i < 0 || i >= n_samples) return AF_ERR_INDEX;
    const int64_t lo = tok_offset_host[i], hi = tok_offset_host[i + 1];
    if (hi < lo) return AF_ERR_INVALID_ARG;
    h_src[j] = lo;
    h_idx[j] = (int32_t)i;
    T += hi - lo;
    if (T >= ((int64_t)1 << 31)) return AF_ERR_CAPACITY;
    h_cu[j + 1] = (int32_t)T;
    if (rpc > 0) chunks += (hi - lo + rpc - 1) / rpc;
    h_chunk[j + 1] = (int32_t)chunks;   // chunks <= T + B < 2^31 + 2^31: checked below
    if (chunks >= ((int64_t)1 << 31)) return AF_ERR_CAPACITY;
  }
  if (T_out) *T_out = T;
  if (chunks_out) *chunks_out = chunks;
  return T > token_capacity ? AF_ERR_CAPACITY : AF_OK;
}

// Builds the table ([src_row][cu][idx][chunk_cu]) in a pinned staging slot and queues the kernel
// that brings it to the device.
static af_status stage_sequence_table(af_ctx* c, const int64_t* tok_offset_host, int64_t n_samples,
                                      const int32_t* idx_host, int32_t B, int64_t rows_per_chunk,
                                      int64_t token_capacity, PackSeqTable* tab, int64_t* T_out, cudaStream_t s) {
  // staging slot (pinned): wait until the copy that last used it has been consumed
  const int slot = c->pack_slot;
  c->pack_slot = (slot + 1) % kPackRing;
  if (c->pack_evt_live[slot] && cudaEventSynchronize(c->pack_evt[slot]) != cudaSuccess) return AF_ERR_CUDA;
  const size_t bytes = pack_meta_bytes(B);
  if (c->pack_host_cap[slot] < bytes) {
    if (c->pack_host[slot]) cudaFreeHost(c->pack_host[slot]);
    c->pack_host[slot] = nullptr; c->pack_host_cap[slot] = 0;
    size_t want = bytes < 4096 ? 4096 : bytes * 2;
    if (cudaMallocHost(&c->pack_host[slot], want) != cudaSuccess) { cudaGetLastError(); return AF_ERR_WORKSPACE; }
    c->pack_host_cap[slot] = want;
  }
  af_status st = ws_grow(c->pack_meta, bytes);
  if (st != AF_OK) return st;

  const size_t off_cu = ((size_t)B * 8 + 15) & ~(size_t)15;
  const size_t off_idx = off_cu + (((size_t)(B + 1) * 4 + 15) & ~(size_t)15);
  const size_t off_chunk = off_idx + (((size_t)B * 4 + 15) & ~(size_t)15);
  char* hb = static_cast<char*>(c->pack_host[slot]);
  int64_t chunks = 0;
  st = fill_sequence_table(tok_offset_host, n_samples, idx_host, B, rows_per_chunk, token_capacity,
                           reinterpret_cast<int64_t*>(hb), reinterpret_cast<int32_t*>(hb + off_cu),
                           reinterpret_cast<int32_t*>(hb + off_idx), reinterpret_cast<int32_t*>(hb + off_chunk), T_out,
                           &chunks);
  if (st != AF_OK) return st;

  char* db = static_cast<char*>(c->pack_meta.p);
  if (launch_pack_meta_fetch(db, hb, bytes, s) != cudaSuccess) return AF_ERR_CUDA;
  if (!c->pack_evt_live[slot]) {
    if (cudaEventCreateWithFlags(&c->pack_evt[slot], cudaEventDisableTiming) != cudaSuccess) return AF_ERR_CUDA;
    c->pack_evt_live[slot] = true;
  }
  if (cudaEventRecord(c->pack_evt[slot], s) != cudaSuccess) return AF_ERR_CUDA;
  *tab = PackSeqTable{reinterpret_cast<const int64_t*>(db), reinterpret_cast<const int32_t*>(db + off_cu),
                      reinterpret_cast<const int32_t*>(db + off_idx),
                      reinterpret_cast<const int32_t*>(db + off_chunk), (int)chunks};
  return AF_OK;
}

af_status af_pack_microbatch(af_ctx* c, const af_store_view* store, const int32_t* idx_host,
                             int32_t B, const af_packed* out, int64_t* T_out, void* stream) {
  NvtxRange range("af_pack_microbatch");
  if (!c || !store || !out || B < 0 || (B > 0 && !idx_host) || !store->tok_offset_host ||
      !out->cu_seqlens || store->n_samples < 0 || store->d < 1)
    return AF_ERR_INVALID_ARG;
  if ((store->hidden == nullptr) != (out->hidden == nullptr) ||
      (store->target == nullptr) != (out->target == nullptr) ||
      (store->old_logp == nullptr) != (out->old_logp == nullptr) ||
      (store->ref_logp == nullptr) != (out->ref_logp == nullptr) ||
      (store->adv == nullptr) != (out->adv_seq == nullptr))
    return AF_ERR_INVALID_ARG;
  if (store->hidden && (store->d % 8 != 0 || !aligned16(store->hidden) || !aligned16(out->hidden)))
    return AF_ERR_ALIGNMENT;
  if (B > out->seq_capacity) return AF_ERR_CAPACITY;
  DeviceGuard guard(c->device);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int rpc = store->hidden ? pack_rows_per_chunk(store->d) : 0;
  int64_t T = 0;
  if (B >= 1 && B <= kPackInlineSeqs && rpc > 0) {
    // few sequences: the table travels in the kernel's parameters, one launch does everything
    PackTableInline inl;
    int64_t chunks = 0;
    const af_status st = fill_sequence_table(store->tok_offset_host, store->n_samples, idx_host, B, rpc,
                                             out->token_capacity, inl.src_row, inl.cu, inl.idx, inl.chunk_cu, &T,
                                             &chunks);
    if (T_out) *T_out = T;
    if (st != AF_OK) return st;
    if (T > 0)
      return launch_pack_inline(*store, *out, inl, B, T, c->sm_count, c->d_err, s) == cudaSuccess ? AF_OK : AF_ERR_CUDA;
    // only empty sequences: the staged path below writes cu_seqlens and the advantages
  }
  PackSeqTable tab{};
  const af_status st = stage_sequence_table(c, store->tok_offset_host, store->n_samples, idx_host, B, rpc,
                                            out->token_capacity, &tab, &T, s);
  if (T_out) *T_out = T;
  if (st != AF_OK) return st;
  return launch_pack(*store, *out, tab, B, T, c->sm_count, c->d_err, s) == cudaSuccess ? AF_OK : AF_ERR_CUDA;
}

af_status af_unpack_microbatch(af_ctx* c, const int64_t* tok_offset_host, int64_t n_samples, const int32_t* idx_host,
                               int32_t B, const af_write_cols* cols, const af_controller_view* table,
                               uint32_t column_bits, int64_t* T_out, void* stream) {
  NvtxRange range("af_unpack_microbatch");
  if (!c || !tok_offset_host || n_samples < 0 || B < 0 || (B > 0 && !idx_host) || !cols || cols->n_cols < 0 ||
      cols->n_cols > AF_MAX_WRITE_COLS)
    return AF_ERR_INVALID_ARG;
  if (table && (table->n_samples != n_samples || (n_samples > 0 && !table->ready))) return AF_ERR_INVALID_ARG;
  // a sample may be listed once: two writers of one row would have no defined order
  try {
    std::vector<int32_t>& sorted = c->idx_scratch;     // the context's buffer: allocates only when it grows
    sorted.assign(idx_host, idx_host + B);
    std::sort(sorted.begin(), sorted.end());
    if (std::adjacent_find(sorted.begin(), sorted.end()) != sorted.end()) return AF_ERR_INVALID_ARG;
  } catch (...) {   // no exception may cross the C boundary (the copy of the list could not be allocated)
    return AF_ERR_WORKSPACE;
  }
  DeviceGuard guard(c->device);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  PackSeqTable tab{};
  int64_t T = 0;
  // sizes first (no pointer is touched): the columns may be NULL only if there is nothing to move
  for (int32_t j = 0; j < B; ++j) {
    const int64_t i = idx_host[j];
    if (i < 0 || i >= n_samples) return AF_ERR_INDEX;
    if (tok_offset_host[i + 1] > tok_offset_host[i])
      for (int k = 0; k < cols->n_cols; ++k)
        if (!cols->packed[k] || !cols->store[k]) return AF_ERR_INVALID_ARG;
  }
  const af_status st = stage_sequence_table(c, tok_offset_host, n_samples, idx_host, B, 0, INT64_MAX, &tab, &T, s);
  if (T_out) *T_out = T;
  if (st != AF_OK) return st;
  if (launch_unpack(*cols, tab, B, T, c->sm_count, s) != cudaSuccess) return AF_ERR_CUDA;
  // the status update that follows a write (Section 4.2): after the data, on the same stream
  if (table && column_bits && B > 0 &&
      launch_controller_put(*table, tab.idx, B, column_bits, c->d_err, c->sm_count, s) != cudaSuccess)
    return AF_ERR_CUDA;
  return AF_OK;
}

af_status af_token_logprob(af_ctx* c, const void* hidden, const void* W, const int32_t* target,
                           int64_t T, int32_t d, int32_t V, float* logp, float* entropy, float* lse,
                           void* stream) {
  NvtxRange range("af_token_logprob");
  if (!c || T < 0 || d < 1 || V < 1) return AF_ERR_INVALID_ARG;
  if (T == 0) return AF_OK;
  if (!hidden || !W || !target || !logp) return AF_ERR_INVALID_ARG;
  if (T >= ((int64_t)1 << 31)) return AF_ERR_SHAPE;
  if (d % 8 != 0 || !aligned16(hidden) || !aligned16(W)) return AF_ERR_ALIGNMENT;
  DeviceGuard guard(c->device);
  return launch_token_logprob(c, hidden, W, target, T, d, V, logp, entropy, lse,
                              static_cast<cudaStream_t>(stream));
}

af_status af_token_logprob_shard(af_ctx* c, const void* hidden, const void* W_shard, const int32_t* target,
                                 int64_t T, int32_t d, int32_t V_shard, int32_t v_offset, float* partial_out,
                                 void* stream) {
  NvtxRange range("af_token_logprob_shard");
  if (!c || T < 0 || d < 1 || V_shard < 1 || v_offset < 0) return AF_ERR_INVALID_ARG;
  if (T == 0) return AF_OK;
  if (!hidden || !W_shard || !target || !partial_out) return AF_ERR_INVALID_ARG;
  if (T >= ((int64_t)1 << 31)) return AF_ERR_SHAPE;
  if (d % 8 != 0 || !aligned16(hidden) || !aligned16(W_shard) || !aligned16(partial_out)) return AF_ERR_ALIGNMENT;
  DeviceGuard guard(c->device);
  return launch_token_logprob_shard(c, hidden, W_shard, target, T, d, V_shard, v_offset, partial_out,
                                    static_cast<cudaStream_t>(stream));
}

af_status af_merge_logprob_shards(af_ctx* c, const float* partials, const int32_t* target, int32_t R, int64_t T,
                                  int32_t V_total, float* logp, float* entropy, float* lse, void* stream) {
  NvtxRange range("af_merge_logprob_shards");
  if (!c || T < 0 || R < 1 || V_total < 1) return AF_ERR_INVALID_ARG;
  if (T == 0) return AF_OK;
  if (!partials || !target || !logp) return AF_ERR_INVALID_ARG;
  if (T >= ((int64_t)1 << 31)) return AF_ERR_SHAPE;
  if (!aligned16(partials)) return AF_ERR_ALIGNMENT;
  DeviceGuard guard(c->device);
  return launch_merge_logprob_shards(c, partials, target, R, T, V_total, logp, entropy, lse,
                                     static_cast<cudaStream_t>(stream));
}

af_status af_grpo_advantage(af_ctx* c, const float* reward, const int32_t* group_id, int64_t N,
                            int32_t n_groups, float eps_adv, int32_t ddof, float* adv, void* stream) {
  NvtxRange range("af_grpo_advantage");
  if (!c || N < 0 || n_groups < 0 || (ddof != 0 && ddof != 1) || !(eps_adv > 0.f)) return AF_ERR_INVALID_ARG;
  if (N == 0) return AF_OK;
  if (!reward || !adv || n_groups < 1) return AF_ERR_INVALID_ARG;
  if (!group_id && N % n_groups != 0) return AF_ERR_SHAPE;
  if (group_id && N >= ((int64_t)1 << 31)) return AF_ERR_SHAPE;       // member counts are 32-bit
  DeviceGuard guard(c->device);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (!group_id)
    return launch_advantage(reward, N, n_groups, eps_adv, ddof, adv, c->sm_count, s) == cudaSuccess ? AF_OK : AF_ERR_CUDA;
  const af_status st = ws_grow(c->adv_ws, advantage_ids_workspace_bytes(n_groups));
  if (st != AF_OK) return st;
  return launch_advantage_ids(reward, group_id, N, n_groups, eps_adv, ddof, adv, c->adv_ws.p, c->d_err, c->sm_count,
                              s) == cudaSuccess ? AF_OK : AF_ERR_CUDA;
}

af_status af_policy_loss(af_ctx* c, const float* logp, const float* old_logp, const float* ref_logp,
                         const float* entropy, const float* adv_seq, const int32_t* cu_seqlens,
                         int32_t B, int64_t T, const af_loss_params* params, af_loss_out* out,
                         float* dlogp, void* stream) {
  NvtxRange range("af_policy_loss");
  if (!c || !params || !out || !cu_seqlens || B < 0 || T < 0) return AF_ERR_INVALID_ARG;
  if (T > 0 && (!logp || !old_logp || !ref_logp || !adv_seq || B < 1)) return AF_ERR_INVALID_ARG;
  if (params->agg_mode != 0 && params->agg_mode != 1) return AF_ERR_INVALID_ARG;
  if (T > ((int64_t)1 << 31) - 65536) return AF_ERR_SHAPE;  // token indices are 32-bit in the kernel
  DeviceGuard guard(c->device);
  return launch_policy_loss(logp, old_logp, ref_logp, entropy, adv_seq, cu_seqlens, B, T, *params, out,
                            dlogp, c->loss_ws.p, c->d_err, c->sm_count,
                            static_cast<cudaStream_t>(stream)) == cudaSuccess ? AF_OK : AF_ERR_CUDA;
}

af_status af_policy_loss_backward(af_ctx* c, const void* hidden, const void* W, const int32_t* target,
                                  const float* lse, const float* dlogp, int64_t T, int32_t d, int32_t V,
                                  void* d_hidden, float* d_W, int32_t accumulate_dW, void* stream) {
  NvtxRange range("af_policy_loss_backward");
  if (!c || T < 0 || d < 1 || V < 1) return AF_ERR_INVALID_ARG;
  if (!hidden || !W || !target || !lse || !dlogp || !d_hidden || !d_W) {
    if (T > 0 || !d_W) return AF_ERR_INVALID_ARG;
  }
  if (T >= ((int64_t)1 << 31)) return AF_ERR_SHAPE;
  if (d % 8 != 0 || V % 8 != 0) return AF_ERR_ALIGNMENT;
  if (!aligned16(hidden) || !aligned16(W) || !aligned16(d_hidden) || !aligned16(d_W)) return AF_ERR_ALIGNMENT;
  DeviceGuard guard(c->device);
  return launch_backward(c, hidden, W, target, lse, dlogp, T, d, V, d_hidden, d_W,
                         accumulate_dW ? 1 : 0, static_cast<cudaStream_t>(stream));
}

af_status af_policy_loss_backward_shard(af_ctx* c, const void* hidden, const void* W_shard, const int32_t* target,
                                        const float* lse, const float* dlogp, int64_t T, int32_t d, int32_t V_shard,
                                        int32_t v_offset, void* d_hidden_partial, float* d_W_shard,
                                        int32_t accumulate_dW, void* stream) {
  NvtxRange range("af_policy_loss_backward_shard");
  if (!c || T < 0 || d < 1 || V_shard < 1 || v_offset < 0) return AF_ERR_INVALID_ARG;
  if (!hidden || !W_shard || !target || !lse || !dlogp || !d_hidden_partial || !d_W_shard) {
    if (T > 0 || !d_W_shard) return AF_ERR_INVALID_ARG;
  }
  if (T >= ((int64_t)1 << 31)) return AF_ERR_SHAPE;
  if (d % 8 != 0 || V_shard % 8 != 0) return AF_ERR_ALIGNMENT;
  if (!aligned16(hidden) || !aligned16(W_shard) || !aligned16(d_hidden_partial) || !aligned16(d_W_shard))
    return AF_ERR_ALIGNMENT;
  DeviceGuard guard(c->device);
  return launch_backward(c, hidden, W_shard, target, lse, dlogp, T, d, V_shard, d_hidden_partial, d_W_shard,
                         accumulate_dW ? 1 : 0, static_cast<cudaStream_t>(stream), v_offset);
}

static bool table_ok(const af_controller_view* t) {
  return t && t->n_samples >= 0 && (t->n_samples == 0 || (t->ready && t->consumed));
}

af_status af_policy_update(af_ctx* c, const void* hidden, const void* W, const int32_t* target,
                           const float* old_logp, const float* ref_logp, const float* adv_seq,
                           const int32_t* cu_seqlens, int32_t B, int64_t T, int32_t d, int32_t V,
                           const af_loss_params* params, af_loss_out* out, float* logp, float* entropy, float* lse,
                           float* dlogp, void* d_hidden, float* d_W, int32_t accumulate_dW, void* stream) {
  NvtxRange range("af_policy_update");
  if (!c || !params || !out || !cu_seqlens || B < 0 || T < 0 || d < 1 || V < 1 || !d_W) return AF_ERR_INVALID_ARG;
  if (T > 0 && (!hidden || !W || !target || !old_logp || !ref_logp || !adv_seq || !logp || !lse || !d_hidden || B < 1))
    return AF_ERR_INVALID_ARG;
  if (params->agg_mode != 0 && params->agg_mode != 1) return AF_ERR_INVALID_ARG;
  if (T > ((int64_t)1 << 31) - 65536) return AF_ERR_SHAPE;
  if (d % 8 != 0 || V % 8 != 0) return AF_ERR_ALIGNMENT;
  if (!aligned16(hidden) || !aligned16(W) || !aligned16(d_hidden) || !aligned16(d_W)) return AF_ERR_ALIGNMENT;
  DeviceGuard guard(c->device);
  return launch_policy_update(c, hidden, W, target, old_logp, ref_logp, adv_seq, cu_seqlens, B, T, d, V, *params, out,
                              logp, entropy, lse, dlogp, d_hidden, d_W, accumulate_dW ? 1 : 0,
                              static_cast<cudaStream_t>(stream));
}

af_status af_controller_put(af_ctx* c, const af_controller_view* table, const int32_t* idx, int64_t n,
                            uint32_t column_bits, void* stream) {
  NvtxRange range("af_controller_put");
  if (!c || !table_ok(table) || n < 0 || (n > 0 && !idx)) return AF_ERR_INVALID_ARG;
  if (table->n_samples >= ((int64_t)1 << 31)) return AF_ERR_SHAPE;
  DeviceGuard guard(c->device);
  return launch_controller_put(*table, idx, n, column_bits, c->d_err, c->sm_count,
                               static_cast<cudaStream_t>(stream)) == cudaSuccess ? AF_OK : AF_ERR_CUDA;
}

af_status af_controller_get(af_ctx* c, const af_controller_view* table, uint32_t column_mask, uint32_t task_bit,
                            int32_t max_samples, int64_t token_budget, int32_t* out_idx, af_get_result* out,
                            void* stream) {
  NvtxRange range("af_controller_get");
  if (!c || !table_ok(table) || !out || max_samples < 0 || (max_samples > 0 && !out_idx)) return AF_ERR_INVALID_ARG;
  if (task_bit == 0 || (task_bit & (task_bit - 1)) != 0) return AF_ERR_INVALID_ARG;
  if (token_budget > 0 && !table->length && table->n_samples > 0) return AF_ERR_INVALID_ARG;
  if (table->n_samples >= ((int64_t)1 << 31)) return AF_ERR_SHAPE;
  DeviceGuard guard(c->device);
  return launch_controller_get(*table, column_mask, task_bit, max_samples, token_budget, out_idx, out,
                               c->ctrl_ws.p, c->sm_count, static_cast<cudaStream_t>(stream)) == cudaSuccess
             ? AF_OK : AF_ERR_CUDA;
}

af_status af_controller_clear(af_ctx* c, const af_controller_view* table, uint32_t column_bits, uint32_t task_bits,
                              void* stream) {
  NvtxRange range("af_controller_clear");
  if (!c || !table_ok(table)) return AF_ERR_INVALID_ARG;
  DeviceGuard guard(c->device);
  return launch_controller_clear(*table, column_bits, task_bits, c->sm_count,
                                 static_cast<cudaStream_t>(stream)) == cudaSuccess ? AF_OK : AF_ERR_CUDA;
}

}  // extern "C"
