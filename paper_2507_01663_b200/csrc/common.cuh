// Shared host-side declarations of the asyncflow library: the context, workspace buffers and
// the internal launchers each .cu file provides to the C-ABI layer (api.cu).
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <vector>

#include "../../include/asyncflow.h"

namespace af {

constexpr int kPackRing = 8;  // pinned staging slots for af_pack_microbatch metadata
constexpr int kDeviceBlockBytes = 1024;  // the context's small device block: error word, tile clock, rank slots
constexpr int kTileClockWord = 16;  // word of that block used as the GEMM tile clock
constexpr int kDieCounterWord = 17;  // two words behind the clock: the per-die rank counters of a GEMM launch
constexpr int kDieTableByte = 512;   // 256 bytes of that block: die (0 / 1) of every SM id, measured at af_create

struct Buf {
  void* p = nullptr;
  size_t cap = 0;
};

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Tensor maps already encoded for this context, keyed by what determines them.  A map depends only
// on the address, shape, pitch and box of the matrix, not on the allocation behind it, so an entry
// stays valid for as long as the caller keeps passing the same buffer; the steady state of a
// training or scoring loop re-encodes nothing.
struct TmapCache {
  static constexpr int kEntries = 32;
  struct Entry {
    const void* base = nullptr;
    uint64_t rows = 0, cols = 0, pitch = 0;
    uint32_t box_rows = 0;
    CUtensorMap map;
  };
  Entry e[kEntries];
  int next = 0;      // round-robin replacement
};

// cudaFuncSetAttribute(MaxDynamicSharedMemorySize) once per kernel and device (the attribute is
// per device, and a process may drive several) instead of on every launch.
struct SmemAttrOnce {
  std::atomic<unsigned long long> done{0};   // bit i: set on device i (devices >= 64 set it every time)
};
template <class Kernel>
inline cudaError_t set_smem_once(SmemAttrOnce& once, Kernel kernel, int bytes) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const unsigned long long bit = dev < 64 ? 1ull << dev : 0ull;
  if (bit && (once.done.load(std::memory_order_acquire) & bit)) return cudaSuccess;
  e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess && bit) once.done.fetch_or(bit, std::memory_order_release);
  return e;
}

}  // namespace af

struct af_ctx {
  int device = 0;
  int sm_count = 0;
  af::EncodeTiledFn encode = nullptr;
  unsigned int* d_err = nullptr;  // kDeviceBlockBytes device block: word 0 = sticky error word, then clock and rank slots

  // tuning
  int v_splits = 0;         // 0 = automatic
  int bwd_token_block = 0;  // 0 = default
  int gemm_pair = 1;        // 1 = CTA-pair GEMM variant (the default), 0 = one CTA per tile
  int die_aware = 0;        // pair variant: deal row tiles to pairs by the die they run on
  int die0_sms = 0;         // SMs on the die of the first SM probed (0: the measurement was not clear-cut; no die-aware dealing)
  int die_map_reason = 0;   // why not, if so (see diemap.cu)
  cudaEvent_t dw_ready = nullptr;  // caller's event recorded once d_W is complete (af_set_dw_ready_event)

  af::TmapCache tmaps;      // tensor maps of the GEMM operands seen so far
  std::vector<int32_t> idx_scratch;  // host copy of an index list (duplicate check of the write-back); grows, never shrinks

  // workspace (device)
  af::Buf partial;    // [splits, T] float4 online-softmax partials
  af::Buf loss_ws;    // per-block partial sums + ticket of the loss reduction
  af::Buf pack_meta;  // per-call sequence table of af_pack_microbatch
  af::Buf dz;         // dZ [Tc, V] bf16 (backward, one token block)
  af::Buf ctrl_ws;    // per-block aggregates of af_controller_get
  af::Buf zlog;       // fp32 logits [Tc, V] of one token block (fused actor update)
  af::Buf adv_ws;     // per-group accumulators of af_grpo_advantage with group ids

  // pinned staging ring for pack metadata
  void* pack_host[af::kPackRing] = {};
  size_t pack_host_cap[af::kPackRing] = {};
  cudaEvent_t pack_evt[af::kPackRing] = {};
  bool pack_evt_live[af::kPackRing] = {};
  int pack_slot = 0;
};

namespace af {

af_status ws_grow(Buf& b, size_t bytes);

// Measures which SMs share a die (device table of 256 bytes indexed by SM id); false if unclear.
bool measure_die_map(int sm_count, unsigned char* d_table, int* die0_sms, int* reason);

// One warp waits (at most a millisecond) on a barrier nobody arrives at; sets AF_DEVERR_WATCHDOG.
cudaError_t launch_bounded_wait_selftest(unsigned int* d_err, unsigned int* waited_us, cudaStream_t s);

// ---- launchers (each returns the cudaGetLastError of its launches) --------------------------
struct PackSeqTable {     // device views into ctx->pack_meta for one call
  const int64_t* src_row; // [B] first store row of sequence j
  const int32_t* cu;      // [B+1]
  const int32_t* idx;     // [B]
  const int32_t* chunk_cu;// [B+1] first bulk-copy chunk of sequence j (hidden column)
  int n_chunks;           // chunk_cu[B]
};
// Copy `bytes` (rounded up to 16) from pinned, device-mapped host memory to the device with a kernel.
cudaError_t launch_pack_meta_fetch(void* dst_dev, const void* src_pinned, size_t bytes, cudaStream_t s);
// Rows of the hidden column per bulk-copy chunk for hidden size d (0: rows too wide, no chunks).
int pack_rows_per_chunk(int32_t d);
// Per-token 4-byte columns in packed order -> the store rows of their samples.
cudaError_t launch_unpack(const af_write_cols& cols, const PackSeqTable& tab, int32_t B, int64_t T, int sm_count,
                          cudaStream_t s);
cudaError_t launch_pack(const af_store_view& st, const af_packed& out, const PackSeqTable& tab,
                        int32_t B, int64_t T, int sm_count, unsigned int* d_err, cudaStream_t s);
// The same table for a micro-batch of at most kPackInlineSeqs sequences, small enough to travel in the
// kernel's parameters: no staging buffer, no fetch kernel, nothing for the host to wait on.
constexpr int kPackInlineSeqs = 512;
struct PackTableInline {
  int64_t src_row[kPackInlineSeqs];
  int32_t cu[kPackInlineSeqs + 1];
  int32_t idx[kPackInlineSeqs];
  int32_t chunk_cu[kPackInlineSeqs + 1];
};
// Packs with the table passed by value.  Needs hidden rows that fit a bulk-copy chunk, T > 0 and
// 1 <= B <= kPackInlineSeqs (the caller checks).
cudaError_t launch_pack_inline(const af_store_view& st, const af_packed& out, const PackTableInline& tab,
                               int32_t B, int64_t T, int sm_count, unsigned int* d_err, cudaStream_t s);

cudaError_t launch_advantage(const float* reward, int64_t N, int32_t n_groups, float eps_adv, int32_t ddof,
                             float* adv, int sm_count, cudaStream_t s);                  // contiguous groups
size_t advantage_ids_workspace_bytes(int32_t n_groups);
cudaError_t launch_advantage_ids(const float* reward, const int32_t* group_id, int64_t N, int32_t n_groups,
                                 float eps_adv, int32_t ddof, float* adv, void* ws, unsigned int* d_err,
                                 int sm_count, cudaStream_t s);                            // membership by id

size_t loss_workspace_bytes(int sm_count);
cudaError_t launch_policy_loss(const float* logp, const float* old_logp, const float* ref_logp,
                               const float* entropy, const float* adv_seq, const int32_t* cu,
                               int32_t B, int64_t T, const af_loss_params& p, af_loss_out* out,
                               float* dlogp, void* ws, unsigned int* d_err, int sm_count,
                               cudaStream_t s);

size_t controller_workspace_bytes(int sm_count);
cudaError_t launch_controller_put(const af_controller_view& v, const int32_t* idx, int64_t n, uint32_t bits,
                                  unsigned int* d_err, int sm_count, cudaStream_t s);
cudaError_t launch_controller_clear(const af_controller_view& v, uint32_t column_bits, uint32_t task_bits,
                                    int sm_count, cudaStream_t s);
cudaError_t launch_controller_get(const af_controller_view& v, uint32_t mask, uint32_t task_bit, int32_t max_samples,
                                  int64_t token_budget, int32_t* out_idx, af_get_result* out, void* ws,
                                  int sm_count, cudaStream_t s);

int logprob_pick_splits(int64_t T, int32_t d, int32_t V, int sm_count, bool pair, int requested, int die0_pairs);
// The work decomposition launch_token_logprob would use (no device needed); see af_plan_token_logprob.
void plan_token_logprob(int64_t T, int32_t d, int32_t V, int sm_count, int die0_sms, int requested_splits, bool pair,
                        bool die_aware, af_gemm_plan* plan);
void plan_units(const af_gemm_plan& plan, int rank, int* first, int* stride, int* end);
af_status launch_token_logprob(af_ctx* ctx, const void* hidden, const void* W,
                               const int32_t* target, int64_t T, int32_t d, int32_t V,
                               float* logp, float* entropy, float* lse, cudaStream_t s);

af_status launch_token_logprob_shard(af_ctx* ctx, const void* hidden, const void* W_shard,
                                     const int32_t* target, int64_t T, int32_t d, int32_t V_shard,
                                     int32_t v_offset, float* partial_out, cudaStream_t s);
af_status launch_merge_logprob_shards(af_ctx* ctx, const float* partials, const int32_t* target, int32_t R,
                                      int64_t T, int32_t V_total, float* logp, float* entropy, float* lse,
                                      cudaStream_t s);

af_status launch_token_logprob_z(af_ctx* ctx, const void* hidden, const void* W,
                                 const int32_t* target, int64_t T, int32_t d, int32_t V,
                                 float* logp, float* entropy, float* lse, float* z, cudaStream_t s);
int64_t backward_token_block(const af_ctx* ctx, int64_t T);
af_status launch_backward_products(af_ctx* ctx, const void* hidden_blk, const void* W, const void* dz_blk,
                                   int64_t tc, int32_t d, int32_t V, void* d_hidden_blk, float* d_W,
                                   int32_t accumulate_dW, bool last_block, cudaStream_t s);
af_status launch_policy_update(af_ctx* ctx, const void* hidden, const void* W, const int32_t* target,
                               const float* old_logp, const float* ref_logp, const float* adv_seq,
                               const int32_t* cu_seqlens, int32_t B, int64_t T, int32_t d, int32_t V,
                               const af_loss_params& params, af_loss_out* out, float* logp, float* entropy,
                               float* lse, float* dlogp, void* d_hidden, float* d_W, int32_t accumulate_dW,
                               cudaStream_t s);

af_status launch_backward(af_ctx* ctx, const void* hidden, const void* W, const int32_t* target,
                          const float* lse, const float* dlogp, int64_t T, int32_t d, int32_t V,
                          void* d_hidden, float* d_W, int32_t accumulate_dW, cudaStream_t s,
                          int32_t v_offset = 0);

}  // namespace af
