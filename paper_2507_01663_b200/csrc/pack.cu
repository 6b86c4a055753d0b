// af_pack_microbatch kernels: gather the token rows of the indexed samples into cu_seqlens-packed
// tensors.  Pure data movement (HBM-bound): every payload byte is read once and written once,
// untouched, so the result is bit-exact by construction.
//
// Layout: sample idx[j] owns the contiguous store rows src_row[j] .. src_row[j]+len-1 and the
// packed rows cu[j] .. cu[j+1]-1, so the hidden column of a sequence is ONE contiguous byte range
// on both sides.  It is cut into chunks of whole rows (at most kChunkBytes) and every chunk moves
// with two bulk-copy (TMA) instructions, global -> shared -> global, issued by a single thread
// per CTA through a ring of shared-memory stages: no payload byte passes through a register, and
// the number of bytes in flight does not depend on how many threads are resident.  Rows wider
// than a chunk fall back to a warp-per-row copy with 128-bit loads and stores.  The 4-byte
// columns are gathered one thread per token, by the other warps of the same CTAs (a kernel of its
// own only on the fallback path).
#include <cstring>

#include "common.cuh"
#include "device_util.cuh"
#include "umma.cuh"

namespace af {
namespace {

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
__device__ __forceinline__ void st_stream(uint4* p, const uint4& v) {
  asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};"
               :: "l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

constexpr int kRowUnroll = 8;

// One warp per packed row, grid-stride.  words = d / 8 (16-byte words per row).
__global__ void __launch_bounds__(256) pack_rows_kernel(const uint4* __restrict__ src,
                                                        uint4* __restrict__ dst,
                                                        const int64_t* __restrict__ src_row,
                                                        const int32_t* __restrict__ cu, int B,
                                                        int T, int words) {
  const int lane = threadIdx.x & 31;
  const int warps_per_block = blockDim.x >> 5;
  const int64_t warp0 = (int64_t)blockIdx.x * warps_per_block + (threadIdx.x >> 5);
  const int64_t nwarps = (int64_t)gridDim.x * warps_per_block;
  for (int64_t t = warp0; t < T; t += nwarps) {
    const int j = find_seq(cu, B, (int)t);
    const int64_t srow = __ldg(src_row + j) + (t - __ldg(cu + j));
    const uint4* s = src + srow * words;
    uint4* o = dst + t * (int64_t)words;
    for (int w = lane; w < words; w += 32 * kRowUnroll) {   // all loads of a batch before its stores
      uint4 v[kRowUnroll];
#pragma unroll
      for (int u = 0; u < kRowUnroll; ++u) if (w + 32 * u < words) v[u] = ld_stream(s + w + 32 * u);
#pragma unroll
      for (int u = 0; u < kRowUnroll; ++u) if (w + 32 * u < words) st_stream(o + w + 32 * u, v[u]);
    }
  }
}

// ---- bulk-copy (TMA) path ---------------------------------------------------------------------
constexpr int kChunkBytes = 32768;      // most bytes per bulk copy (whole rows)
constexpr int kCopyStages = 6;          // shared-memory ring: 6 x 32 KB
constexpr int kCopyAhead = 4;           // loads in flight ahead of the store being issued
constexpr int kCopySmemBytes = kCopyStages * kChunkBytes + 128 /*alignment*/ + 64 /*barriers*/;

__device__ __forceinline__ void bulk_load(uint32_t dst_smem, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               :: "r"(dst_smem), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void bulk_store(void* dst, uint32_t src_smem, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
               :: "l"(dst), "r"(src_smem), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int kPending>
__device__ __forceinline__ void bulk_wait_read() {   // at most kPending stores still reading shared memory
  asm volatile("cp.async.bulk.wait_group.read %0;" :: "n"(kPending) : "memory");
}
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// Sequence of a packed token (see find_seq) by plain loads: the table may sit in shared memory.
__device__ __forceinline__ int seq_of(const int32_t* cu, int B, int t) {
  int lo = 0, hi = B;
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (cu[mid] <= t) lo = mid; else hi = mid;
  }
  return lo;
}

// Walks the chunks of consecutive sequences: sequence j owns chunks chunk_cu[j] .. chunk_cu[j+1]-1,
// each `rows_per_chunk` rows except the last one of the sequence.  (Plain loads: global or shared table.)
struct ChunkCursor {
  const int64_t* src_row; const int32_t* cu; const int32_t* chunk_cu;
  int B, rows_per_chunk;
  int j, first_chunk, next_first, dst_row0, len;
  int64_t src_row0;
  __device__ void seek(int c) {   // largest j with chunk_cu[j] <= c (sequences without rows own no chunk)
    j = seq_of(chunk_cu, B, c);
    load();
  }
  __device__ void load() {
    first_chunk = chunk_cu[j];
    next_first = chunk_cu[j + 1];
    dst_row0 = cu[j];
    len = cu[j + 1] - dst_row0;
    src_row0 = src_row[j];
  }
  // source row, packed row and row count of chunk c (c never decreases between calls)
  __device__ void at(int c, int64_t& srow, int64_t& drow, int& rows) {
    while (c >= next_first && j + 1 < B) { ++j; load(); }
    const int r0 = (c - first_chunk) * rows_per_chunk;
    rows = len - r0 < rows_per_chunk ? len - r0 : rows_per_chunk;
    srow = src_row0 + r0;
    drow = (int64_t)dst_row0 + r0;
  }
};

// The 4-byte columns of a packed micro-batch and what their gather needs of the sequence table.
struct PackCols {
  const int32_t* s_target; const float* s_old; const float* s_ref; const float* s_adv;
  int32_t* o_target; float* o_old; float* o_ref; float* o_adv; int32_t* o_seq; int32_t* o_cu;
  const int64_t* src_row; const int32_t* cu; const int32_t* idx;
  int B, T;
};
// Items first, first + stride, ...: item i is packed token i (its columns and sequence id), and for
// i <= B also cu_seqlens[i] and the advantage of sequence i.
__device__ __forceinline__ void gather_cols(const PackCols& c, int64_t first, int64_t stride) {
  for (int64_t i = first; i < c.T || i <= c.B; i += stride) {
    if (i <= c.B) c.o_cu[i] = c.cu[i];
    if (i < c.B && c.o_adv) c.o_adv[i] = __ldg(c.s_adv + c.idx[i]);
    if (i < c.T) {
      const int j = seq_of(c.cu, c.B, (int)i);
      const int64_t srow = c.src_row[j] + (i - c.cu[j]);
      if (c.o_target) c.o_target[i] = __ldg(c.s_target + srow);
      if (c.o_old) c.o_old[i] = __ldg(c.s_old + srow);
      if (c.o_ref) c.o_ref[i] = __ldg(c.s_ref + srow);
      if (c.o_seq) c.o_seq[i] = j;
    }
  }
}

// One CTA per SM.  Its first thread moves the contiguous chunk range
// [n_chunks b / grid, n_chunks (b+1) / grid) of the hidden column through the ring; warps 1 .. 7
// meanwhile gather the 4-byte columns (grid-stride over the tokens), so that a micro-batch is packed
// by one launch and the small columns cost no launch or drain of their own.
constexpr int kBulkThreads = 256;
__device__ __forceinline__ void pack_bulk_body(
    const uint8_t* __restrict__ src, uint8_t* __restrict__ dst, const int64_t* src_row, const int32_t* cu,
    const int32_t* chunk_cu, int B, int n_chunks, int rows_per_chunk, int row_bytes, unsigned int* d_err,
    const PackCols& cols, uint8_t* smem_raw, int* abort_flag) {
  if (threadIdx.x >= 32) {
    constexpr int kColThreads = kBulkThreads - 32;
    gather_cols(cols, (int64_t)blockIdx.x * kColThreads + (threadIdx.x - 32), (int64_t)gridDim.x * kColThreads);
    return;
  }
  if (threadIdx.x != 0) return;
  const uint32_t raw = umma::smem_u32(smem_raw);
  const uint32_t ring = (raw + 127u) & ~127u;
  const uint32_t bars = ring + kCopyStages * kChunkBytes;
  *abort_flag = 0;
  for (int s = 0; s < kCopyStages; ++s) umma::mbar_init(bars + 8u * s, 1);
  umma::fence_mbar_init();

  const int c_begin = (int)(((int64_t)n_chunks * blockIdx.x) / gridDim.x);
  const int c_end = (int)(((int64_t)n_chunks * (blockIdx.x + 1)) / gridDim.x);
  const int n = c_end - c_begin;
  if (n <= 0) return;

  ChunkCursor lc{src_row, cu, chunk_cu, B, rows_per_chunk};   // cursor of the loads
  ChunkCursor sc = lc;                                         // cursor of the stores
  lc.seek(c_begin);
  sc.seek(c_begin);
  auto issue_load = [&](int i) {
    int64_t srow, drow; int rows;
    lc.at(c_begin + i, srow, drow, rows);
    const int st = i % kCopyStages;
    const uint32_t bytes = (uint32_t)rows * (uint32_t)row_bytes;
    umma::mbar_arrive_expect_tx(bars + 8u * st, bytes);
    bulk_load(ring + st * kChunkBytes, src + srow * row_bytes, bytes, bars + 8u * st);
  };
  for (int i = 0; i < kCopyAhead && i < n; ++i) issue_load(i);
  for (int i = 0; i < n; ++i) {
    const int st = i % kCopyStages;
    if (!umma::mbar_wait(bars + 8u * st, (uint32_t)(i / kCopyStages) & 1u, abort_flag)) break;
    int64_t srow, drow; int rows;
    sc.at(c_begin + i, srow, drow, rows);
    bulk_store(dst + drow * row_bytes, ring + st * kChunkBytes, (uint32_t)rows * (uint32_t)row_bytes);
    bulk_commit();
    if (i + kCopyAhead < n) {
      // the stage of load i + kCopyAhead was last read by store i + kCopyAhead - kCopyStages
      bulk_wait_read<kCopyStages - kCopyAhead>();
      issue_load(i + kCopyAhead);
    }
  }
  bulk_wait_all();
  if (*abort_flag) atomicOr(d_err, umma::kWatchdogBit);
}

__global__ void __launch_bounds__(kBulkThreads, 1) pack_rows_bulk_kernel(
    const uint8_t* __restrict__ src, uint8_t* __restrict__ dst, const int64_t* __restrict__ src_row,
    const int32_t* __restrict__ cu, const int32_t* __restrict__ chunk_cu, int B, int n_chunks,
    int rows_per_chunk, int row_bytes, unsigned int* d_err, const PackCols cols) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ int abort_flag;
  pack_bulk_body(src, dst, src_row, cu, chunk_cu, B, n_chunks, rows_per_chunk, row_bytes, d_err, cols, smem_raw,
                 &abort_flag);
}

// The same with the sequence table in the kernel's parameters (B <= kSeqs): every CTA copies the B
// entries it needs into shared memory and works from there.  Two sizes: parameters beyond 4 KB make
// a launch noticeably slower on the host, so small batches use a table that stays below that.
template <int kSeqs>
struct InlineTable {
  int64_t src_row[kSeqs];
  int32_t cu[kSeqs + 1];
  int32_t idx[kSeqs];
  int32_t chunk_cu[kSeqs + 1];
};
constexpr int kSmallInlineSeqs = 128;
static_assert(sizeof(InlineTable<kSmallInlineSeqs>) + 256 <= 4096, "the small table keeps the launch within 4 KB of parameters");

template <int kSeqs>
__global__ void __launch_bounds__(kBulkThreads, 1) pack_rows_bulk_inline_kernel(
    const uint8_t* __restrict__ src, uint8_t* __restrict__ dst, const __grid_constant__ InlineTable<kSeqs> tab, int B,
    int n_chunks, int rows_per_chunk, int row_bytes, unsigned int* d_err, const PackCols cols_in) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ int abort_flag;
  __shared__ int64_t s_src_row[kSeqs];
  __shared__ int32_t s_cu[kSeqs + 1], s_idx[kSeqs], s_chunk_cu[kSeqs + 1];
  for (int i = threadIdx.x; i <= B; i += kBulkThreads) {
    s_cu[i] = tab.cu[i];
    s_chunk_cu[i] = tab.chunk_cu[i];
    if (i < B) { s_src_row[i] = tab.src_row[i]; s_idx[i] = tab.idx[i]; }
  }
  __syncthreads();
  PackCols cols = cols_in;
  cols.src_row = s_src_row; cols.cu = s_cu; cols.idx = s_idx;
  pack_bulk_body(src, dst, s_src_row, s_cu, s_chunk_cu, B, n_chunks, rows_per_chunk, row_bytes, d_err, cols,
                 smem_raw, &abort_flag);
}

// One thread per packed token for the 4-byte columns; the first B threads also gather adv.
__global__ void __launch_bounds__(256) pack_cols_kernel(const PackCols c) {
  gather_cols(c, (int64_t)blockIdx.x * blockDim.x + threadIdx.x, (int64_t)gridDim.x * blockDim.x);
}

// The inverse for results: one thread per packed token writes up to four 4-byte columns to the
// store rows of the token's sample.
struct UnpackCols {
  const uint32_t* packed[AF_MAX_WRITE_COLS];
  uint32_t* store[AF_MAX_WRITE_COLS];
  int n;
};
__global__ void __launch_bounds__(256) unpack_cols_kernel(UnpackCols c, const int64_t* __restrict__ src_row,
                                                         const int32_t* __restrict__ cu, int B, int T) {
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < T; i += stride) {
    const int j = find_seq(cu, B, (int)i);
    const int64_t row = __ldg(src_row + j) + (i - __ldg(cu + j));
#pragma unroll
    for (int k = 0; k < AF_MAX_WRITE_COLS; ++k)
      if (k < c.n) c.store[k][row] = __ldg(c.packed[k] + i);
  }
}

}  // namespace

cudaError_t launch_unpack(const af_write_cols& cols, const PackSeqTable& tab, int32_t B, int64_t T, int sm_count,
                          cudaStream_t s) {
  if (T == 0 || cols.n_cols == 0) return cudaSuccess;
  UnpackCols c{};
  c.n = cols.n_cols;
  for (int k = 0; k < cols.n_cols; ++k) {
    c.packed[k] = static_cast<const uint32_t*>(cols.packed[k]);
    c.store[k] = static_cast<uint32_t*>(cols.store[k]);
  }
  int64_t blocks = (T + 255) / 256;
  if (blocks > (int64_t)sm_count * 8) blocks = (int64_t)sm_count * 8;
  unpack_cols_kernel<<<(int)blocks, 256, 0, s>>>(c, tab.src_row, tab.cu, B, (int)T);
  return cudaGetLastError();
}

// Brings the per-call sequence table from pinned host memory to the device with a kernel (the
// pinned buffer is mapped into the device's address space) instead of a host-to-device memcpy:
// a memcpy would queue on the copy engine, behind whatever bulk transfers the application has in
// flight (weights, the next batch of the store), and stall the whole micro-batch behind them.
namespace {
__global__ void __launch_bounds__(256) pack_meta_fetch_kernel(uint4* __restrict__ dst,
                                                             const uint4* __restrict__ src_pinned, int n_words) {
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n_words; i += gridDim.x * blockDim.x) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(src_pinned + i));
    dst[i] = v;
  }
}
}  // namespace

cudaError_t launch_pack_meta_fetch(void* dst_dev, const void* src_pinned, size_t bytes, cudaStream_t s) {
  const int n_words = (int)((bytes + 15) / 16);
  if (n_words == 0) return cudaSuccess;
  int blocks = (n_words + 255) / 256;
  if (blocks > 64) blocks = 64;
  pack_meta_fetch_kernel<<<blocks, 256, 0, s>>>(static_cast<uint4*>(dst_dev), static_cast<const uint4*>(src_pinned), n_words);
  return cudaGetLastError();
}

int pack_rows_per_chunk(int32_t d) {
  const int64_t row_bytes = (int64_t)d * 2;
  return row_bytes <= kChunkBytes ? (int)(kChunkBytes / row_bytes) : 0;
}

cudaError_t launch_pack(const af_store_view& st, const af_packed& out, const PackSeqTable& tab,
                        int32_t B, int64_t T, int sm_count, unsigned int* d_err, cudaStream_t s) {
  const PackCols cols{st.target, st.old_logp, st.ref_logp, st.adv, out.target, out.old_logp, out.ref_logp,
                      out.adv_seq, out.seq_id, out.cu_seqlens, tab.src_row, tab.cu, tab.idx, B, (int)T};
  const int rpc = pack_rows_per_chunk(st.d);
  if (T > 0 && out.hidden && rpc > 0 && tab.n_chunks > 0) {
    // the usual case: one launch moves the hidden rows and gathers the small columns
    static SmemAttrOnce once;
    cudaError_t e = set_smem_once(once, pack_rows_bulk_kernel, kCopySmemBytes);
    if (e != cudaSuccess) return e;
    const int grid = tab.n_chunks < sm_count ? tab.n_chunks : sm_count;
    pack_rows_bulk_kernel<<<grid, kBulkThreads, kCopySmemBytes, s>>>(
        (const uint8_t*)st.hidden, (uint8_t*)out.hidden, tab.src_row, tab.cu, tab.chunk_cu, B,
        tab.n_chunks, rpc, st.d * 2, d_err, cols);
    return cudaGetLastError();
  }
  {
    int64_t items = T > (int64_t)B + 1 ? T : (int64_t)B + 1;
    int blocks = (int)((items + 255) / 256);
    if (blocks > sm_count * 8) blocks = sm_count * 8;
    pack_cols_kernel<<<blocks, 256, 0, s>>>(cols);
  }
  if (T > 0 && out.hidden) {   // rows wider than a chunk
    const int words = st.d / 8;
    int64_t blocks = (T + 7) / 8;  // 8 warps per block
    if (blocks > sm_count * 8) blocks = sm_count * 8;
    pack_rows_kernel<<<(int)blocks, 256, 0, s>>>((const uint4*)st.hidden, (uint4*)out.hidden,
                                                 tab.src_row, tab.cu, B, (int)T, words);
  }
  return cudaGetLastError();
}

namespace {
template <int kSeqs>
cudaError_t launch_inline(const af_store_view& st, const af_packed& out, const PackTableInline& full, int32_t B,
                          const PackCols& cols, int sm_count, unsigned int* d_err, cudaStream_t s) {
  static SmemAttrOnce once;
  cudaError_t e = set_smem_once(once, pack_rows_bulk_inline_kernel<kSeqs>, kCopySmemBytes);
  if (e != cudaSuccess) return e;
  InlineTable<kSeqs> tab;
  std::memcpy(tab.src_row, full.src_row, sizeof(int64_t) * B);
  std::memcpy(tab.cu, full.cu, sizeof(int32_t) * (B + 1));
  std::memcpy(tab.idx, full.idx, sizeof(int32_t) * B);
  std::memcpy(tab.chunk_cu, full.chunk_cu, sizeof(int32_t) * (B + 1));
  const int n_chunks = full.chunk_cu[B];
  const int grid = n_chunks < sm_count ? n_chunks : sm_count;
  pack_rows_bulk_inline_kernel<kSeqs><<<grid, kBulkThreads, kCopySmemBytes, s>>>(
      (const uint8_t*)st.hidden, (uint8_t*)out.hidden, tab, B, n_chunks, pack_rows_per_chunk(st.d), st.d * 2, d_err,
      cols);
  return cudaGetLastError();
}
}  // namespace

cudaError_t launch_pack_inline(const af_store_view& st, const af_packed& out, const PackTableInline& tab,
                               int32_t B, int64_t T, int sm_count, unsigned int* d_err, cudaStream_t s) {
  const PackCols cols{st.target, st.old_logp, st.ref_logp, st.adv, out.target, out.old_logp, out.ref_logp,
                      out.adv_seq, out.seq_id, out.cu_seqlens, nullptr, nullptr, nullptr, B, (int)T};
  return B <= kSmallInlineSeqs ? launch_inline<kSmallInlineSeqs>(st, out, tab, B, cols, sm_count, d_err, s)
                               : launch_inline<kPackInlineSeqs>(st, out, tab, B, cols, sm_count, d_err, s);
}

}  // namespace af
