// af_pack_microbatch kernels: gather the token rows of the indexed samples into cu_seqlens-packed
// tensors.  Pure data movement (HBM-bound): every payload byte is read once and written once,
// as 16-byte words, so the result is bit-exact by construction.
//
// Layout: sample idx[j] owns the contiguous store rows src_row[j] .. src_row[j]+len-1, and the
// packed rows cu[j] .. cu[j+1]-1.  A warp copies one token row (d*2 bytes) at a time; its
// sequence is found by a binary search over cu (B+1 ints, L1/L2 resident).
#include "common.cuh"

namespace af {
namespace {

__device__ __forceinline__ int find_seq(const int32_t* __restrict__ cu, int B, int t) {
  // largest j in [0, B) with cu[j] <= t  (cu is non-decreasing, cu[0] = 0, t < cu[B])
  int lo = 0, hi = B;
  while (hi - lo > 1) {
    int mid = (lo + hi) >> 1;
    if (__ldg(cu + mid) <= t) lo = mid; else hi = mid;
  }
  return lo;
}

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
    int w = lane;
    for (; w + 32 * (kRowUnroll - 1) < words; w += 32 * kRowUnroll) {
      uint4 v[kRowUnroll];
#pragma unroll
      for (int u = 0; u < kRowUnroll; ++u) v[u] = ld_stream(s + w + 32 * u);
#pragma unroll
      for (int u = 0; u < kRowUnroll; ++u) st_stream(o + w + 32 * u, v[u]);
    }
    for (; w < words; w += 32) st_stream(o + w, ld_stream(s + w));
  }
}

// One thread per packed token for the 4-byte columns; the first B threads also gather adv.
__global__ void __launch_bounds__(256) pack_cols_kernel(
    const int32_t* __restrict__ s_target, const float* __restrict__ s_old,
    const float* __restrict__ s_ref, const float* __restrict__ s_adv,
    int32_t* __restrict__ o_target, float* __restrict__ o_old, float* __restrict__ o_ref,
    float* __restrict__ o_adv, int32_t* __restrict__ o_seq, int32_t* __restrict__ o_cu,
    const int64_t* __restrict__ src_row, const int32_t* __restrict__ cu,
    const int32_t* __restrict__ idx, int B, int T) {
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < T || i <= B; i += stride) {
    if (i <= B) o_cu[i] = __ldg(cu + i);
    if (i < B && o_adv) o_adv[i] = __ldg(s_adv + __ldg(idx + i));
    if (i < T) {
      const int j = find_seq(cu, B, (int)i);
      const int64_t srow = __ldg(src_row + j) + (i - __ldg(cu + j));
      if (o_target) o_target[i] = __ldg(s_target + srow);
      if (o_old) o_old[i] = __ldg(s_old + srow);
      if (o_ref) o_ref[i] = __ldg(s_ref + srow);
      if (o_seq) o_seq[i] = j;
    }
  }
}

}  // namespace

cudaError_t launch_pack(const af_store_view& st, const af_packed& out, const PackSeqTable& tab,
                        int32_t B, int64_t T, int sm_count, cudaStream_t s) {
  {
    int64_t items = T > (int64_t)B + 1 ? T : (int64_t)B + 1;
    int blocks = (int)((items + 255) / 256);
    if (blocks > sm_count * 8) blocks = sm_count * 8;
    pack_cols_kernel<<<blocks, 256, 0, s>>>(st.target, st.old_logp, st.ref_logp, st.adv,
                                            out.target, out.old_logp, out.ref_logp, out.adv_seq,
                                            out.seq_id, out.cu_seqlens, tab.src_row, tab.cu,
                                            tab.idx, B, (int)T);
  }
  if (T > 0 && out.hidden) {
    const int words = st.d / 8;
    int64_t blocks = (T + 7) / 8;  // 8 warps per block
    if (blocks > sm_count * 8) blocks = sm_count * 8;
    pack_rows_kernel<<<(int)blocks, 256, 0, s>>>((const uint4*)st.hidden, (uint4*)out.hidden,
                                                 tab.src_row, tab.cu, B, (int)T, words);
  }
  return cudaGetLastError();
}

}  // namespace af
