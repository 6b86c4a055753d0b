// af_policy_loss kernel: clipped-ratio GRPO policy loss + k3 KL penalty, forward and dL/dlogp,
// in one pass over the packed tokens (12-16 B read, 4 B written per token: HBM-bound).
//
// A CTA owns a contiguous range of 2048-token chunks.  One thread feeds a ring of shared-memory
// stages with bulk copies (TMA) of the chunk's logp / old / ref / entropy slices, up to three
// chunks ahead, so the bytes in flight do not depend on how many threads are resident; each thread then
// reads two groups of 4 consecutive tokens (128 tokens apart, so that a warp's 128-bit accesses stay
// contiguous) from shared memory with one 128-bit load per group and column.  At full bandwidth the
// kernel runs at the SM's instruction-issue limit, so the work per thread that does not depend on
// the token count (sequence lookup, barrier waits, loop control) is spread over 8 tokens.  Warps run
// free of one another inside the chunk loop: a "full" mbarrier per stage announces the data, an
// "empty" mbarrier per stage (one arrival per warp) tells the feeding thread when the stage can
// be refilled -- there is no block-wide barrier per chunk.
//
// The cu_seqlens entries (and advantages) of the sequences the CTA's tokens belong to are staged
// in a shared-memory window, normally once per CTA; a thread finds its sequence by galloping
// forward from where it was in the previous chunk.  The window is re-staged when a chunk runs
// past it; a chunk that touches more sequences than a window holds (piles of empty sequences)
// searches cu_seqlens in global memory instead.  Tokens of one sequence are contiguous, so a
// thread sums its tokens run by run and scales each run by 1/L_i once (the per-sequence mean of
// agg_mode 0); runs are combined with warp shuffles, per-block sums go to the workspace in fp64
// and the last block to finish adds them in a fixed order -- no float atomics, so results are
// bit-reproducible.  Buffers that are not 16-byte aligned, and the last 1-3 tokens of a batch
// whose length is not a multiple of 4, are read with plain loads instead.
#include "loss_math.cuh"
#include "umma.cuh"

namespace af {
namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kGroup = 4;                                 // consecutive tokens per 128-bit access
constexpr int kGroups = 2;                                // such groups per thread, 128 tokens apart
constexpr int kTokPerThread = kGroup * kGroups;
constexpr int kWarpTokens = 32 * kTokPerThread;           // a warp owns 256 consecutive tokens of a chunk
constexpr int kChunk = kThreads * kTokPerThread;          // tokens per chunk = per ring stage
constexpr int kStages = 3;                                // ring depth: up to 3 chunks in flight
constexpr int kColBytes = kChunk * 4;                     // one column slice of a stage
constexpr int kStageBytes = 4 * kColBytes;                // logp | old | ref | entropy
constexpr int kRingSmemBytes = kStages * kStageBytes + 128 /*alignment*/ + 64 /*barriers*/;
constexpr int kNumSums = 4;  // pg, k3, entropy, clipped count
constexpr int kWindow = 1025;  // cu_seqlens entries staged at a time (1024 sequences)

struct LossWs {            // 64-byte header, then double partial[blocks][kNumSums]
  unsigned int ticket;
  unsigned int pad[15];
};
__device__ __forceinline__ double* ws_partial(LossWs* ws, int block) {
  return reinterpret_cast<double*>(ws + 1) + (size_t)block * kNumSums;
}


__device__ __forceinline__ void bulk_load(uint32_t dst_smem, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               :: "r"(dst_smem), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ float4 lds128(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
  return v;
}


// The same search done by one warp, 32 probes per step (2 steps for B = 512, 4 for B = 10^6).
__device__ __forceinline__ int find_seq_warp(const int32_t* __restrict__ cu, int B, int t, int lane) {
  int lo = 0, hi = B;  // invariant: cu[lo] <= t < cu[hi]
  while (hi - lo > 1) {
    const int span = hi - lo;
    const int step = (span + 31) / 32;
    const int probe = lo + (lane + 1) * step;  // probes lo+step, lo+2 step, ...
    const bool le = probe < hi && __ldg(cu + probe) <= t;
    const unsigned m = __ballot_sync(0xffffffffu, le);
    const int k = __popc(m);                   // probes are ordered, so the set bits are a prefix
    const int nlo = lo + k * step;
    const int nhi = nlo + step < hi ? nlo + step : hi;
    lo = nlo; hi = nhi;
  }
  return lo;
}

__global__ void __launch_bounds__(kThreads, 2) policy_loss_kernel(
    const float* __restrict__ logp, const float* __restrict__ old_logp,
    const float* __restrict__ ref_logp, const float* __restrict__ entropy,
    const float* __restrict__ adv_seq, const int32_t* __restrict__ cu, int B, int T,
    af_loss_params prm, af_loss_out* __restrict__ out, float* __restrict__ dlogp, LossWs* ws,
    unsigned int* d_err, int vec_ok) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ int s_win[kWindow];      // cu_seqlens[s_first .. s_first + s_count - 1]
  __shared__ float s_adv[kWindow];    // adv_seq of the same sequences
  __shared__ int s_first, s_count, s_cover;   // tokens < s_cover lie inside the staged window
  __shared__ int abort_flag;
  const uint32_t ring = (umma::smem_u32(smem_raw) + 127u) & ~127u;
  const uint32_t bars = ring + kStages * kStageBytes;
  auto full_bar = [&](int st) { return bars + 8u * st; };
  auto empty_bar = [&](int st) { return bars + 8u * (kStages + st); };
  const float lo_b = 1.f - prm.clip_lo, hi_b = 1.f + prm.clip_hi;
  const float w_all = lossmath::batch_weight(prm, B, T);
  const float nbeta = -prm.kl_coef;
  float acc_pg = 0.f, acc_kl = 0.f, acc_ent = 0.f;
  int acc_clip = 0;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

  const int n_chunks = (T + kChunk - 1) / kChunk;
  const int c_begin = (int)(((int64_t)n_chunks * blockIdx.x) / gridDim.x);
  const int n_mine = (int)(((int64_t)n_chunks * (blockIdx.x + 1)) / gridDim.x) - c_begin;
  const int n_cols = entropy ? 4 : 3;

  // feeding thread: bulk copies of chunk i's column slices into ring stage i % kStages.  A slice
  // is copied up to its last whole group of 4 tokens (16 bytes).
  auto issue = [&](int i) {
    const int c0 = (c_begin + i) * kChunk;
    const int ntok = T - c0 < kChunk ? T - c0 : kChunk;
    const uint32_t nb = (uint32_t)(ntok & ~3) * 4u;
    const uint32_t bar = full_bar(i % kStages);
    if (nb == 0) { umma::mbar_arrive(bar); return; }
    const uint32_t dst = ring + (i % kStages) * kStageBytes;
    umma::mbar_arrive_expect_tx(bar, nb * n_cols);
    bulk_load(dst, logp + c0, nb, bar);
    bulk_load(dst + kColBytes, old_logp + c0, nb, bar);
    bulk_load(dst + 2 * kColBytes, ref_logp + c0, nb, bar);
    if (entropy) bulk_load(dst + 3 * kColBytes, entropy + c0, nb, bar);
  };
  // cu_seqlens must be non-decreasing (its ends are checked by the last block): every entry is
  // compared with its successor once, spread over the grid; a violation only raises the flag --
  // nothing below indexes memory with a value taken from cu_seqlens
  for (int q = blockIdx.x * kThreads + threadIdx.x; q < B; q += gridDim.x * kThreads)
    if (__ldg(cu + q) > __ldg(cu + q + 1)) atomicOr(d_err, AF_DEVERR_CU_SEQLENS);
  if (threadIdx.x == 0) {
    abort_flag = 0;
    s_first = 0; s_count = 0; s_cover = -1;
    if (vec_ok) {
      for (int s = 0; s < kStages; ++s) { umma::mbar_init(full_bar(s), 1); umma::mbar_init(empty_bar(s), kWarps); }
      umma::fence_mbar_init();
      for (int i = 0; i < kStages && i < n_mine; ++i) issue(i);
    }
  }
  __syncthreads();

  int hint = 0;        // this thread's position in the window at the previous chunk
  bool ok = true;      // false once a wait ran out of time: the warp keeps the block-wide barriers
                       // of the loop in step with the others but touches no more data
  for (int i = 0; i < n_mine; ++i) {
    const int c0 = (c_begin + i) * kChunk;
    const int c_last = (T - c0 > kChunk ? c0 + kChunk : T) - 1;   // last token of the chunk
    if (c_last >= s_cover) {
      // (re)stage the window from the chunk's first sequence on; block-uniform and rare
      __syncthreads();
      if (warp == 0) {
        const int j = find_seq_warp(cu, B, c0, lane);
        if (lane == 0) {
          const int cnt = B + 1 - j < kWindow ? B + 1 - j : kWindow;
          s_first = j; s_count = cnt;
        }
      }
      __syncthreads();
      const int j = s_first, cnt = s_count;
      for (int q = threadIdx.x; q < cnt; q += kThreads) {
        s_win[q] = __ldg(cu + j + q);
        s_adv[q] = j + q < B ? __ldg(adv_seq + j + q) : 0.f;
      }
      if (threadIdx.x == 0) s_cover = __ldg(cu + j + cnt - 1);   // tokens below the last staged entry
      hint = 0;
      __syncthreads();
    }
    const int j0 = s_first, nw = s_count;
    const bool staged = c_last < s_cover;
    const int st = i % kStages;
    if (vec_ok && ok) {
      // the stage chunk i-1 used is refilled with chunk i + kStages - 1 once every warp has left it
      if (threadIdx.x == 0 && i >= 1 && i + kStages - 1 < n_mine) {
        if (umma::mbar_wait(empty_bar((i - 1) % kStages), (uint32_t)((i - 1) / kStages) & 1u, &abort_flag))
          issue(i + kStages - 1);
      }
      ok = __all_sync(0xffffffffu, umma::mbar_wait(full_bar(st), (uint32_t)(i / kStages) & 1u, &abort_flag));
    }
    if (!ok) continue;

    // token of slot k of this thread: group k / 4 starts 128 tokens after the previous one
    const int t0 = c0 + warp * kWarpTokens + lane * kGroup;
    auto tok = [&](int k) { return t0 + (k / kGroup) * (32 * kGroup) + (k % kGroup); };
    const int n = tok(kTokPerThread - 1) < T ? kTokPerThread : -1;      // -1: some slot lies past the end
    float lp[kTokPerThread], ol[kTokPerThread], rf[kTokPerThread], en[kTokPerThread], g[kTokPerThread];
#pragma unroll
    for (int k = 0; k < kTokPerThread; ++k) en[k] = 0.f;
    if (n == kTokPerThread && vec_ok) {
#pragma unroll
      for (int q = 0; q < kGroups; ++q) {
        const uint32_t src = ring + st * kStageBytes + (uint32_t)(tok(q * kGroup) - c0) * 4u;
        const float4 a = lds128(src), b = lds128(src + kColBytes), r = lds128(src + 2 * kColBytes);
        lp[4 * q] = a.x; lp[4 * q + 1] = a.y; lp[4 * q + 2] = a.z; lp[4 * q + 3] = a.w;
        ol[4 * q] = b.x; ol[4 * q + 1] = b.y; ol[4 * q + 2] = b.z; ol[4 * q + 3] = b.w;
        rf[4 * q] = r.x; rf[4 * q + 1] = r.y; rf[4 * q + 2] = r.z; rf[4 * q + 3] = r.w;
        if (entropy) {
          const float4 e = lds128(src + 3 * kColBytes);
          en[4 * q] = e.x; en[4 * q + 1] = e.y; en[4 * q + 2] = e.z; en[4 * q + 3] = e.w;
        }
      }
    } else {
#pragma unroll
      for (int k = 0; k < kTokPerThread; ++k) {
        const int t = tok(k);
        if (t < T) {
          lp[k] = __ldg(logp + t); ol[k] = __ldg(old_logp + t); rf[k] = __ldg(ref_logp + t);
          if (entropy) en[k] = __ldg(entropy + t);
        }
      }
    }
    if (vec_ok) {   // the values are in registers: this warp is done with the stage
      __syncwarp();
      if (lane == 0) umma::mbar_arrive(empty_bar(st));
    }
    if (t0 < T) {
      int j, seq_beg, seq_end;
      if (staged) {
        // gallop forward from the previous position, then bisect: s_win[lo] <= t0 < s_win[hi]
        int lo = hint, hi, step = 1;
        for (;;) {
          hi = lo + step;
          if (hi >= nw - 1) { hi = nw - 1; break; }
          if (s_win[hi] > t0) break;
          lo = hi; step <<= 1;
        }
        while (hi - lo > 1) {
          const int mid = (lo + hi) >> 1;
          if (s_win[mid] <= t0) lo = mid; else hi = mid;
        }
        hint = lo;
        j = j0 + lo; seq_beg = s_win[lo]; seq_end = s_win[lo + 1];
      } else {
        j = find_seq(cu, B, t0); seq_beg = __ldg(cu + j); seq_end = __ldg(cu + j + 1);
      }
      const int j_max = staged ? j0 + nw - 2 : B - 1;   // last sequence this thread may step to
      float A = staged ? s_adv[j - j0] : __ldg(adv_seq + j);
      float inv_len = lossmath::inv_length(prm, seq_end - seq_beg);
      float run_pg = 0.f, run_kl = 0.f;
#pragma unroll
      for (int k = 0; k < kTokPerThread; ++k) {
        const int t = tok(k);                 // increasing in k: the thread walks forward through the sequences
        if (t < T) {
          if (t >= seq_end) {  // run of sequence j ends: scale it once, move to the next sequence
            acc_pg += run_pg * inv_len; acc_kl += run_kl * inv_len;
            run_pg = 0.f; run_kl = 0.f;
            while (t >= seq_end && j < j_max) {
              ++j;
              seq_beg = seq_end;
              seq_end = staged ? s_win[j - j0 + 1] : __ldg(cu + j + 1);
            }
            A = staged ? s_adv[j - j0] : __ldg(adv_seq + j);
            inv_len = lossmath::inv_length(prm, seq_end - seq_beg);
          }
          const lossmath::TokenTerms tt = lossmath::token_terms(lp[k], ol[k], rf[k], A, lo_b, hi_b, nbeta);
          run_pg += tt.pg;
          run_kl += tt.k3;
          acc_ent += en[k];
          acc_clip += tt.clipped ? 1 : 0;
          g[k] = (w_all * inv_len) * tt.grad;
        }
      }
      acc_pg += run_pg * inv_len; acc_kl += run_kl * inv_len;
      if (dlogp) {
        if (n == kTokPerThread && vec_ok) {
#pragma unroll
          for (int q = 0; q < kGroups; ++q)
            *reinterpret_cast<float4*>(dlogp + tok(q * kGroup)) = make_float4(g[4 * q], g[4 * q + 1], g[4 * q + 2], g[4 * q + 3]);
        } else {
#pragma unroll
          for (int k = 0; k < kTokPerThread; ++k) if (tok(k) < T) dlogp[tok(k)] = g[k];
        }
      }
    }
  }

  __syncthreads();
  if (abort_flag) {   // a bulk copy did not arrive in time: flag it, let copies in flight land
    if (threadIdx.x == 0) atomicOr(d_err, umma::kWatchdogBit);
    __nanosleep(1000000);
  }

  // block reduction: warp shuffles, then fp64 across warps (fixed order)
  __shared__ double s_part[kThreads / 32][kNumSums];
  __shared__ int s_last;
  double v[kNumSums] = {(double)acc_pg, (double)acc_kl, (double)acc_ent, (double)acc_clip};
#pragma unroll
  for (int q = 0; q < kNumSums; ++q)
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v[q] += __shfl_xor_sync(0xffffffffu, v[q], o);
  if (lane == 0)
    for (int q = 0; q < kNumSums; ++q) s_part[warp][q] = v[q];
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int q = 0; q < kNumSums; ++q) {
      double t = 0.0;
      for (int w = 0; w < kThreads / 32; ++w) t += s_part[w][q];
      ws_partial(ws, blockIdx.x)[q] = t;
    }
    __threadfence();
    const unsigned int ticket = atomicAdd(&ws->ticket, 1u);
    s_last = (ticket == gridDim.x - 1);
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  if (warp == 0) {
    double tot[kNumSums] = {0.0, 0.0, 0.0, 0.0};
    for (int b = lane; b < (int)gridDim.x; b += 32)
      for (int q = 0; q < kNumSums; ++q) tot[q] += __ldcg(ws_partial(ws, b) + q);
#pragma unroll
    for (int q = 0; q < kNumSums; ++q)
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) tot[q] += __shfl_xor_sync(0xffffffffu, tot[q], o);
    if (lane == 0) {
      const double w = (double)w_all;
      af_loss_out r;
      r.pg_loss = (float)(w * tot[0]);
      r.kl_mean = (float)(w * tot[1]);
      r.loss = (float)(w * tot[0] + (double)prm.kl_coef * (w * tot[1]));
      r.entropy_mean = T > 0 ? (float)(tot[2] / (double)T) : 0.f;
      r.clip_frac = T > 0 ? (float)(tot[3] / (double)T) : 0.f;
      r.reserved = 0;
      r.n_tokens = T;
      *out = r;
      if (__ldg(cu) != 0 || __ldg(cu + B) != T) atomicOr(d_err, AF_DEVERR_CU_SEQLENS);
      ws->ticket = 0;  // ready for the next call on this stream
    }
  }
}

}  // namespace

size_t loss_workspace_bytes(int sm_count) {
  return 64 + (size_t)sm_count * 8 * kNumSums * sizeof(double);
}

cudaError_t launch_policy_loss(const float* logp, const float* old_logp, const float* ref_logp,
                               const float* entropy, const float* adv_seq, const int32_t* cu,
                               int32_t B, int64_t T, const af_loss_params& p, af_loss_out* out,
                               float* dlogp, void* ws, unsigned int* d_err, int sm_count,
                               cudaStream_t s) {
  {
    static SmemAttrOnce once;
    cudaError_t e = set_smem_once(once, policy_loss_kernel, kRingSmemBytes);
    if (e != cudaSuccess) return e;
  }
  const int64_t chunks = (T + kChunk - 1) / kChunk;
  // two CTAs per SM, each over a contiguous range of chunks (grid <= the workspace's 8 blocks per SM)
  const int blocks = (int)(chunks < 1 ? 1 : (chunks < (int64_t)sm_count * 2 ? chunks : (int64_t)sm_count * 2));
  auto al = [](const void* q) { return (reinterpret_cast<uintptr_t>(q) & 15) == 0; };
  const int vec_ok = al(logp) && al(old_logp) && al(ref_logp) && al(entropy) && al(dlogp);
  policy_loss_kernel<<<blocks, kThreads, kRingSmemBytes, s>>>(logp, old_logp, ref_logp, entropy, adv_seq, cu,
                                                              B, (int)T, p, out, dlogp, (LossWs*)ws, d_err,
                                                              vec_ok);
  return cudaGetLastError();
}

}  // namespace af
