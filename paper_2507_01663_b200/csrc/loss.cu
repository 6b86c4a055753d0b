// af_policy_loss kernel: clipped-ratio GRPO policy loss + k3 KL penalty, forward and dL/dlogp,
// in one pass over the packed tokens (12-16 B read, 4 B written per token: HBM-bound).
//
// A block walks chunks of 1024-4096 tokens.  Per chunk, two warps locate the first and last
// sequence it touches with a 32-way search over cu_seqlens and the block stages that window in
// shared memory; token loads are issued before the lookup so both latencies overlap.  Each thread
// owns 4 consecutive tokens (128-bit loads/stores).  Tokens of one sequence are contiguous, so a
// thread sums its tokens run by run and scales each run by 1/L_i once (the per-sequence mean of
// agg_mode 0); runs are combined with warp shuffles, per-block sums go to the workspace in fp64
// and the last block to finish adds them in a fixed order -- no float atomics, so results are
// bit-reproducible.
#include "common.cuh"

namespace af {
namespace {

constexpr int kThreads = 256;
constexpr int kTokPerThread = 4;
constexpr int kMaxSub = 4;                                // most passes of a block over one chunk
constexpr int kPass = kThreads * kTokPerThread;           // tokens per pass
constexpr int kMaxChunk = kPass * kMaxSub;                // most tokens per sequence-window lookup
constexpr int kNumSums = 4;  // pg, k3, entropy, clipped count

struct LossWs {            // 64-byte header, then double partial[blocks][kNumSums]
  unsigned int ticket;
  unsigned int pad[15];
};
__device__ __forceinline__ double* ws_partial(LossWs* ws, int block) {
  return reinterpret_cast<double*>(ws + 1) + (size_t)block * kNumSums;
}

constexpr float kLog2e = 1.4426950408889634f;
constexpr int kWindow = kMaxChunk + 1;  // most cu_seqlens entries a chunk can touch unless empty sequences pile up

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// largest j in [0, B) with cu[j] <= t  (cu non-decreasing, cu[0] = 0, t < cu[B])
__device__ __forceinline__ int find_seq(const int32_t* __restrict__ cu, int B, int t) {
  int lo = 0, hi = B;
  while (hi - lo > 1) {
    int mid = (lo + hi) >> 1;
    if (__ldg(cu + mid) <= t) lo = mid; else hi = mid;
  }
  return lo;
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

__global__ void __launch_bounds__(kThreads, 4) policy_loss_kernel(
    const float* __restrict__ logp, const float* __restrict__ old_logp,
    const float* __restrict__ ref_logp, const float* __restrict__ entropy,
    const float* __restrict__ adv_seq, const int32_t* __restrict__ cu, int B, int T,
    af_loss_params prm, af_loss_out* __restrict__ out, float* __restrict__ dlogp, LossWs* ws,
    unsigned int* d_err, int vec_ok, int n_sub) {
  __shared__ int s_cu[2][kWindow];
  __shared__ int s_j0[2], s_j1[2];
  const float lo_b = 1.f - prm.clip_lo, hi_b = 1.f + prm.clip_hi;
  const float w_all = prm.agg_mode == 0 ? (B > 0 ? prm.loss_scale / (float)B : 0.f)
                                        : (T > 0 ? prm.loss_scale / (float)T : 0.f);
  const float nbeta = -prm.kl_coef;
  float acc_pg = 0.f, acc_kl = 0.f, acc_ent = 0.f;
  int acc_clip = 0;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

  const int kChunk = kPass * n_sub;   // tokens that share one sequence-window lookup
  const int n_chunks = (T + kChunk - 1) / kChunk;
  int buf = 0;
  for (int c = blockIdx.x; c < n_chunks; c += gridDim.x, buf ^= 1) {
    const int c0 = c * kChunk;
    const int c_last = (T - c0 > kChunk ? c0 + kChunk : T) - 1;   // last token of the chunk
    // the chunk's window of cu_seqlens: entries j0 .. j1+1 (first and last sequence it touches)
    if (warp == 0) {
      const int j = find_seq_warp(cu, B, c0, lane);
      if (lane == 0) s_j0[buf] = j;
    } else if (warp == 1) {
      const int j = find_seq_warp(cu, B, c_last, lane);
      if (lane == 0) s_j1[buf] = j;
    }
    __syncthreads();
    const int j0 = s_j0[buf];
    const int nw = s_j1[buf] - j0 + 2;
    const bool staged = nw <= kWindow;
    int* win = s_cu[buf];
    if (staged)
      for (int i = threadIdx.x; i < nw; i += kThreads) win[i] = __ldg(cu + j0 + i);
    __syncthreads();

#pragma unroll 1
    for (int sub = 0; sub < n_sub; ++sub) {
      const int t0 = c0 + sub * kPass + threadIdx.x * kTokPerThread;
      const int n = t0 < T ? ((T - t0) < kTokPerThread ? (T - t0) : kTokPerThread) : 0;
      float lp[4], ol[4], rf[4], en[4] = {0.f, 0.f, 0.f, 0.f}, g[4];
      if (n == 4 && vec_ok) {
        const float4 a = __ldg(reinterpret_cast<const float4*>(logp + t0));
        const float4 b = __ldg(reinterpret_cast<const float4*>(old_logp + t0));
        const float4 r = __ldg(reinterpret_cast<const float4*>(ref_logp + t0));
        lp[0] = a.x; lp[1] = a.y; lp[2] = a.z; lp[3] = a.w;
        ol[0] = b.x; ol[1] = b.y; ol[2] = b.z; ol[3] = b.w;
        rf[0] = r.x; rf[1] = r.y; rf[2] = r.z; rf[3] = r.w;
        if (entropy) {
          const float4 e = __ldg(reinterpret_cast<const float4*>(entropy + t0));
          en[0] = e.x; en[1] = e.y; en[2] = e.z; en[3] = e.w;
        }
      } else {
        for (int k = 0; k < n; ++k) {
          lp[k] = __ldg(logp + t0 + k); ol[k] = __ldg(old_logp + t0 + k); rf[k] = __ldg(ref_logp + t0 + k);
          if (entropy) en[k] = __ldg(entropy + t0 + k);
        }
      }
      if (n > 0) {
        int j, seq_beg, seq_end;
        if (staged) {
          int lo = 0, hi = nw - 1;  // win[lo] <= t0, and t0 < win[hi] unless cu_seqlens is malformed
          while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (win[mid] <= t0) lo = mid; else hi = mid;
          }
          j = j0 + lo; seq_beg = win[lo]; seq_end = win[lo + 1];
        } else {
          j = find_seq(cu, B, t0); seq_beg = __ldg(cu + j); seq_end = __ldg(cu + j + 1);
        }
        const int j_max = staged ? j0 + nw - 2 : B - 1;   // last sequence this thread may step to
        float A = __ldg(adv_seq + j);
        float inv_len = prm.agg_mode == 0 ? __frcp_rn((float)(seq_end - seq_beg)) : 1.f;
        float run_pg = 0.f, run_kl = 0.f;
#pragma unroll
        for (int k = 0; k < kTokPerThread; ++k) {
          if (k < n) {
            const int t = t0 + k;
            if (t >= seq_end) {  // run of sequence j ends: scale it once, move to the next sequence
              acc_pg += run_pg * inv_len; acc_kl += run_kl * inv_len;
              run_pg = 0.f; run_kl = 0.f;
              while (t >= seq_end && j < j_max) {
                ++j;
                seq_beg = seq_end;
                seq_end = staged ? win[j - j0 + 1] : __ldg(cu + j + 1);
              }
              A = __ldg(adv_seq + j);
              inv_len = prm.agg_mode == 0 ? __frcp_rn((float)(seq_end - seq_beg)) : 1.f;
            }
            const float rho = ex2f((lp[k] - ol[k]) * kLog2e);
            const float s1 = rho * A;
            const float s2 = fminf(fmaxf(rho, lo_b), hi_b) * A;
            const bool clipped = s2 < s1;
            const float delta = rf[k] - lp[k];
            const float em1 = ex2f(delta * kLog2e) - 1.f;   // exactly 0 when ref == logp
            run_pg -= fminf(s1, s2);
            run_kl += em1 - delta;
            acc_ent += en[k];
            acc_clip += clipped ? 1 : 0;
            g[k] = (w_all * inv_len) * fmaf(nbeta, em1, clipped ? 0.f : -s1);
          }
        }
        acc_pg += run_pg * inv_len; acc_kl += run_kl * inv_len;
        if (dlogp) {
          if (n == 4 && vec_ok) {
            *reinterpret_cast<float4*>(dlogp + t0) = make_float4(g[0], g[1], g[2], g[3]);
          } else {
            for (int k = 0; k < n; ++k) dlogp[t0 + k] = g[k];
          }
        }
    }
    }
    // no barrier here: the next chunk uses the other window buffer, and its first barrier
    // orders this chunk's reads before the chunk after it reuses this buffer
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
  // large batches amortise the sequence-window lookup over several passes; small ones keep one
  // pass per block so that every SM has work
  int n_sub = 1;
  while (n_sub < kMaxSub && T / ((int64_t)kPass * n_sub * 2) >= (int64_t)sm_count * 4) n_sub *= 2;
  const int64_t chunk = (int64_t)kPass * n_sub;
  int64_t chunks = (T + chunk - 1) / chunk;
  int blocks = (int)(chunks < 1 ? 1 : (chunks < (int64_t)sm_count * 8 ? chunks : (int64_t)sm_count * 8));
  auto al = [](const void* q) { return (reinterpret_cast<uintptr_t>(q) & 15) == 0; };
  const int vec_ok = al(logp) && al(old_logp) && al(ref_logp) && al(entropy) && al(dlogp);
  policy_loss_kernel<<<blocks, kThreads, 0, s>>>(logp, old_logp, ref_logp, entropy, adv_seq, cu, B,
                                                 (int)T, p, out, dlogp, (LossWs*)ws, d_err, vec_ok, n_sub);
  return cudaGetLastError();
}

}  // namespace af
