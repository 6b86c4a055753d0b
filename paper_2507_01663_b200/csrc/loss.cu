// af_policy_loss kernel: clipped-ratio GRPO policy loss + k3 KL penalty, forward and dL/dlogp,
// in one pass over the packed tokens (12-16 B read, 4 B written per token: HBM-bound).
//
// Each thread owns 4 consecutive tokens (128-bit loads/stores).  Tokens of one sequence are
// contiguous (cu_seqlens), so a thread sums its tokens run by run and scales each run by
// 1/L_i once (the per-sequence mean of agg_mode 0); runs are then combined with warp shuffles,
// per-block sums go to the workspace in fp64 and the last block to finish adds them in a fixed
// order -- no float atomics, so results are bit-reproducible.
#include "common.cuh"

namespace af {
namespace {

constexpr int kThreads = 256;
constexpr int kTokPerThread = 4;
constexpr int kChunk = kThreads * kTokPerThread;
constexpr int kNumSums = 4;  // pg, k3, entropy, clipped count

struct LossWs {            // 64-byte header, then double partial[blocks][kNumSums]
  unsigned int ticket;
  unsigned int pad[15];
};
__device__ __forceinline__ double* ws_partial(LossWs* ws, int block) {
  return reinterpret_cast<double*>(ws + 1) + (size_t)block * kNumSums;
}

__device__ __forceinline__ int find_seq(const int32_t* __restrict__ cu, int B, int t) {
  int lo = 0, hi = B;
  while (hi - lo > 1) {
    int mid = (lo + hi) >> 1;
    if (__ldg(cu + mid) <= t) lo = mid; else hi = mid;
  }
  return lo;
}

__global__ void __launch_bounds__(kThreads) policy_loss_kernel(
    const float* __restrict__ logp, const float* __restrict__ old_logp,
    const float* __restrict__ ref_logp, const float* __restrict__ entropy,
    const float* __restrict__ adv_seq, const int32_t* __restrict__ cu, int B, int T,
    af_loss_params prm, af_loss_out* __restrict__ out, float* __restrict__ dlogp, LossWs* ws,
    unsigned int* d_err, int vec_ok) {
  const float lo_b = 1.f - prm.clip_lo, hi_b = 1.f + prm.clip_hi;
  const float w_all = prm.agg_mode == 0 ? (B > 0 ? prm.loss_scale / (float)B : 0.f)
                                        : (T > 0 ? prm.loss_scale / (float)T : 0.f);
  float acc_pg = 0.f, acc_kl = 0.f, acc_ent = 0.f;
  int acc_clip = 0;

  const int n_chunks = (T + kChunk - 1) / kChunk;
  for (int c = blockIdx.x; c < n_chunks; c += gridDim.x) {
    const int t0 = c * kChunk + threadIdx.x * kTokPerThread;
    if (t0 >= T) continue;
    const int n = (T - t0) < kTokPerThread ? (T - t0) : kTokPerThread;
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
    int j = find_seq(cu, B, t0);
    int seq_end = __ldg(cu + j + 1);
    float A = __ldg(adv_seq + j);
    float inv_len = prm.agg_mode == 0 ? 1.f / (float)(seq_end - __ldg(cu + j)) : 1.f;
    float run_pg = 0.f, run_kl = 0.f;
#pragma unroll
    for (int k = 0; k < kTokPerThread; ++k) {
      if (k < n) {
        const int t = t0 + k;
        if (t >= seq_end) {  // run of sequence j ends: scale it once, move to the next sequence
          acc_pg += run_pg * inv_len; acc_kl += run_kl * inv_len;
          run_pg = 0.f; run_kl = 0.f;
          while (t >= seq_end && j < B - 1) { ++j; seq_end = __ldg(cu + j + 1); }
          A = __ldg(adv_seq + j);
          inv_len = prm.agg_mode == 0 ? 1.f / (float)(seq_end - __ldg(cu + j)) : 1.f;
        }
        const float rho = expf(lp[k] - ol[k]);
        const float s1 = rho * A;
        const float s2 = fminf(fmaxf(rho, lo_b), hi_b) * A;
        const bool clipped = s2 < s1;
        const float delta = rf[k] - lp[k];
        const float em1 = expm1f(delta);
        run_pg += -fminf(s1, s2);
        run_kl += em1 - delta;
        acc_ent += en[k];
        acc_clip += clipped ? 1 : 0;
        g[k] = (w_all * inv_len) * ((clipped ? 0.f : -s1) - prm.kl_coef * em1);
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

  // block reduction: warp shuffles, then fp64 across warps (fixed order)
  __shared__ double s_part[kThreads / 32][kNumSums];
  __shared__ int s_last;
  double v[kNumSums] = {(double)acc_pg, (double)acc_kl, (double)acc_ent, (double)acc_clip};
#pragma unroll
  for (int q = 0; q < kNumSums; ++q)
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v[q] += __shfl_xor_sync(0xffffffffu, v[q], o);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
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
  int64_t chunks = (T + kChunk - 1) / kChunk;
  int blocks = (int)(chunks < 1 ? 1 : (chunks < (int64_t)sm_count * 8 ? chunks : (int64_t)sm_count * 8));
  auto al = [](const void* q) { return (reinterpret_cast<uintptr_t>(q) & 15) == 0; };
  const int vec_ok = al(logp) && al(old_logp) && al(ref_logp) && al(entropy) && al(dlogp);
  policy_loss_kernel<<<blocks, kThreads, 0, s>>>(logp, old_logp, ref_logp, entropy, adv_seq, cu, B,
                                                 (int)T, p, out, dlogp, (LossWs*)ws, d_err, vec_ok);
  return cudaGetLastError();
}

}  // namespace af
