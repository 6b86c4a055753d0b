// af_policy_update: forward, loss and backward of one packed micro-batch in one call (the
// actor-update task), token block by token block.
//
// Run as three separate calls, the actor update computes the logits twice: once for the log-probs
// and once more, block by block, for dZ.  Here a block's logits are kept in fp32 between the two
// uses (scratch of one block, like dZ: [T, V] is never materialised), so the second GEMM becomes a
// memory-bound pass:
//   per block   1. Z = H_blk W^T on the tensor cores; the epilogue keeps the online-softmax
//                  statistics AND stores Z (fp32) -> logp, entropy, lse of the block's tokens;
//               2. one CTA per token row: g_t from (logp, old, ref, advantage, sequence length)
//                  with the loss kernel's own arithmetic, then dZ = g_t (1{v = y_t} - exp(z - lse_t))
//                  in bf16 (reads 4 V, writes 2 V bytes per token);
//               3. dH_blk = dZ W and dW += dZ^T H_blk as in af_policy_loss_backward.
//   at the end  the loss scalars over all tokens, by the loss kernel itself.
// The results are those of the three calls with the same token block (same accumulators, same
// per-token arithmetic), and 2 of their 8 T d V products are gone.
#include "loss_math.cuh"

namespace af {
namespace {

constexpr int kThreads = 256;



// One CTA per token row of the block.  z: [rows, V] fp32 logits; dz: [rows, V] bf16.  V % 8 == 0.
__global__ void __launch_bounds__(kThreads) dz_from_logits_kernel(
    const float* __restrict__ z, __nv_bfloat16* __restrict__ dz, int V, const int32_t* __restrict__ target,
    const float* __restrict__ lse, const float* __restrict__ logp, const float* __restrict__ old_logp,
    const float* __restrict__ ref_logp, const float* __restrict__ adv_seq, const int32_t* __restrict__ cu,
    int B, int T, int t0, af_loss_params prm, float* __restrict__ dlogp) {
  __shared__ float s_g;
  const int row = blockIdx.x;          // token t0 + row of the batch; all per-token pointers start at t0
  if (threadIdx.x == 0) {
    const int t = t0 + row;
    const int j = find_seq(cu, B, t);
    const int len = __ldg(cu + j + 1) - __ldg(cu + j);
    const lossmath::TokenTerms tt = lossmath::token_terms(__ldg(logp + row), __ldg(old_logp + row), __ldg(ref_logp + row),
                                                          __ldg(adv_seq + j), 1.f - prm.clip_lo, 1.f + prm.clip_hi,
                                                          -prm.kl_coef);
    const float g = (lossmath::batch_weight(prm, B, T) * lossmath::inv_length(prm, len)) * tt.grad;
    s_g = g;
    if (dlogp) dlogp[row] = g;
  }
  __syncthreads();
  const float g = s_g;
  const float nl = -__ldg(lse + row) * lossmath::kLog2e;
  const int y = __ldg(target + row);
  const float4* zr = reinterpret_cast<const float4*>(z + (size_t)row * V);
  uint4* out = reinterpret_cast<uint4*>(dz + (size_t)row * V);
  for (int c8 = threadIdx.x; c8 * 8 < V; c8 += kThreads) {      // 8 columns per thread per step
    const float4 a = __ldcs(zr + 2 * c8), b = __ldcs(zr + 2 * c8 + 1);
    float v[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
    for (int k = 0; k < 8; ++k) v[k] = -g * lossmath::ex2f(fmaf(v[k], lossmath::kLog2e, nl));
    const int yl = y - c8 * 8;
    if (yl >= 0 && yl < 8) {
#pragma unroll
      for (int k = 0; k < 8; ++k) if (k == yl) v[k] += g;
    }
    out[c8] = make_uint4(pack_bf16x2(v[0], v[1]), pack_bf16x2(v[2], v[3]), pack_bf16x2(v[4], v[5]),
                         pack_bf16x2(v[6], v[7]));
  }
}

}  // namespace

af_status launch_policy_update(af_ctx* ctx, const void* hidden, const void* W, const int32_t* target,
                               const float* old_logp, const float* ref_logp, const float* adv_seq,
                               const int32_t* cu_seqlens, int32_t B, int64_t T, int32_t d, int32_t V,
                               const af_loss_params& params, af_loss_out* out, float* logp, float* entropy,
                               float* lse, float* dlogp, void* d_hidden, float* d_W, int32_t accumulate_dW,
                               cudaStream_t s) {
  const int64_t Tc = backward_token_block(ctx, T);
  af_status st;
  if ((st = ws_grow(ctx->dz, (size_t)Tc * V * 2)) != AF_OK) return st;
  if ((st = ws_grow(ctx->zlog, (size_t)Tc * V * 4)) != AF_OK) return st;
  if (accumulate_dW < 0) return AF_OK;  // reserve only
  if (T == 0) {
    if (!accumulate_dW && cudaMemsetAsync(d_W, 0, (size_t)V * d * sizeof(float), s) != cudaSuccess) return AF_ERR_CUDA;
    if (ctx->dw_ready && cudaEventRecord(ctx->dw_ready, s) != cudaSuccess) return AF_ERR_CUDA;
  }
  const __nv_bfloat16* H = static_cast<const __nv_bfloat16*>(hidden);
  __nv_bfloat16* dz = static_cast<__nv_bfloat16*>(ctx->dz.p);
  float* zlog = static_cast<float*>(ctx->zlog.p);
  bool first = true;
  for (int64_t t0 = 0; t0 < T; t0 += Tc, first = false) {
    const int64_t tc = (T - t0) < Tc ? (T - t0) : Tc;
    // 1. logits of the block: statistics -> logp / entropy / lse, values -> zlog
    st = launch_token_logprob_z(ctx, H + t0 * d, W, target + t0, tc, d, V, logp + t0,
                                entropy ? entropy + t0 : nullptr, lse + t0, zlog, s);
    if (st != AF_OK) return st;
    // 2. per-token gradient of the loss and dZ
    dz_from_logits_kernel<<<(int)tc, kThreads, 0, s>>>(zlog, dz, V, target + t0, lse + t0, logp + t0, old_logp + t0,
                                                       ref_logp + t0, adv_seq, cu_seqlens, B, (int)T, (int)t0, params,
                                                       dlogp ? dlogp + t0 : nullptr);
    if (cudaGetLastError() != cudaSuccess) return AF_ERR_CUDA;
    // 3. the two products that consume dZ
    st = launch_backward_products(ctx, H + t0 * d, W, dz, tc, d, V, static_cast<__nv_bfloat16*>(d_hidden) + t0 * d,
                                  d_W, (!first || accumulate_dW) ? 1 : 0, t0 + Tc >= T, s);
    if (st != AF_OK) return st;
  }
  // loss scalars over the whole batch, from the log-probs just written
  return launch_policy_loss(logp, old_logp, ref_logp, entropy, adv_seq, cu_seqlens, B, T, params, out, nullptr,
                            ctx->loss_ws.p, ctx->d_err, ctx->sm_count, s) == cudaSuccess ? AF_OK : AF_ERR_CUDA;
}

}  // namespace af
