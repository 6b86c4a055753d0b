// Per-token arithmetic of the clipped-ratio policy loss with the k3 KL penalty, shared by the
// loss kernel and the fused actor update so that both produce the same bits.
#pragma once

#include "common.cuh"

namespace af {
namespace lossmath {

constexpr float kLog2e = 1.4426950408889634f;

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

struct TokenTerms {
  float pg;       // -min(rho A, clip(rho) A)
  float k3;       // exp(delta) - delta - 1, delta = ref - logp
  float grad;     // d(pg + beta k3) / dlogp before the token's weight
  bool clipped;   // clip(rho) A < rho A (strictly)
};

// lo_b = 1 - clip_lo, hi_b = 1 + clip_hi, nbeta = -kl_coef.
__device__ __forceinline__ TokenTerms token_terms(float logp, float old_logp, float ref_logp, float A,
                                                  float lo_b, float hi_b, float nbeta) {
  TokenTerms t;
  const float rho = ex2f((logp - old_logp) * kLog2e);
  const float s1 = rho * A;
  const float s2 = fminf(fmaxf(rho, lo_b), hi_b) * A;
  t.clipped = s2 < s1;
  const float delta = ref_logp - logp;
  // exp(delta) - 1 and k3 = exp(delta) - delta - 1.  Near the reference policy both are tiny
  // differences of numbers near 1, where the approximate exp2 (about 2^-22 relative on a value
  // near 1) would leave k3 = delta^2 / 2 with an absolute error of 2.4e-7: several 1e-3 relative at
  // |delta| = 0.01.  For |delta| < 1/4 the series is used instead (truncation below 2e-8 relative),
  // k3 = delta^2 (1/2 + delta/6 + ... + delta^5/5040) without any cancellation, exp(delta) - 1 =
  // delta + k3; both are exactly 0 when ref == logp.
  float em1 = ex2f(delta * kLog2e) - 1.f;
  float k3 = em1 - delta;
  if (fabsf(delta) < 0.25f) {
    float q = fmaf(delta, 1.f / 5040.f, 1.f / 720.f);
    q = fmaf(delta, q, 1.f / 120.f);
    q = fmaf(delta, q, 1.f / 24.f);
    q = fmaf(delta, q, 1.f / 6.f);
    q = fmaf(delta, q, 0.5f);
    k3 = delta * delta * q;
    em1 = delta + k3;
  }
  t.pg = -fminf(s1, s2);
  t.k3 = k3;
  t.grad = fmaf(nbeta, em1, t.clipped ? 0.f : -s1);
  return t;
}

// Weight of the whole batch in the aggregation, and of a token of a sequence of `len` tokens.
__device__ __forceinline__ float batch_weight(const af_loss_params& prm, int B, int T) {
  return prm.agg_mode == 0 ? (B > 0 ? prm.loss_scale / (float)B : 0.f) : (T > 0 ? prm.loss_scale / (float)T : 0.f);
}
__device__ __forceinline__ float inv_length(const af_loss_params& prm, int len) {
  return prm.agg_mode == 0 ? __frcp_rn((float)len) : 1.f;
}

}  // namespace lossmath
}  // namespace af
