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
  const float em1 = ex2f(delta * kLog2e) - 1.f;   // exactly 0 when ref == logp
  t.pg = -fminf(s1, s2);
  t.k3 = em1 - delta;
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
