// Per-token arithmetic of the clipped-ratio policy loss with the k3 KL penalty, shared by the
// loss kernel and the fused actor update so that both produce the same bits.
#pragma once

#include "common.cuh"
#include "device_util.cuh"

namespace af {
namespace lossmath {

using af::ex2f;
using af::kLog2e;

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
  // exp(delta) - 1 (for the gradient) comes from the approximate exp2: about 2^-22 relative on a
  // value near 1, i.e. 2.4e-7 absolute, which no gradient tolerance notices.  k3 = exp(delta) -
  // delta - 1 would inherit that absolute error, and near the reference policy (k3 = delta^2 / 2)
  // it is several 1e-3 relative at |delta| = 0.01: for |delta| < 1/32 k3 is therefore taken from
  // its series delta^2 (1/2 + delta/6) (truncation delta^2/12 < 8e-5 relative, no cancellation,
  // exactly 0 when ref == logp); from 1/32 on the direct form is good to 5e-4.  The loss kernel runs
  // at its issue limit when it streams at full bandwidth (every instruction per token costs it
  // about 0.9 % of its GB/s; a six-term series for both quantities cost 10 %), hence the short
  // series.  Explicit roundings: the loss kernel and the fused
  // update must produce the same bits, so the compiler may not contract these differently at the
  // two call sites.
  const float em1 = __fadd_rn(ex2f(__fmul_rn(delta, kLog2e)), -1.f);
  const float k3_direct = __fadd_rn(em1, -delta);
  const float k3_series = __fmul_rn(__fmul_rn(delta, delta), fmaf(delta, 1.f / 6.f, 0.5f));
  const float k3 = fabsf(delta) < 0.03125f ? k3_series : k3_direct;
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
