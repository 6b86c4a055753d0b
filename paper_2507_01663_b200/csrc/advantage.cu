// af_grpo_advantage kernels: adv_i = (r_i - mean_g) / (std_g + eps) within each prompt's group.
//
// Contiguous groups (group_id == NULL), 4 B read + 4 B written per sample:
//   G a power of two in 4..512 (every GRPO workload here) and 16-byte aligned buffers: a thread
//   owns 4 consecutive rewards of each of four groups (G <= 16) or 16 rewards of one group
//   (G >= 32), the adjacent lanes of a group combine their sums with shuffles, four independent
//   128-bit loads are in flight per thread;
//   other G < 16: a kernel per group size (a lane owns 16 / G whole groups, staged through a
//   warp-private slice of shared memory); G = 1, 2 and unaligned buffers: one thread per group;
//   other G <= 512: a warp stages a run of whole groups in its slice of shared memory, a team of
//   lanes takes each group into registers, the slice streams out again (no block-wide barrier);
//   G <= 4096: a block stages a run of whole groups in shared memory with 128-bit loads, reduces
//   each group with warp shuffles (two passes: mean, then squared deviations) and writes the
//   advantages back coalesced;  larger groups: one block per group.
// Arbitrary membership (group_id given) lives in advantage_ids.cu.
#include "common.cuh"

namespace af {
namespace {

constexpr int kThreads = 256;
constexpr int kStage = 4096;             // samples staged per block iteration (16 KB)
constexpr int kMaxGroupsStaged = 1024;   // groups per block iteration

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Sum over `team` consecutive lanes (team a power of two <= 32).
__device__ __forceinline__ double team_sum(double v, int team) {
  for (int o = team >> 1; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Statistics are accumulated in fp64: a group of equal, non-dyadic rewards must come out with
// deviations ~1e-17 (as in exact arithmetic: zero), not ~1e-8, because they are divided by eps.
__device__ __forceinline__ double inv_scale(double ssq, int64_t n, int ddof, float eps) {
  const int64_t denom = n - ddof;
  const double sigma = denom > 0 ? sqrt(ssq / (double)denom) : 0.0;
  return 1.0 / (sigma + (double)eps);
}

// Small contiguous groups (G <= 32): one thread per group.  A thread reads its group's G
// consecutive rewards into registers (128-bit loads when G % 4 == 0), takes the two sums in fp64
// and writes G advantages back; adjacent threads own adjacent groups, so a warp covers one
// contiguous 32*G*4-byte span -- no shared memory, no shuffles, no barriers.
constexpr int kSmallG = 32;
template <int kCap>  // kCap = 4, 8, 16 or 32 >= G: bounds the register array
__global__ void __launch_bounds__(kThreads) advantage_small_group_kernel(
    const float* __restrict__ reward, float* __restrict__ adv, int64_t n_groups, int G, float eps,
    int ddof, int vec_ok) {
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; g < n_groups; g += stride) {
    const float* src = reward + g * G;
    float* dst = adv + g * G;
    float r[kCap];
    if (vec_ok) {
#pragma unroll
      for (int q = 0; q < kCap / 4; ++q) {
        if (q * 4 < G) {
          const float4 v = __ldg(reinterpret_cast<const float4*>(src) + q);
          r[q * 4 + 0] = v.x; r[q * 4 + 1] = v.y; r[q * 4 + 2] = v.z; r[q * 4 + 3] = v.w;
        }
      }
    } else {
#pragma unroll
      for (int k = 0; k < kCap; ++k) if (k < G) r[k] = __ldg(src + k);
    }
    double s = 0.0;
#pragma unroll
    for (int k = 0; k < kCap; ++k) if (k < G) s += (double)r[k];
    const double mu = s / (double)G;
    double q2 = 0.0;
#pragma unroll
    for (int k = 0; k < kCap; ++k) if (k < G) { const double dv = (double)r[k] - mu; q2 += dv * dv; }
    const double inv = inv_scale(q2, G, ddof, eps);
#pragma unroll
    for (int k = 0; k < kCap; ++k) if (k < G) r[k] = (float)(((double)r[k] - mu) * inv);
    if (vec_ok) {
#pragma unroll
      for (int q = 0; q < kCap / 4; ++q)
        if (q * 4 < G)
          reinterpret_cast<float4*>(dst)[q] = make_float4(r[q * 4 + 0], r[q * 4 + 1], r[q * 4 + 2], r[q * 4 + 3]);
    } else {
#pragma unroll
      for (int k = 0; k < kCap; ++k) if (k < G) dst[k] = r[k];
    }
  }
}

// Power-of-two groups, 4 <= G <= 16 (correct up to 128).  Thread v of the flat index space owns rewards 4v .. 4v+3;
// a group is `team` = G/4 adjacent lanes of one warp (teams never straddle a warp because the
// warp's first index is a multiple of 32 and team divides 32).  A warp takes kRowUnroll
// consecutive 512-byte rows, a block kRowUnroll * 8 of them, and there is one block per such run
// (blocks that come and go in address order stream better than a resident grid striding through
// memory: 6.2-6.5 against 5.6-5.8 TB/s at G = 8).  Loads and stores carry the streaming hint.
// The mean is taken in fp64 (see inv_scale) and split into a float pair (hi, lo); the deviation
// (x - hi) - lo then carries only fp32 rounding relative to itself -- exactly zero for a group of
// equal rewards.  Squared deviations, root and reciprocal run in fp32 (approximate root and
// reciprocal, ~2 ulp), far inside the tolerance on an advantage of magnitude <= sqrt(G).
constexpr int kRowUnroll = 4;
__global__ void __launch_bounds__(kThreads) advantage_pow2_kernel(
    const float4* __restrict__ reward, float4* __restrict__ adv, int64_t n_vec, int G, float eps, int ddof) {
  const int team = G >> 2;
  const double inv_g = 1.0 / (double)G;                    // exact: G is a power of two
  const float inv_denom = G - ddof > 0 ? 1.f / (float)(G - ddof) : 0.f;
  const int lane = threadIdx.x & 31;
  const int64_t warp_first = ((int64_t)blockIdx.x * blockDim.x + (threadIdx.x & ~31)) * kRowUnroll;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x * kRowUnroll;
  for (int64_t base = warp_first; base < n_vec; base += stride) {   // warp-uniform trip count (one trip unless capped)
    const float4* src = reward + base + lane;
    float4* dst = adv + base + lane;
    const int64_t left = n_vec - base - lane;             // rows u with u * 32 < left exist
    float4 r[kRowUnroll];
#pragma unroll
    for (int u = 0; u < kRowUnroll; ++u) r[u] = u * 32 < left ? __ldcs(src + u * 32) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int u = 0; u < kRowUnroll; ++u) {
      double s = ((double)r[u].x + (double)r[u].y) + ((double)r[u].z + (double)r[u].w);
      for (int o = team >> 1; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      const double mu = s * inv_g;
      const float mu_hi = (float)mu;
      const float mu_lo = (float)(mu - (double)mu_hi);
      const float d0 = (r[u].x - mu_hi) - mu_lo, d1 = (r[u].y - mu_hi) - mu_lo;
      const float d2 = (r[u].z - mu_hi) - mu_lo, d3 = (r[u].w - mu_hi) - mu_lo;
      float q = fmaf(d0, d0, fmaf(d1, d1, fmaf(d2, d2, d3 * d3)));
      for (int o = team >> 1; o > 0; o >>= 1) q += __shfl_xor_sync(0xffffffffu, q, o);
      const float var = q * inv_denom;
      const float sigma = var > 0.f ? var * rsqrtf(var) : 0.f;
      const float inv = __frcp_rn(sigma + eps);
      if (u * 32 < left) __stcs(dst + u * 32, make_float4(d0 * inv, d1 * inv, d2 * inv, d3 * inv));
    }
  }
}

// Power-of-two groups, 32 <= G <= 512.  A thread owns 16 rewards of ONE group (four 128-bit loads),
// a group is `team` = G/16 adjacent lanes, a warp takes 2 KB of consecutive rewards.  Load k of a
// team covers `team` consecutive 16-byte pieces, so every load instruction of the warp asks for
// whole 32-byte sectors only.  Against the kernel above at the same G there are log2(G/16) shuffle
// steps per reduction instead of log2(G/4), once per 16 rewards instead of once per 4, and one root
// and reciprocal per 16 rewards: at G = 64 the issue slots were 66 % busy there.  Arithmetic as above.
__global__ void __launch_bounds__(kThreads) advantage_wide_kernel(
    const float4* __restrict__ reward, float4* __restrict__ adv, int64_t n_vec, int G, float eps, int ddof) {
  constexpr int kVecPerWarp = 128;                          // 32 lanes x 4 float4
  const int team = G >> 4;
  const double inv_g = 1.0 / (double)G;                    // exact: G is a power of two
  const float inv_denom = G - ddof > 0 ? 1.f / (float)(G - ddof) : 0.f;
  const int lane = threadIdx.x & 31;
  const int t = lane & (team - 1), g = lane / team;
  const int64_t warps = (int64_t)gridDim.x * (kThreads / 32);
  for (int64_t wv = ((int64_t)blockIdx.x * (kThreads / 32) + (threadIdx.x >> 5)) * kVecPerWarp; wv < n_vec;
       wv += warps * kVecPerWarp) {                          // warp-uniform trip count
    const int64_t gv = wv + (int64_t)g * (G >> 2) + t;     // this lane's first piece of its group
    const bool live = gv < n_vec;                           // N is a multiple of G: a group is whole or absent
    float4 r[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) r[k] = live ? __ldcs(reward + gv + k * team) : make_float4(0.f, 0.f, 0.f, 0.f);
    double s = 0.0;
#pragma unroll
    for (int k = 0; k < 4; ++k) s += ((double)r[k].x + (double)r[k].y) + ((double)r[k].z + (double)r[k].w);
    for (int o = team >> 1; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    const double mu = s * inv_g;
    const float mu_hi = (float)mu;
    const float mu_lo = (float)(mu - (double)mu_hi);
    float q = 0.f;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      r[k].x = (r[k].x - mu_hi) - mu_lo; r[k].y = (r[k].y - mu_hi) - mu_lo;
      r[k].z = (r[k].z - mu_hi) - mu_lo; r[k].w = (r[k].w - mu_hi) - mu_lo;
      q = fmaf(r[k].x, r[k].x, fmaf(r[k].y, r[k].y, fmaf(r[k].z, r[k].z, fmaf(r[k].w, r[k].w, q))));
    }
    for (int o = team >> 1; o > 0; o >>= 1) q += __shfl_xor_sync(0xffffffffu, q, o);
    const float var = q * inv_denom;
    const float sigma = var > 0.f ? var * rsqrtf(var) : 0.f;
    const float inv = __frcp_rn(sigma + eps);
    if (live) {
#pragma unroll
      for (int k = 0; k < 4; ++k)
        __stcs(adv + gv + k * team, make_float4(r[k].x * inv, r[k].y * inv, r[k].z * inv, r[k].w * inv));
    }
  }
}

// Group sizes below 16 that are not a power of two, known at compile time.  A lane owns
// M = 16 / G whole groups (E = M G rewards); a warp copies 32 E consecutive rewards into its slice
// of shared memory with coalesced 128-bit streaming loads, placing lane l's share at l * (E | 1)
// (an odd stride: the lanes then read and write different banks), works on registers with every
// loop unrolled, and streams the advantages out the same way.  Arithmetic as in the kernels above.
template <int G>
__global__ void __launch_bounds__(kThreads) advantage_fixed_kernel(
    const float* __restrict__ reward, float* __restrict__ adv, int64_t n_groups, float eps, int ddof) {
  constexpr int M = 16 / G, E = M * G, EP = E | 1, CH = 32 * E;
  __shared__ float stage[(kThreads / 32) * 32 * EP];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  float* s = stage + warp * 32 * EP;
  const double inv_g = 1.0 / (double)G;
  const float inv_denom = G - ddof > 0 ? 1.f / (float)(G - ddof) : 0.f;
  const int64_t n_iter = (n_groups + 32 * M - 1) / (32 * M);
  const int64_t warps = (int64_t)gridDim.x * (kThreads / 32);
  for (int64_t it = (int64_t)blockIdx.x * (kThreads / 32) + warp; it < n_iter; it += warps) {
    const int64_t g0 = it * 32 * M;
    const int64_t left = (n_groups - g0) * G;                 // rewards from here to the end
    const int cnt = left < CH ? (int)left : CH;
    const float* src = reward + g0 * G;                       // 128 E bytes per iteration: 16-byte aligned
    float* dst = adv + g0 * G;
    if (cnt == CH) {
#pragma unroll
      for (int i = lane; i < CH / 4; i += 32) {
        const float4 v = __ldcs(reinterpret_cast<const float4*>(src) + i);
        const int f = 4 * i;
        s[(f / E) * EP + f % E] = v.x;
        s[((f + 1) / E) * EP + (f + 1) % E] = v.y;
        s[((f + 2) / E) * EP + (f + 2) % E] = v.z;
        s[((f + 3) / E) * EP + (f + 3) % E] = v.w;
      }
    } else {
      for (int f = lane; f < cnt; f += 32) s[(f / E) * EP + f % E] = __ldcs(src + f);
    }
    __syncwarp();
    float* mine = s + lane * EP;
#pragma unroll
    for (int gi = 0; gi < M; ++gi) {
      if ((int64_t)(lane * M + gi) * G < cnt) {               // this group exists (groups are whole)
        float r[G];
        double sum = 0.0;
#pragma unroll
        for (int k = 0; k < G; ++k) { r[k] = mine[gi * G + k]; sum += (double)r[k]; }
        const double mu = sum * inv_g;
        const float mu_hi = (float)mu;
        const float mu_lo = (float)(mu - (double)mu_hi);
        float q = 0.f;
#pragma unroll
        for (int k = 0; k < G; ++k) { r[k] = (r[k] - mu_hi) - mu_lo; q = fmaf(r[k], r[k], q); }
        const float var = q * inv_denom;
        const float sigma = var > 0.f ? var * rsqrtf(var) : 0.f;
        const float inv = __frcp_rn(sigma + eps);
#pragma unroll
        for (int k = 0; k < G; ++k) mine[gi * G + k] = r[k] * inv;
      }
    }
    __syncwarp();
    if (cnt == CH) {
#pragma unroll
      for (int i = lane; i < CH / 4; i += 32) {
        const int f = 4 * i;
        __stcs(reinterpret_cast<float4*>(dst) + i,
               make_float4(s[(f / E) * EP + f % E], s[((f + 1) / E) * EP + (f + 1) % E],
                           s[((f + 2) / E) * EP + (f + 2) % E], s[((f + 3) / E) * EP + (f + 3) % E]));
      }
    } else {
      for (int f = lane; f < cnt; f += 32) __stcs(dst + f, s[(f / E) * EP + f % E]);
    }
    __syncwarp();                                             // the slice is refilled next
  }
}

template <int G>
void launch_advantage_fixed(const float* reward, float* adv, int64_t n_groups, float eps, int ddof, cudaStream_t s) {
  constexpr int M = 16 / G;
  const int64_t n_iter = (n_groups + 32 * M - 1) / (32 * M);
  int64_t blocks = (n_iter + kThreads / 32 - 1) / (kThreads / 32);
  if (blocks > (int64_t)1 << 30) blocks = (int64_t)1 << 30;
  advantage_fixed_kernel<G><<<(int)blocks, kThreads, 0, s>>>(reward, adv, n_groups, eps, ddof);
}

// Any group size up to 512 (used for 16 < G <= 512 that are not a power of two).  A warp copies
// a run of whole groups -- 32 / team of them, at most 512 rewards -- into its own slice of shared
// memory with coalesced 128-bit streaming loads, `team` adjacent lanes (a power of two, at most 16
// rewards per lane) take one group each from there into registers, do the arithmetic of the
// kernels above and put the advantages back, and the warp streams the slice out again.  Only
// __syncwarp: warps do not wait for one another.
constexpr int kWarpStage = 512;          // rewards per warp slice
constexpr int kAnyPerLane = 16;
template <bool kLanePerGroup>             // team == 1
__global__ void __launch_bounds__(kThreads, 4) advantage_any_kernel(
    const float* __restrict__ reward, float* __restrict__ adv, int64_t n_groups, int G, int team, float eps, int ddof) {
  __shared__ __align__(16) float stage[(kThreads / 32) * kWarpStage];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  float* s = stage + warp * kWarpStage;
  const int gw = 32 / team;                                   // groups per warp iteration
  const int g = lane / team, t = lane & (team - 1);
  const int chunk = gw * G;                                   // <= kWarpStage
  const bool vec = (chunk & 3) == 0;                          // every full chunk then starts 16-byte aligned
  const double inv_g = 1.0 / (double)G;
  const float inv_denom = G - ddof > 0 ? 1.f / (float)(G - ddof) : 0.f;
  // one lane per group and an even G: lanes would read the same bank; start each lane's walk
  // through its group at a different element instead
  const int rot = (kLanePerGroup && (G & 1) == 0) ? g % G : 0;
  // element i of this lane's share of its group: its position in the group, or -1
  auto pos = [&](int i, bool live) -> int {
    int j;
    bool ok;
    if (kLanePerGroup) { j = i + rot; if (j >= G) j -= G; ok = i < G; }
    else { j = t + i * team; ok = j < G; }
    return ok && live ? j : -1;
  };
  const int64_t n_iter = (n_groups + gw - 1) / gw;
  const int64_t warps = (int64_t)gridDim.x * (kThreads / 32);
  for (int64_t it = (int64_t)blockIdx.x * (kThreads / 32) + warp; it < n_iter; it += warps) {
    const int64_t g0 = it * gw;
    const int ng = (int)((n_groups - g0) < gw ? (n_groups - g0) : gw);
    const int cnt = ng * G;
    const float* src = reward + g0 * G;
    float* dst = adv + g0 * G;
    if (vec && cnt == chunk) {
      for (int i = lane; i < (chunk >> 2); i += 32)
        reinterpret_cast<float4*>(s)[i] = __ldcs(reinterpret_cast<const float4*>(src) + i);
    } else {
      for (int i = lane; i < cnt; i += 32) s[i] = __ldcs(src + i);
    }
    __syncwarp();
    const bool live = g < ng;
    float* mine = s + g * G;
    float r[kAnyPerLane];
    double sum = 0.0;
#pragma unroll
    for (int i = 0; i < kAnyPerLane; ++i) {
      const int j = pos(i, live);
      r[i] = j >= 0 ? mine[j] : 0.f;
      sum += (double)r[i];
    }
    for (int o = team >> 1; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    const double mu = sum * inv_g;
    const float mu_hi = (float)mu;
    const float mu_lo = (float)(mu - (double)mu_hi);
    float q = 0.f;
#pragma unroll
    for (int i = 0; i < kAnyPerLane; ++i) {
      r[i] = pos(i, live) >= 0 ? (r[i] - mu_hi) - mu_lo : 0.f;
      q = fmaf(r[i], r[i], q);
    }
    for (int o = team >> 1; o > 0; o >>= 1) q += __shfl_xor_sync(0xffffffffu, q, o);
    const float var = q * inv_denom;
    const float sigma = var > 0.f ? var * rsqrtf(var) : 0.f;
    const float inv = __frcp_rn(sigma + eps);
#pragma unroll
    for (int i = 0; i < kAnyPerLane; ++i) {
      const int j = pos(i, live);
      if (j >= 0) mine[j] = r[i] * inv;
    }
    __syncwarp();
    if (vec && cnt == chunk) {
      for (int i = lane; i < (chunk >> 2); i += 32)
        __stcs(reinterpret_cast<float4*>(dst) + i, reinterpret_cast<const float4*>(s)[i]);
    } else {
      for (int i = lane; i < cnt; i += 32) __stcs(dst + i, s[i]);
    }
    __syncwarp();                                             // the slice is refilled next
  }
}

// Groups of equal size G, G <= kStage: each block iteration owns `gpb` whole groups.
__global__ void __launch_bounds__(kThreads) advantage_contiguous_kernel(
    const float* __restrict__ reward, float* __restrict__ adv, int64_t n_groups, int G, int gpb,
    float eps, int ddof) {
  __shared__ __align__(16) float sr[kStage];
  __shared__ double s_mu[kMaxGroupsStaged];   // per staged group
  __shared__ double s_inv[kMaxGroupsStaged];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  // team of lanes per group: smallest power of two >= G, capped at a warp
  int team = 1;
  while (team < G && team < 32) team <<= 1;
  const int teams_per_warp = 32 / team;
  const int64_t n_iter = (n_groups + gpb - 1) / gpb;
  for (int64_t it = blockIdx.x; it < n_iter; it += gridDim.x) {
    const int64_t g0 = it * gpb;
    const int ng = (int)((n_groups - g0) < gpb ? (n_groups - g0) : gpb);
    const int64_t base = g0 * G;
    const int cnt = ng * G;
    // stage: vector loads when the run is 16-byte aligned
    if (((base & 3) == 0) && ((reinterpret_cast<uintptr_t>(reward) & 15) == 0)) {
      const float4* r4 = reinterpret_cast<const float4*>(reward + base);
      for (int i = threadIdx.x; i < (cnt >> 2); i += kThreads)
        reinterpret_cast<float4*>(sr)[i] = __ldg(r4 + i);
      for (int i = (cnt & ~3) + threadIdx.x; i < cnt; i += kThreads) sr[i] = __ldg(reward + base + i);
    } else {
      for (int i = threadIdx.x; i < cnt; i += kThreads) sr[i] = __ldg(reward + base + i);
    }
    __syncthreads();
    if (G == 1) {
      for (int i = threadIdx.x; i < cnt; i += kThreads) adv[base + i] = 0.f;  // (r - r) / (0 + eps)
      __syncthreads();
      continue;
    }
    // statistics: one team of lanes per group
    const int teams = (kThreads / 32) * teams_per_warp;
    for (int gl = warp * teams_per_warp + lane / team; gl - (lane / team) < ng; gl += teams) {
      // all lanes of the warp iterate together; lanes of a team past the end idle with zeros
      const bool live = gl < ng;
      const int tl = lane % team;
      double s = 0.0;
      if (live) for (int k = tl; k < G; k += team) s += (double)sr[gl * G + k];
      s = team_sum(s, team);
      const double mu = s / (double)G;
      double q = 0.0;
      if (live) for (int k = tl; k < G; k += team) { const double dv = (double)sr[gl * G + k] - mu; q += dv * dv; }
      q = team_sum(q, team);
      if (live && tl == 0) { s_mu[gl] = mu; s_inv[gl] = inv_scale(q, G, ddof, eps); }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < cnt; i += kThreads) {
      const int gl = i / G;
      adv[base + i] = (float)(((double)sr[i] - s_mu[gl]) * s_inv[gl]);
    }
    __syncthreads();
  }
}

__device__ double block_sum(double v, double* scratch) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  v = warp_sum(v);
  __syncthreads();
  if (lane == 0) scratch[warp] = v;
  __syncthreads();
  double t = 0.0;
  for (int w = 0; w < kThreads / 32; ++w) t += scratch[w];  // fixed order, same in every thread
  return t;
}

// One block per group: members are where group_id == g (or the contiguous range when ids is NULL
// and the group is too large to stage).
__global__ void __launch_bounds__(kThreads) advantage_scan_kernel(
    const float* __restrict__ reward, const int32_t* __restrict__ ids, float* __restrict__ adv,
    int64_t N, int64_t G_contig, float eps, int ddof) {
  __shared__ double scratch[kThreads / 32];
  const int g = blockIdx.x;
  const int64_t lo = ids ? 0 : (int64_t)g * G_contig;
  const int64_t hi = ids ? N : lo + G_contig;
  double s = 0.0, c = 0.0;
  for (int64_t i = lo + threadIdx.x; i < hi; i += kThreads)
    if (!ids || __ldg(ids + i) == g) { s += (double)__ldg(reward + i); c += 1.0; }
  const double n = block_sum(c, scratch);
  const double tot = block_sum(s, scratch);
  if (n == 0.0) return;
  const double mu = tot / n;
  double q = 0.0;
  for (int64_t i = lo + threadIdx.x; i < hi; i += kThreads)
    if (!ids || __ldg(ids + i) == g) { const double dv = (double)__ldg(reward + i) - mu; q += dv * dv; }
  const double ssq = block_sum(q, scratch);
  const double inv = inv_scale(ssq, (int64_t)n, ddof, eps);
  for (int64_t i = lo + threadIdx.x; i < hi; i += kThreads)
    if (!ids || __ldg(ids + i) == g) adv[i] = (float)(((double)__ldg(reward + i) - mu) * inv);
}

}  // namespace

cudaError_t launch_advantage(const float* reward, int64_t N, int32_t n_groups, float eps_adv, int32_t ddof,
                             float* adv, int sm_count, cudaStream_t s) {
  if (N == 0 || n_groups == 0) return cudaSuccess;
  {
    const int64_t G = N / n_groups;
    const bool aligned = ((reinterpret_cast<uintptr_t>(reward) | reinterpret_cast<uintptr_t>(adv)) & 15) == 0;
    if (G >= 32 && G <= 512 && (G & (G - 1)) == 0 && aligned) {
      const int64_t n_vec = N / 4;
      int64_t blocks = (n_vec + (int64_t)kThreads * 4 - 1) / ((int64_t)kThreads * 4);   // 16 KB of rewards per block
      if (blocks > (int64_t)1 << 30) blocks = (int64_t)1 << 30;
      advantage_wide_kernel<<<(int)blocks, kThreads, 0, s>>>(reinterpret_cast<const float4*>(reward),
                                                             reinterpret_cast<float4*>(adv), n_vec, (int)G,
                                                             eps_adv, ddof);
    } else if (G >= 4 && G <= 16 && (G & (G - 1)) == 0 && aligned) {
      const int64_t n_vec = N / 4;
      int64_t blocks = (n_vec + (int64_t)kThreads * kRowUnroll - 1) / ((int64_t)kThreads * kRowUnroll);
      if (blocks > (int64_t)1 << 30) blocks = (int64_t)1 << 30;
      advantage_pow2_kernel<<<(int)blocks, kThreads, 0, s>>>(reinterpret_cast<const float4*>(reward),
                                                             reinterpret_cast<float4*>(adv), n_vec, (int)G,
                                                             eps_adv, ddof);
    } else if (aligned && (G == 3 || (G >= 5 && G <= 7) || (G >= 9 && G <= 15))) {
      switch ((int)G) {
        case 3: launch_advantage_fixed<3>(reward, adv, n_groups, eps_adv, ddof, s); break;
        case 5: launch_advantage_fixed<5>(reward, adv, n_groups, eps_adv, ddof, s); break;
        case 6: launch_advantage_fixed<6>(reward, adv, n_groups, eps_adv, ddof, s); break;
        case 7: launch_advantage_fixed<7>(reward, adv, n_groups, eps_adv, ddof, s); break;
        case 9: launch_advantage_fixed<9>(reward, adv, n_groups, eps_adv, ddof, s); break;
        case 10: launch_advantage_fixed<10>(reward, adv, n_groups, eps_adv, ddof, s); break;
        case 11: launch_advantage_fixed<11>(reward, adv, n_groups, eps_adv, ddof, s); break;
        case 12: launch_advantage_fixed<12>(reward, adv, n_groups, eps_adv, ddof, s); break;
        case 13: launch_advantage_fixed<13>(reward, adv, n_groups, eps_adv, ddof, s); break;
        case 14: launch_advantage_fixed<14>(reward, adv, n_groups, eps_adv, ddof, s); break;
        default: launch_advantage_fixed<15>(reward, adv, n_groups, eps_adv, ddof, s); break;
      }
    } else if (G > 16 && G <= 512 && aligned) {
      // (smaller groups fill too little of a warp's slice: one thread per group is faster there)
      int team = 1;
      while (team * kAnyPerLane < G) team <<= 1;                     // 1, 2, 4, ... 32
      const int64_t n_iter = (n_groups + 32 / team - 1) / (32 / team);
      int64_t blocks = (n_iter + kThreads / 32 - 1) / (kThreads / 32);
      if (blocks > (int64_t)1 << 30) blocks = (int64_t)1 << 30;
      if (team == 1)
        advantage_any_kernel<true><<<(int)blocks, kThreads, 0, s>>>(reward, adv, n_groups, (int)G, team, eps_adv, ddof);
      else
        advantage_any_kernel<false><<<(int)blocks, kThreads, 0, s>>>(reward, adv, n_groups, (int)G, team, eps_adv, ddof);
    } else if (G >= 1 && G <= kSmallG) {
      const int vec_ok = (G % 4 == 0) && ((reinterpret_cast<uintptr_t>(reward) & 15) == 0) &&
                         ((reinterpret_cast<uintptr_t>(adv) & 15) == 0);
      int64_t blocks = (n_groups + kThreads - 1) / kThreads;
      if (blocks > (int64_t)sm_count * 8) blocks = (int64_t)sm_count * 8;
      if (G <= 4)
        advantage_small_group_kernel<4><<<(int)blocks, kThreads, 0, s>>>(reward, adv, n_groups, (int)G, eps_adv, ddof, vec_ok);
      else if (G <= 8)
        advantage_small_group_kernel<8><<<(int)blocks, kThreads, 0, s>>>(reward, adv, n_groups, (int)G, eps_adv, ddof, vec_ok);
      else if (G <= 16)
        advantage_small_group_kernel<16><<<(int)blocks, kThreads, 0, s>>>(reward, adv, n_groups, (int)G, eps_adv, ddof, vec_ok);
      else
        advantage_small_group_kernel<32><<<(int)blocks, kThreads, 0, s>>>(reward, adv, n_groups, (int)G, eps_adv, ddof, vec_ok);
    } else if (G <= kStage && G >= 1) {
      int gpb = (int)(kStage / G);
      // keep every SM busy before making block iterations large
      const int64_t want = (n_groups + (int64_t)sm_count * 4 - 1) / ((int64_t)sm_count * 4);
      if (gpb > want) gpb = (int)(want > 0 ? want : 1);
      if (gpb > kMaxGroupsStaged) gpb = kMaxGroupsStaged;
      int64_t iters = (n_groups + gpb - 1) / gpb;
      int blocks = (int)(iters < (int64_t)sm_count * 8 ? iters : (int64_t)sm_count * 8);
      advantage_contiguous_kernel<<<blocks, kThreads, 0, s>>>(reward, adv, n_groups, (int)G, gpb,
                                                              eps_adv, ddof);
    } else {
      advantage_scan_kernel<<<n_groups, kThreads, 0, s>>>(reward, nullptr, adv, N, G, eps_adv, ddof);
    }
  }
  return cudaGetLastError();
}

}  // namespace af
