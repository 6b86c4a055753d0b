// af_grpo_advantage with arbitrary group membership (group_id given): O(N) work whatever the
// number of groups, and bit-reproducible although the members of a group are met in no fixed
// order.
//
// A group's statistics are accumulated with INTEGER atomics on exact fixed-point values, so the
// sums do not depend on the order in which the atomics land:
//   pass 1  count_g and M_g = max |r_i| of every group (atomicAdd / atomicMax on the float's bits);
//   pass 2  S_g = sum_i k_i with k_i = round(r_i 2^(60 - e_g)), 2^e_g the power of two above M_g
//           (|k_i| <= 2^60; exact for every reward within 2^-37 of the group's largest), in 128 bits;
//   pass 3  Q_g = sum_i round(D_i^2 2^-(2 b_g - 90)) with D_i = n_g k_i - S_g (n_g times the
//           deviation from the mean, an exact integer: 0 for a group of equal rewards) and
//           2^b_g > |D_i|, again in 128 bits -- at least 40 significant bits are left even when a
//           group's rewards differ only in their last fp32 bits;
//   finish  per group: sigma from Q_g, then the factor that turns D_i into an advantage;
//   pass 4  adv_i = D_i * factor_g.
// A 128-bit sum is two 64-bit atomics (the low word's carry goes to the high word); the lanes of a
// warp that hold the same group first combine their values, so a batch made of a few huge groups
// issues one pair of atomics per warp, not per sample.  Every pass streams ids and rewards once
// (8 B per sample, 12 B in the last): 36 B per sample in all.
// An id outside [0, n_groups) gets a NaN advantage and raises AF_DEVERR_GROUP_ID.
#include <math.h>

#include "common.cuh"

namespace af {
namespace {

constexpr int kThreads = 256;

struct __align__(16) GroupAcc {
  unsigned int count;
  unsigned int max_bits;        // bits of max |r| (order-preserving for non-negative floats)
  unsigned long long s_lo, s_hi;  // S_g, two's complement
  unsigned long long q_lo, q_hi;  // Q_g
  double factor;                // adv_i = D_i * factor  (written by the finishing kernel)
  double pad[2];
};
static_assert(sizeof(GroupAcc) == 64, "one accumulator per 64-byte sector pair");

typedef __int128 i128;
typedef unsigned __int128 u128;

__device__ __forceinline__ void atomic_add128(unsigned long long* lo, unsigned long long* hi, u128 v) {
  const unsigned long long vlo = (unsigned long long)v, vhi = (unsigned long long)(v >> 64);
  const unsigned long long old = atomicAdd(lo, vlo);
  const unsigned long long carry = (old + vlo < old) ? 1ull : 0ull;      // the low word wrapped
  if (vhi + carry) atomicAdd(hi, vhi + carry);
}

// Sum of a non-negative 62-bit value over the lanes in `peers` (all of which call this together).
__device__ __forceinline__ u128 peers_sum62(unsigned peers, unsigned long long v) {
  const unsigned l0 = __reduce_add_sync(peers, (unsigned)(v & 0x1FFFFFu));
  const unsigned l1 = __reduce_add_sync(peers, (unsigned)((v >> 21) & 0x1FFFFFu));
  const unsigned l2 = __reduce_add_sync(peers, (unsigned)(v >> 42));
  return (u128)l0 + ((u128)l1 << 21) + ((u128)l2 << 42);
}
// The same for a value below 2^90 given as (hi < 2^26, lo).
__device__ __forceinline__ u128 peers_sum90(unsigned peers, unsigned long long hi, unsigned long long lo) {
  u128 s = peers_sum62(peers, lo & 0x3FFFFFFFFFFFFFFFull);
  s += (u128)__reduce_add_sync(peers, (unsigned)(lo >> 62)) << 62;
  s += (u128)__reduce_add_sync(peers, (unsigned)hi) << 64;
  return s;
}

__device__ __forceinline__ double to_double(i128 v) {
  const bool neg = v < 0;
  const u128 m = neg ? (u128)(-v) : (u128)v;
  const double d = (double)(unsigned long long)(m >> 64) * 18446744073709551616.0 + (double)(unsigned long long)m;
  return neg ? -d : d;
}

// exponent e with |r| < 2^e for every member, from the bits of the group's largest |r|
__device__ __forceinline__ int scale_exponent(unsigned int max_bits) { return ilogbf(__uint_as_float(max_bits)) + 1; }
__device__ __forceinline__ bool finite_positive(unsigned int max_bits) {
  return max_bits != 0u && max_bits < 0x7F800000u;
}
__device__ __forceinline__ long long fixed_point(float r, int e) { return __double2ll_rn(scalbn((double)r, 60 - e)); }
__device__ __forceinline__ int ceil_log2(unsigned int n) { return n <= 1 ? 0 : 32 - __clz(n - 1); }

__global__ void __launch_bounds__(kThreads) adv_ids_count_kernel(
    const float* __restrict__ reward, const int32_t* __restrict__ ids, int64_t N, int n_groups, GroupAcc* acc,
    unsigned int* d_err) {
  const int64_t stride = (int64_t)gridDim.x * kThreads;
  for (int64_t base = (int64_t)blockIdx.x * kThreads; base < N; base += stride) {
    const int64_t i = base + threadIdx.x;
    const bool in = i < N;
    const int g = in ? __ldg(ids + i) : -1;
    const bool ok = in && g >= 0 && g < n_groups;
    if (in && !ok) atomicOr(d_err, AF_DEVERR_GROUP_ID);
    const unsigned bits = ok ? __float_as_uint(fabsf(__ldg(reward + i))) : 0u;
    const unsigned live = __ballot_sync(0xffffffffu, ok);
    if (!ok) continue;
    const unsigned peers = __match_any_sync(live, g);
    const unsigned mx = __reduce_max_sync(peers, bits);
    if ((int)(threadIdx.x & 31) == __ffs(peers) - 1) {
      atomicAdd(&acc[g].count, (unsigned)__popc(peers));
      atomicMax(&acc[g].max_bits, mx);
    }
  }
}

__global__ void __launch_bounds__(kThreads) adv_ids_sum_kernel(
    const float* __restrict__ reward, const int32_t* __restrict__ ids, int64_t N, int n_groups, GroupAcc* acc) {
  const int64_t stride = (int64_t)gridDim.x * kThreads;
  for (int64_t base = (int64_t)blockIdx.x * kThreads; base < N; base += stride) {
    const int64_t i = base + threadIdx.x;
    const int g = i < N ? __ldg(ids + i) : -1;
    const bool ok = g >= 0 && g < n_groups;
    const unsigned live = __ballot_sync(0xffffffffu, ok);
    if (!ok) continue;
    const unsigned mb = __ldg(&acc[g].max_bits);
    const unsigned peers = __match_any_sync(live, g);
    if (!finite_positive(mb)) continue;                       // all zero (nothing to add) or not finite
    const long long k = fixed_point(__ldg(reward + i), scale_exponent(mb));
    // shift into [0, 2^61] for the unsigned lane sums, take the shift out again afterwards
    const u128 sum = peers_sum62(peers, (unsigned long long)(k + (1ll << 60)));
    if ((int)(threadIdx.x & 31) == __ffs(peers) - 1) {
      const i128 s = (i128)sum - ((i128)__popc(peers) << 60);
      atomic_add128(&acc[g].s_lo, &acc[g].s_hi, (u128)s);
    }
  }
}

// What the later passes read of a group (fields no kernel is still adding to).
struct GroupSums {
  unsigned int count, max_bits;
  unsigned long long s_lo, s_hi;
};
__device__ __forceinline__ GroupSums load_sums(const GroupAcc* acc, int g) {
  const uint2 cm = __ldg(reinterpret_cast<const uint2*>(&acc[g].count));
  return GroupSums{cm.x, cm.y, __ldg(&acc[g].s_lo), __ldg(&acc[g].s_hi)};
}
__device__ __forceinline__ i128 deviation_times_n(const GroupSums& a, float r) {
  const i128 S = (i128)(((u128)a.s_hi << 64) | (u128)a.s_lo);
  return (i128)a.count * (i128)fixed_point(r, scale_exponent(a.max_bits)) - S;
}

__global__ void __launch_bounds__(kThreads) adv_ids_sumsq_kernel(
    const float* __restrict__ reward, const int32_t* __restrict__ ids, int64_t N, int n_groups, GroupAcc* acc) {
  const int64_t stride = (int64_t)gridDim.x * kThreads;
  for (int64_t base = (int64_t)blockIdx.x * kThreads; base < N; base += stride) {
    const int64_t i = base + threadIdx.x;
    const int g = i < N ? __ldg(ids + i) : -1;
    const bool ok = g >= 0 && g < n_groups;
    const unsigned live = __ballot_sync(0xffffffffu, ok);
    if (!ok) continue;
    const GroupSums a = load_sums(acc, g);
    const unsigned peers = __match_any_sync(live, g);
    if (!finite_positive(a.max_bits)) continue;
    const double x = to_double(deviation_times_n(a, __ldg(reward + i)));      // |x| < 2^b
    const int b = ceil_log2(a.count) + 61;
    const double u = rint(scalbn(x * x, 90 - 2 * b));                           // integer-valued, < 2^90
    const unsigned long long hi = (unsigned long long)(u * (1.0 / 18446744073709551616.0));
    const unsigned long long lo = (unsigned long long)(u - (double)hi * 18446744073709551616.0);
    const u128 sum = peers_sum90(peers, hi, lo);
    if ((int)(threadIdx.x & 31) == __ffs(peers) - 1) atomic_add128(&acc[g].q_lo, &acc[g].q_hi, sum);
  }
}

// Per group: sigma = sqrt(sum dev^2 / (n - ddof)) with dev_i = D_i / (n 2^(60-e)), and the factor
// 1 / ((sigma + eps) n 2^(60-e)) that turns D_i into the advantage.
__global__ void __launch_bounds__(kThreads) adv_ids_finish_kernel(GroupAcc* acc, int n_groups, float eps, int ddof) {
  const int g = blockIdx.x * kThreads + threadIdx.x;
  if (g >= n_groups) return;
  GroupAcc a = acc[g];
  double factor = 0.0;                                          // empty or all-zero group: advantages 0
  if (a.count > 0 && a.max_bits >= 0x7F800000u) {
    factor = __longlong_as_double(0x7FF8000000000000ll);        // a reward is inf or NaN
  } else if (a.count > 0 && a.max_bits != 0u) {
    const int e = scale_exponent(a.max_bits), b = ceil_log2(a.count) + 61;
    const double n = (double)a.count;
    const double unit = scalbn(1.0 / n, e - 60);                // one unit of D_i as a reward difference
    const double Q = (double)a.q_hi * 18446744073709551616.0 + (double)a.q_lo;
    const double ssq = scalbn(Q, 2 * b - 90) * unit * unit;     // sum of squared deviations
    const long long denom = (long long)a.count - ddof;
    const double sigma = denom > 0 ? sqrt(ssq / (double)denom) : 0.0;
    factor = unit / (sigma + (double)eps);
  }
  acc[g].factor = factor;
}

__global__ void __launch_bounds__(kThreads) adv_ids_write_kernel(
    const float* __restrict__ reward, const int32_t* __restrict__ ids, int64_t N, int n_groups,
    const GroupAcc* __restrict__ acc, float* __restrict__ adv) {
  const int64_t stride = (int64_t)gridDim.x * kThreads;
  for (int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x; i < N; i += stride) {
    const int g = __ldg(ids + i);
    if (g < 0 || g >= n_groups) { adv[i] = __int_as_float(0x7fc00000); continue; }
    const GroupSums a = load_sums(acc, g);
    float out = 0.f;
    if (a.max_bits >= 0x7F800000u) out = __int_as_float(0x7fc00000);
    else if (a.max_bits != 0u) out = (float)(to_double(deviation_times_n(a, __ldg(reward + i))) * __ldg(&acc[g].factor));
    adv[i] = out;
  }
}

}  // namespace

size_t advantage_ids_workspace_bytes(int32_t n_groups) { return (size_t)(n_groups > 0 ? n_groups : 1) * sizeof(GroupAcc); }

cudaError_t launch_advantage_ids(const float* reward, const int32_t* group_id, int64_t N, int32_t n_groups,
                                 float eps_adv, int32_t ddof, float* adv, void* ws, unsigned int* d_err,
                                 int sm_count, cudaStream_t s) {
  GroupAcc* acc = static_cast<GroupAcc*>(ws);
  cudaError_t e = cudaMemsetAsync(acc, 0, (size_t)n_groups * sizeof(GroupAcc), s);
  if (e != cudaSuccess) return e;
  int64_t want = (N + kThreads - 1) / kThreads;
  const int grid = (int)(want < (int64_t)sm_count * 16 ? want : (int64_t)sm_count * 16);
  adv_ids_count_kernel<<<grid, kThreads, 0, s>>>(reward, group_id, N, n_groups, acc, d_err);
  adv_ids_sum_kernel<<<grid, kThreads, 0, s>>>(reward, group_id, N, n_groups, acc);
  adv_ids_sumsq_kernel<<<grid, kThreads, 0, s>>>(reward, group_id, N, n_groups, acc);
  adv_ids_finish_kernel<<<(n_groups + kThreads - 1) / kThreads, kThreads, 0, s>>>(acc, n_groups, eps_adv, ddof);
  adv_ids_write_kernel<<<grid, kThreads, 0, s>>>(reward, group_id, N, n_groups, acc, adv);
  return cudaGetLastError();
}

}  // namespace af
