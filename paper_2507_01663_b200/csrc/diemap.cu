// Which SMs share a die (and with it a half of L2)?  Measured once per context, not assumed: the SM
// ids of a B200 interleave the two dies irregularly and the dies need not have the same number of
// SMs enabled.
//
// One block per SM times a chain of dependent L2 loads (ld.global.cg, the line warmed first) for
// each of kAddr addresses about a megabyte apart.  An address lives in one half of L2; SMs of that
// die see it some 35-40 cycles sooner than SMs of the other.  Centred per address over all SMs, two
// SMs of the same die have latency vectors that point the same way, two SMs of different dies
// opposite ways: the sign of the dot product with one reference SM splits the SMs into the dies.
#include <algorithm>
#include <cmath>
#include <vector>

#include "common.cuh"

namespace af {
namespace {

constexpr int kAddr = 32, kChain = 48, kMaxSmid = 256;
constexpr size_t kStrideWords = (1u << 20) / 4 + 64;
constexpr int kProbeSmem = 200 * 1024;     // so that two blocks cannot share an SM

__global__ void __launch_bounds__(32) die_probe_kernel(const unsigned* buf, unsigned* started, int n_blocks,
                                                       unsigned* out_smid, unsigned* out_lat) {
  if (threadIdx.x != 0) return;
  unsigned smid;
  asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
  out_smid[blockIdx.x] = smid;
  // keep the block resident until all have started (so that every SM hosts one), but never for long
  atomicAdd(started, 1u);
  for (int spin = 0; spin < 20000; ++spin) {
    unsigned seen;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(started) : "memory");
    if (seen >= (unsigned)n_blocks) break;
    __nanosleep(100);
  }
  for (int k = 0; k < kAddr; ++k) {
    const unsigned* p = buf + (size_t)k * kStrideWords;
    unsigned off = 0;
    for (int r = 0; r < 8; ++r) {
      unsigned x;
      asm volatile("ld.global.cg.u32 %0, [%1];" : "=r"(x) : "l"(p + off) : "memory");
      off = x;                                     // the buffer holds zeros: the chain stays on its line
    }
    unsigned best = 0xffffffffu;
    for (int rep = 0; rep < 3; ++rep) {              // the quietest of three chains
      const long long t0 = clock64();
      for (int r = 0; r < kChain; ++r) {
        unsigned x;
        asm volatile("ld.global.cg.u32 %0, [%1];" : "=r"(x) : "l"(p + off) : "memory");
        off = x;
      }
      const long long t1 = clock64();
      const unsigned dt = (unsigned)(t1 - t0);
      best = dt < best ? dt : best;
    }
    out_lat[blockIdx.x * kAddr + k] = best + off;
  }
}

}  // namespace

namespace {
// One measurement.  Returns 0 and fills `table` / *die0_sms, or the reason it is not clear-cut:
// 1 a CUDA call failed, 2 an SM id out of range or seen twice, 3 an SM between the two groups,
// 4 an SM pair straddling the dies, 5 a lopsided split.
int measure_once(int sm_count, std::vector<unsigned char>& table, int* die0_sms) {
  unsigned *buf = nullptr, *scratch = nullptr;
  const size_t buf_bytes = (size_t)kAddr * kStrideWords * 4 + 4096;
  const size_t scratch_words = 1 + (size_t)sm_count * (1 + kAddr);
  bool ok = false;
  std::vector<unsigned> host(scratch_words);
  do {
    if (cudaMalloc(&buf, buf_bytes) != cudaSuccess || cudaMalloc(&scratch, scratch_words * 4) != cudaSuccess) break;
    if (cudaMemset(buf, 0, buf_bytes) != cudaSuccess || cudaMemset(scratch, 0, scratch_words * 4) != cudaSuccess) break;
    if (cudaFuncSetAttribute(die_probe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kProbeSmem) != cudaSuccess) break;
    die_probe_kernel<<<sm_count, 32, kProbeSmem>>>(buf, scratch, sm_count, scratch + 1, scratch + 1 + sm_count);
    if (cudaDeviceSynchronize() != cudaSuccess) break;
    if (cudaMemcpy(host.data(), scratch, scratch_words * 4, cudaMemcpyDeviceToHost) != cudaSuccess) break;
    ok = true;
  } while (false);
  if (buf) cudaFree(buf);
  if (scratch) cudaFree(scratch);
  if (!ok) { cudaGetLastError(); return 1; }

  const unsigned* smid = host.data() + 1;
  const unsigned* lat = host.data() + 1 + sm_count;
  // every SM id below kMaxSmid, each seen once
  std::vector<int> block_of(kMaxSmid, -1);
  for (int b = 0; b < sm_count; ++b) {
    if (smid[b] >= (unsigned)kMaxSmid || block_of[smid[b]] >= 0) return 2;
    block_of[smid[b]] = b;
  }
  std::vector<double> mean(kAddr, 0.0);
  for (int k = 0; k < kAddr; ++k) {
    for (int b = 0; b < sm_count; ++b) mean[k] += lat[b * kAddr + k];
    mean[k] /= sm_count;
  }
  // cosine between every SM's centred latency vector and the first block's: same die > 0, other die < 0
  std::vector<double> dot(sm_count);
  double norm0 = 0.0, weakest = 1.0;
  for (int k = 0; k < kAddr; ++k) norm0 += (lat[k] - mean[k]) * (lat[k] - mean[k]);
  for (int b = 0; b < sm_count; ++b) {
    double s = 0.0, nb = 0.0;
    for (int k = 0; k < kAddr; ++k) {
      const double zb = lat[b * kAddr + k] - mean[k];
      s += zb * (lat[k] - mean[k]);
      nb += zb * zb;
    }
    if (!(nb > 0.0) || !(norm0 > 0.0)) return 3;
    dot[b] = s / std::sqrt(nb * norm0);
    weakest = std::min(weakest, std::fabs(dot[b]));
  }
  if (weakest < 0.15) return 3;                              // some SM sits between the two groups: no clear split
  table.assign(kMaxSmid, 0);
  int n0 = 0;
  for (int b = 0; b < sm_count; ++b) {
    const unsigned char die = dot[b] > 0.0 ? 0 : 1;          // die 0 = the die of the first block's SM
    table[smid[b]] = die;
    n0 += die == 0;
  }
  // SM pairs (ids 2k, 2k+1) host CTA pairs: they must not straddle the dies, and both dies must be there
  for (int k = 0; 2 * k + 1 < kMaxSmid; ++k)
    if (block_of[2 * k] >= 0 && block_of[2 * k + 1] >= 0 && table[2 * k] != table[2 * k + 1]) return 4;
  if (n0 % 2 != 0 || n0 < sm_count / 4 || n0 > 3 * sm_count / 4) return 5;
  *die0_sms = n0;
  return 0;
}
}  // namespace

// Fills table[smid] = 0 / 1 (device, kMaxSmid bytes) and *die0_sms.  The measurement is repeated a few
// times if it does not come out clear-cut (another process on the GPU, a profiler's instrumentation);
// if it never does, returns false with *reason set (table untouched) and the caller deals the work
// without regard to dies.
bool measure_die_map(int sm_count, unsigned char* d_table, int* die0_sms, int* reason) {
  *die0_sms = 0;
  *reason = 1;
  if (sm_count < 4 || sm_count > kMaxSmid) return false;
  try {
    std::vector<unsigned char> table;
    for (int attempt = 0; attempt < 4; ++attempt) {
      int n0 = 0;
      *reason = measure_once(sm_count, table, &n0);
      if (*reason != 0) continue;
      if (cudaMemcpy(d_table, table.data(), kMaxSmid, cudaMemcpyHostToDevice) != cudaSuccess) { cudaGetLastError(); *reason = 1; return false; }
      *die0_sms = n0;
      return true;
    }
  } catch (...) {       // host allocation failed: no exception may reach the C boundary
    *reason = 1;
  }
  return false;
}

}  // namespace af
