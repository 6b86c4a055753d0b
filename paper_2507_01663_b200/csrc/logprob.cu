// af_token_logprob: LM-head GEMM (tcgen05 / TMEM, TMA-fed) with the online log-softmax, target
// pick and entropy sums fused into its epilogue, so the [T,V] logits never leave the SM.
//
// Each epilogue thread owns one token row.  Sweeping the vocabulary tiles of its unit it keeps
//   m = running max,  s = sum exp(z - m),  u = sum exp(z - m) * z,  zy = z at the target
// in registers.  A unit covers one of S vocabulary ranges; the S partial states of a token are
// written to the workspace and combined by merge_partials_kernel:
//   lse = M + log sum_i s_i e^{m_i - M},  logp = zy - lse,  entropy = lse - (sum_i u_i e^{m_i-M}) / S.
#include <mutex>

#include "device_util.cuh"
#include "gemm_launch.cuh"

namespace af {
namespace {



// kStoreZ: also write the fp32 logits of the tile to z [T, ldz] (one token block of the fused actor
// update, which turns them into dZ without a second GEMM).
template <bool kStoreZ>
struct LogprobEpiT {
  struct Params {
    const int32_t* target;  // [T]
    float4* partial;        // [S, T]
    int T, V;
    int v_offset;           // vocabulary id of W's first row (0 unless W is one shard of the head)
    float* z;               // [T, ldz] fp32 logits (kStoreZ only)
    int64_t ldz;
  };
  struct State {
    float m, s, u, zy;
    int y;
  };
  static constexpr bool kStaged = false;   // nothing is stored per tile: no staging buffer needed
  static __device__ __forceinline__ void unit_begin(State& st, const Params& p, int row, int, int) {
    st.m = -INFINITY; st.s = 0.f; st.u = 0.f; st.zy = -INFINITY;
    const int y = row < p.T ? __ldg(p.target + row) - p.v_offset : -1;
    st.y = (y >= 0 && y < p.V) ? y : -1;                          // outside this W's rows: no column matches
  }
  static __device__ __forceinline__ void chunk(State& st, const Params& p, int row, int col0,
                                               const uint32_t (&v)[32], uint8_t*) {
    if (col0 >= p.V) return;
    float z[32];
#pragma unroll
    for (int j = 0; j < 32; ++j) z[j] = __uint_as_float(v[j]);
    if constexpr (kStoreZ) {
      // a lane owns one row: eight 16-byte stores fill one 128-byte line of that row
      if (row < p.T) {
        float* dst = p.z + (size_t)row * p.ldz + col0;
        if (col0 + 32 <= p.V) {
#pragma unroll
          for (int q = 0; q < 8; ++q)
            reinterpret_cast<float4*>(dst)[q] = make_float4(z[4 * q], z[4 * q + 1], z[4 * q + 2], z[4 * q + 3]);
        } else {
#pragma unroll
          for (int j = 0; j < 32; ++j) if (col0 + j < p.V) dst[j] = z[j];
        }
      }
    }
    if (col0 + 32 > p.V) {  // ragged vocabulary tail: columns >= V hold zero-fill, not logits
#pragma unroll
      for (int j = 0; j < 32; ++j) if (col0 + j >= p.V) z[j] = -1.0e30f;
    }
    float mx = z[0];
#pragma unroll
    for (int j = 1; j < 32; ++j) mx = fmaxf(mx, z[j]);
    const float m_new = fmaxf(st.m, mx);
    const float sc = ex2f((st.m - m_new) * kLog2e);  // 0 on the first chunk (m = -inf)
    float s = st.s * sc, u = st.u * sc;
    const float nm = -m_new * kLog2e;
#pragma unroll
    for (int j = 0; j < 32; ++j) {
      const float e = ex2f(fmaf(z[j], kLog2e, nm));
      s += e;
      u = fmaf(e, z[j], u);
    }
    st.m = m_new; st.s = s; st.u = u;
    const int yl = st.y - col0;
    if (yl >= 0 && yl < 32) {
#pragma unroll
      for (int j = 0; j < 32; ++j) if (j == yl) st.zy = z[j];
    }
  }
  static __device__ __forceinline__ void unit_end(State& st, const Params& p, int row, int split) {
    if (row < p.T) p.partial[(size_t)split * p.T + row] = make_float4(st.m, st.s, st.u, st.zy);
  }
};
using LogprobEpi = LogprobEpiT<false>;

// Combines the S partial states of every token.  With `combined` set the result stays a partial
// state (m, s, u, zy) -- the statistics of one vocabulary shard -- and nothing else is written.
__global__ void __launch_bounds__(256) merge_partials_kernel(
    const float4* __restrict__ partial, const int32_t* __restrict__ target, int T, int V, int S,
    float* __restrict__ logp, float* __restrict__ entropy, float* __restrict__ lse_out,
    float4* __restrict__ combined, unsigned int* d_err) {
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= T) return;
  float M = -INFINITY;
  for (int i = 0; i < S; ++i) M = fmaxf(M, __ldg(&partial[(size_t)i * T + t]).x);
  float s = 0.f, u = 0.f, zy = -INFINITY;
  for (int i = 0; i < S; ++i) {
    const float4 q = __ldg(&partial[(size_t)i * T + t]);
    const float w = ex2f((q.x - M) * kLog2e);
    s = fmaf(q.y, w, s);
    u = fmaf(q.z, w, u);
    zy = fmaxf(zy, q.w);  // exactly one range holds the target; the others report -inf
  }
  if (combined) { combined[t] = make_float4(M, s, u, zy); return; }
  const float lse = M + kLn2 * log2f(s);
  const int y = __ldg(target + t);
  float lp = zy - lse;
  if (y < 0 || y >= V) {
    lp = __int_as_float(0x7fc00000);
    atomicOr(d_err, AF_DEVERR_TARGET_RANGE);
  }
  logp[t] = lp;
  if (entropy) entropy[t] = lse - u / s;
  if (lse_out) lse_out[t] = lse;
}

}  // namespace

// Number of vocabulary ranges S per row tile.  A worker (a CTA, or a CTA pair) runs units w,
// w + workers, ..., each unit being ceil(n_tiles / S) tiles long, so the launch lasts about
// ceil(m_tiles S / workers) * ceil(n_tiles / S) tile times: S is chosen to minimise that product
// (wave quantisation decides it for small batches).  The workers alive at one time sweep the
// vocabulary over ceil(workers / S) row tiles whose hidden-state panels should stay L2-resident
// while W streams past once, which rules out small S for wide hidden sizes.  More than 8 ranges are
// only allowed while S * T stays small (partials buffer).
int logprob_pick_splits(int64_t T, int32_t d, int32_t V, int sm_count, bool pair, int requested, int die0_pairs) {
  const int tile_rows = pair ? umma::kPairBM : umma::kBM;
  const int workers = pair ? (sm_count / 2 > 0 ? sm_count / 2 : 1) : (sm_count > 0 ? sm_count : 1);
  const int64_t m_tiles = (T + tile_rows - 1) / tile_rows;
  const int n_tiles = (V + umma::kBN - 1) / umma::kBN;
  if (requested > 0) return requested < n_tiles ? requested : n_tiles;
  if (m_tiles < 1) return 1;
  // bytes of hidden-state rows kept in L2.  Pairs sharing a row tile may sit on different dies, each
  // of which then caches the panel in its own half of L2, so pairs get the smaller budget; with the
  // row tiles dealt by die a panel lives in one half only and the budget holds per die, i.e. for the
  // row tiles half of the pairs keep alive
  const int64_t kPanelBudget = pair ? (48ll << 20) : (72ll << 20);
  // by die: the panels of the die with more pairs.  Its half of L2 also holds lines of the other
  // die's panels and the weight tiles in flight; 19 and 20 row tiles of the 7B head (34.9 and
  // 36.7 MB, parts with 72 + 76 and 70 + 78 SMs) stream W once per wave, which sets this budget
  const int64_t kDiePanelBudget = 36ll << 20;
  const bool by_die = pair && die0_pairs > 0 && die0_pairs < workers;
  const int64_t max_units_many = (int64_t)workers * 8;
  int best = 1;
  double best_cost = 1e300;
  for (int S = 1; S <= 32 && S <= n_tiles; ++S) {
    const int64_t units = m_tiles * S;
    if (S > 8 && units > max_units_many) break;
    // by die only where the launch will really deal that way (no extra round of units)
    const int die_workers = die0_pairs > workers - die0_pairs ? die0_pairs : workers - die0_pairs;
    const bool die_here = by_die && die_split_rows(m_tiles, S, workers, die0_pairs) > 0;
    const int fit_workers = die_here ? die_workers : workers;
    int64_t alive = (fit_workers + S - 1) / S;
    if (alive > m_tiles) alive = m_tiles;
    const bool fits = alive * tile_rows * (int64_t)d * 2 <= (die_here ? kDiePanelBudget : kPanelBudget);
    const int64_t grid = units < workers ? units : workers;
    double cost = (double)((units + grid - 1) / grid) * (double)((n_tiles + S - 1) / S);
    cost *= 1.0 + 0.002 * S;                          // partials written and merged per range
    if (!fits) cost *= 1.25;                          // W re-read from HBM by every row tile
    if (cost < best_cost) { best_cost = cost; best = S; }
  }
  return best;
}

void plan_token_logprob(int64_t T, int32_t d, int32_t V, int sm_count, int die0_sms, int requested_splits, bool pair,
                        bool die_aware, af_gemm_plan* plan) {
  const int die0_pairs = pair && die_aware && die0_sms > 0 ? die0_sms / 2 : 0;
  const int S = logprob_pick_splits(T, d, V, sm_count, pair, requested_splits, die0_pairs);
  umma::GemmShape g = gemm_shape((uint64_t)T, (uint64_t)V, (uint64_t)d, S, pair);
  const int64_t units = (int64_t)g.m_tiles * g.splits;
  const int64_t slots = pair ? sm_count / 2 : sm_count;
  if (pair) deal_by_die(g, (int)slots, die0_pairs);
  plan->m_tiles = g.m_tiles;
  plan->n_tiles = g.n_tiles;
  plan->v_splits = g.splits;
  plan->workers = (int32_t)(units < slots ? units : slots);
  plan->die0_workers = g.die0_pairs;
  plan->die0_row_tiles = g.die0_rows;
}

void plan_units(const af_gemm_plan& plan, int rank, int* first, int* stride, int* end) {
  umma::GemmShape g{};
  g.m_tiles = plan.m_tiles;
  g.splits = plan.v_splits;
  g.die0_pairs = plan.die0_workers;
  g.die0_rows = plan.die0_row_tiles;
  const umma::PairWork w = umma::pair_work(g, rank, plan.workers);   // plain dealing when die0_pairs is 0
  *first = w.base_unit + w.first;
  *stride = w.step;
  *end = w.base_unit + w.end;
}

af_status launch_token_logprob_z(af_ctx* ctx, const void* hidden, const void* W,
                                 const int32_t* target, int64_t T, int32_t d, int32_t V,
                                 float* logp, float* entropy, float* lse, float* z, cudaStream_t s) {
  if (T == 0) return AF_OK;
  const GemmEnv env = gemm_env(ctx);
  const int S = logprob_pick_splits(T, d, V, ctx->sm_count, env.pair, ctx->v_splits, env.die0_pairs);
  af_status st = ws_grow(ctx->partial, (size_t)S * (size_t)T * sizeof(float4));
  if (st != AF_OK) return st;
  const Operand Hop{hidden, (uint64_t)T, (uint64_t)d, (uint64_t)d * 2};
  const Operand Wop{W, (uint64_t)V, (uint64_t)d, (uint64_t)d * 2};
  if (z) {
    LogprobEpiT<true>::Params ep{target, (float4*)ctx->partial.p, (int)T, V, 0, z, (int64_t)V};
    st = run_gemm<LogprobEpiT<true>, false, false>(env, Hop, Wop, S, ep, s);
  } else {
    LogprobEpi::Params ep{target, (float4*)ctx->partial.p, (int)T, V, 0, nullptr, 0};
    st = run_gemm<LogprobEpi, false, false>(env, Hop, Wop, S, ep, s);
  }
  if (st != AF_OK) return st;
  merge_partials_kernel<<<(int)((T + 255) / 256), 256, 0, s>>>((const float4*)ctx->partial.p, target,
                                                              (int)T, V, S, logp, entropy, lse,
                                                              nullptr, ctx->d_err);
  return cudaGetLastError() == cudaSuccess ? AF_OK : AF_ERR_CUDA;
}

af_status launch_token_logprob(af_ctx* ctx, const void* hidden, const void* W,
                               const int32_t* target, int64_t T, int32_t d, int32_t V,
                               float* logp, float* entropy, float* lse, cudaStream_t s) {
  return launch_token_logprob_z(ctx, hidden, W, target, T, d, V, logp, entropy, lse, nullptr, s);
}

// One vocabulary shard: the same GEMM over the shard's rows of W, the ranges of a token combined
// into one partial state instead of a final result.
af_status launch_token_logprob_shard(af_ctx* ctx, const void* hidden, const void* W_shard,
                                     const int32_t* target, int64_t T, int32_t d, int32_t V_shard,
                                     int32_t v_offset, float* partial_out, cudaStream_t s) {
  if (T == 0) return AF_OK;
  const GemmEnv env = gemm_env(ctx);
  const int S = logprob_pick_splits(T, d, V_shard, ctx->sm_count, env.pair, ctx->v_splits, env.die0_pairs);
  af_status st = ws_grow(ctx->partial, (size_t)S * (size_t)T * sizeof(float4));
  if (st != AF_OK) return st;
  const Operand Hop{hidden, (uint64_t)T, (uint64_t)d, (uint64_t)d * 2};
  const Operand Wop{W_shard, (uint64_t)V_shard, (uint64_t)d, (uint64_t)d * 2};
  LogprobEpi::Params ep{target, (float4*)ctx->partial.p, (int)T, V_shard, v_offset, nullptr, 0};
  st = run_gemm<LogprobEpi, false, false>(env, Hop, Wop, S, ep, s);
  if (st != AF_OK) return st;
  merge_partials_kernel<<<(int)((T + 255) / 256), 256, 0, s>>>((const float4*)ctx->partial.p, target,
                                                              (int)T, V_shard, S, nullptr, nullptr, nullptr,
                                                              reinterpret_cast<float4*>(partial_out), ctx->d_err);
  return cudaGetLastError() == cudaSuccess ? AF_OK : AF_ERR_CUDA;
}

af_status launch_merge_logprob_shards(af_ctx* ctx, const float* partials, const int32_t* target, int32_t R,
                                      int64_t T, int32_t V_total, float* logp, float* entropy, float* lse,
                                      cudaStream_t s) {
  if (T == 0) return AF_OK;
  merge_partials_kernel<<<(int)((T + 255) / 256), 256, 0, s>>>(reinterpret_cast<const float4*>(partials), target,
                                                              (int)T, V_total, R, logp, entropy, lse, nullptr,
                                                              ctx->d_err);
  return cudaGetLastError() == cudaSuccess ? AF_OK : AF_ERR_CUDA;
}

}  // namespace af

// =============================================================================================
// af_token_logprob_static -- the same scoring call for callers that must not allocate.
//
// The online-softmax partials normally live in the context's cudaMalloc'ed workspace.  Here they
// live in a fixed array that is part of the library's device image, so the call needs no
// context and performs no allocation of its own.  The array's name is only a host-side handle
// in host code: its device address is looked up once per device with cudaGetSymbolAddress and
// that pointer is what the kernels receive.
// =============================================================================================
namespace af {
namespace {

constexpr int64_t kStaticMaxTokens = 32768;                       // largest T the call accepts
constexpr int64_t kStaticPartialSlots = 4 * kStaticMaxTokens;     // float4 slots: splits x tokens
constexpr size_t kStaticHeaderBytes = 256;                        // private error word lives here
constexpr size_t kStaticScratchBytes = kStaticHeaderBytes + (size_t)kStaticPartialSlots * sizeof(float4);

static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];   // 2 MiB + 256 B

constexpr int kStaticMaxDevices = 64;
struct StaticDeviceState {
  bool ready = false;
  unsigned char* scratch = nullptr;  // device address of g_static_scratch on this device
  int sm_count = 0;
};
StaticDeviceState g_static_state[kStaticMaxDevices];
EncodeTiledFn g_static_encode = nullptr;
std::mutex g_static_mutex;

// Once per device, with that device current: resolve the scratch address, read the SM count,
// and fetch the tensor-map encoder.
af_status static_setup(int dev, StaticDeviceState** out) {
  if (dev < 0 || dev >= kStaticMaxDevices) return AF_ERR_UNSUPPORTED_DEVICE;
  std::lock_guard<std::mutex> lock(g_static_mutex);
  StaticDeviceState& st = g_static_state[dev];
  if (!st.ready) {
    int major = 0, minor = 0, sms = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&minor, cudaDevAttrComputeCapabilityMinor, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
      return AF_ERR_CUDA;
    if (major != 10 || minor != 0) return AF_ERR_UNSUPPORTED_DEVICE;
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) {
      cudaGetLastError();
      return AF_ERR_CUDA;
    }
    if (!g_static_encode) {
      void* fn = nullptr;
      cudaDriverEntryPointQueryResult qres;
      if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
          qres != cudaDriverEntryPointSuccess || !fn)
        return AF_ERR_CUDA;
      g_static_encode = reinterpret_cast<EncodeTiledFn>(fn);
    }
    st.scratch = static_cast<unsigned char*>(p);
    st.sm_count = sms;
    st.ready = true;
  }
  *out = &st;
  return AF_OK;
}

}  // namespace
}  // namespace af

extern "C" af_status af_token_logprob_static(const void* hidden, const void* W, const int32_t* target,
                                             int64_t T, int32_t d, int32_t V, float* logp,
                                             float* entropy, float* lse, uint32_t* device_flags,
                                             void* stream) {
  using namespace af;
  if (T < 0 || d < 1 || V < 1) return AF_ERR_INVALID_ARG;
  if (T > kStaticMaxTokens) return AF_ERR_CAPACITY;   // the fixed scratch holds 32768 tokens at most
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return AF_ERR_CUDA;
  StaticDeviceState* st = nullptr;
  af_status rc = static_setup(dev, &st);
  if (rc != AF_OK) return rc;
  if (T == 0) return AF_OK;
  if (!hidden || !W || !target || !logp) return AF_ERR_INVALID_ARG;
  if (d % 8 != 0 || (reinterpret_cast<uintptr_t>(hidden) & 15u) || (reinterpret_cast<uintptr_t>(W) & 15u))
    return AF_ERR_ALIGNMENT;

  int S = logprob_pick_splits(T, d, V, st->sm_count, false, 0, 0);
  if ((int64_t)S * T > kStaticPartialSlots) S = (int)(kStaticPartialSlots / T);
  unsigned int* err_word = device_flags ? device_flags : reinterpret_cast<unsigned int*>(st->scratch);
  float4* partial = reinterpret_cast<float4*>(st->scratch + kStaticHeaderBytes);

  const GemmEnv env{g_static_encode, st->sm_count, err_word, false, nullptr, nullptr, nullptr, 0};
  const Operand Hop{hidden, (uint64_t)T, (uint64_t)d, (uint64_t)d * 2};
  const Operand Wop{W, (uint64_t)V, (uint64_t)d, (uint64_t)d * 2};
  LogprobEpi::Params ep{target, partial, (int)T, V, 0, nullptr, 0};
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if ((rc = run_gemm<LogprobEpi, false, false>(env, Hop, Wop, S, ep, s)) != AF_OK) return rc;
  merge_partials_kernel<<<(int)((T + 255) / 256), 256, 0, s>>>(partial, target, (int)T, V, S, logp, entropy,
                                                              lse, nullptr, err_word);
  return cudaGetLastError() == cudaSuccess ? AF_OK : AF_ERR_CUDA;
}
