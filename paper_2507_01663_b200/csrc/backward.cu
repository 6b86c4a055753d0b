// af_policy_loss_backward: gradient of the policy loss through log-softmax and the LM head.
//
// Tokens are processed in blocks of Tc rows.  Per block, three tensor-core GEMMs built on the
// same tcgen05 main loop:
//   1. recompute  Z = H_blk W^T  (both operands K-major) and turn it, in the epilogue, into
//        dZ = g_t (1{v = y_t} - exp(z - lse_t))   (bf16), written once as dZ [Tc, V];
//   2. dH_blk = dZ * W        A = dZ [Tc,V] K-major,  B = W [V,d] read MN-major   -> bf16 [Tc, d];
//   3. dW^T  += H_blk^T * dZ  A = H_blk [Tc,d] and B = dZ [Tc,V], both read MN-major; the tile is
//                             computed as [d, V] and stored transposed into fp32 dW [V, d].
// No operand is ever transposed in memory.  The scratch is one block of dZ; [T,V] is never
// materialised and the scratch does not grow with T.
//
// Epilogues hold one output row per lane (the TMEM load shape); storing that directly would write
// 16 bytes to each of 32 different rows per instruction.  The dZ and dH epilogues therefore pass
// their 32x32 chunk through a private, XOR-swizzled shared-memory buffer and store whole 64-byte
// row segments, eight rows per instruction.  The dW product is laid out the other way round: its
// accumulator rows run along d, the contiguous dimension of dW, so 32 lanes holding the same
// vocabulary row write 128 consecutive bytes without any staging.  That orientation also gives the
// product the forward's memory behaviour: the H_blk panels of the row tiles in flight stay in L2
// while dZ streams past them (once per round of row tiles).
#include "device_util.cuh"
#include "gemm_launch.cuh"

namespace af {
namespace {

constexpr int kDefaultTokenBlock = 74 * 128;  // 37 pair tiles (74 CTA tiles) x 14 column tiles of d = 3584: 7 full rounds of 148 SMs


// Store a 32-row x 32-column bf16 chunk (lane L holds row L as 16 packed words) to a row-major
// bf16 matrix: rows row0.., columns col0..; rows >= M and 8-column groups past N are skipped.
// Staging layout: row r occupies 64 bytes = four 16-byte slots; slot q of row r lives at position
// q ^ ((r >> 1) & 3), which makes both the row-per-lane writes and the 8-rows-per-instruction
// reads free of bank conflicts.
__device__ __forceinline__ void store_chunk_bf16(const uint32_t (&w)[16], uint8_t* stage, int lane,
                                                 __nv_bfloat16* C, int64_t ldc, int row0, int col0,
                                                 int M, int N) {
  uint4* st = reinterpret_cast<uint4*>(stage);
#pragma unroll
  for (int q = 0; q < 4; ++q)
    st[lane * 4 + (q ^ ((lane >> 1) & 3))] = make_uint4(w[q * 4 + 0], w[q * 4 + 1], w[q * 4 + 2], w[q * 4 + 3]);
  __syncwarp();
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = i * 8 + (lane >> 2), c = lane & 3;
    const uint4 v = st[r * 4 + (c ^ ((r >> 1) & 3))];
    const int grow = row0 + r, gcol = col0 + c * 8;
    if (grow < M && gcol + 8 <= N) *reinterpret_cast<uint4*>(C + (size_t)grow * ldc + gcol) = v;
  }
  __syncwarp();
}

// ---- epilogue 1: logits tile -> dZ ----------------------------------------------------------------
struct DzEpi {
  struct Params {
    const int32_t* target;  // [rows] of this block
    const float* lse;       // [rows]
    const float* g;         // [rows] dL/dlogp
    __nv_bfloat16* dz;      // [rows, V]
    int rows, V;
    int v_offset;           // vocabulary id of W's first row (0 unless W is one shard of the head)
  };
  struct State {
    float g, nl;
    int y;
  };
  static constexpr bool kStaged = true;
  static __device__ __forceinline__ void unit_begin(State& st, const Params& p, int row, int, int) {
    if (row < p.rows) {
      st.g = __ldg(p.g + row);
      st.nl = -__ldg(p.lse + row) * kLog2e;
      st.y = __ldg(p.target + row) - p.v_offset;   // outside [0, V): no column of this W matches
    } else {
      st.g = 0.f; st.nl = 0.f; st.y = -1;
    }
  }
  static __device__ __forceinline__ void chunk(State& st, const Params& p, int row, int col0,
                                               const uint32_t (&v)[32], uint8_t* stage) {
    if (col0 >= p.V) return;                       // uniform across the warp
    const int lane = threadIdx.x & 31;
    float dzv[32];
#pragma unroll
    for (int j = 0; j < 32; ++j) {
      const float prob = ex2f(fmaf(__uint_as_float(v[j]), kLog2e, st.nl));
      dzv[j] = -st.g * prob;
    }
    const int yl = st.y - col0;
    if (yl >= 0 && yl < 32) {
#pragma unroll
      for (int j = 0; j < 32; ++j) if (j == yl) dzv[j] += st.g;
    }
    uint32_t w[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) w[j] = pack_bf16x2(dzv[2 * j], dzv[2 * j + 1]);
    store_chunk_bf16(w, stage, lane, p.dz, p.V, row - lane, col0, p.rows, p.V);
  }
  static __device__ __forceinline__ void unit_end(State&, const Params&, int, int) {}
};

// ---- epilogue 2: accumulator tile -> bf16 matrix ------------------------------------------------
struct StoreBf16Epi {
  struct Params {
    __nv_bfloat16* C;
    int64_t ldc;
    int M, N;
  };
  struct State {};
  static constexpr bool kStaged = true;
  static __device__ __forceinline__ void unit_begin(State&, const Params&, int, int, int) {}
  static __device__ __forceinline__ void chunk(State&, const Params& p, int row, int col0,
                                               const uint32_t (&v)[32], uint8_t* stage) {
    if (col0 >= p.N) return;
    const int lane = threadIdx.x & 31;
    uint32_t w[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) w[j] = pack_bf16x2(__uint_as_float(v[2 * j]), __uint_as_float(v[2 * j + 1]));
    store_chunk_bf16(w, stage, lane, p.C, p.ldc, row - lane, col0, p.M, p.N);
  }
  static __device__ __forceinline__ void unit_end(State&, const Params&, int, int) {}
};

// ---- epilogue 3: accumulator tile [m, n] -> fp32 matrix C[n, m] (store or add) ------------------
// Lane L holds row m = row0 + L; for a fixed column n the 32 lanes address 32 consecutive floats of
// C's row n: one coalesced 128-byte access per column.
struct StoreF32TransposedEpi {
  struct Params {
    float* C;          // [N, M] row-major
    int64_t ldc;       // elements between consecutive n
    int M, N;
    int accumulate;
  };
  struct State {};
  static constexpr bool kStaged = false;
  static __device__ __forceinline__ void unit_begin(State&, const Params&, int, int, int) {}
  static __device__ __forceinline__ void chunk(State&, const Params& p, int row, int col0,
                                               const uint32_t (&v)[32], uint8_t*) {
    if (col0 >= p.N || row >= p.M) return;
    float* dst = p.C + (size_t)col0 * p.ldc + row;
    if (col0 + 32 <= p.N) {
      if (p.accumulate) {
        float o[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) o[j] = dst[(size_t)j * p.ldc];
#pragma unroll
        for (int j = 0; j < 32; ++j) dst[(size_t)j * p.ldc] = o[j] + __uint_as_float(v[j]);
      } else {
#pragma unroll
        for (int j = 0; j < 32; ++j) dst[(size_t)j * p.ldc] = __uint_as_float(v[j]);
      }
    } else {
#pragma unroll
      for (int j = 0; j < 32; ++j) {
        if (col0 + j < p.N) {
          float w = __uint_as_float(v[j]);
          if (p.accumulate) w += dst[(size_t)j * p.ldc];
          dst[(size_t)j * p.ldc] = w;
        }
      }
    }
  }
  static __device__ __forceinline__ void unit_end(State&, const Params&, int, int) {}
};

}  // namespace

// The two products that consume a block of dZ [tc, V] (bf16):
//   dH_blk = dZ W:        A = dZ (K = v contiguous), B = W read MN-major (n = d contiguous, K = v rows)
//   dW^T  += H_blk^T dZ:  A = H_blk read MN-major (m = d contiguous, K = t rows), B = dZ read MN-major
//                         (n = v contiguous); tile [d, v] stored transposed into dW [V, d].  Vocabulary
//                         ranges are chosen as in the forward: the H_blk panels in flight stay in L2, dZ
//                         streams past them.
af_status launch_backward_products(af_ctx* ctx, const void* hidden_blk, const void* W, const void* dz_blk,
                                   int64_t tc, int32_t d, int32_t V, void* d_hidden_blk, float* d_W,
                                   int32_t accumulate_dW, bool last_block, cudaStream_t s) {
  const GemmEnv env = gemm_env(ctx);
  const uint64_t dB = (uint64_t)d * 2, vB = (uint64_t)V * 2;
  const Operand Hblk{hidden_blk, (uint64_t)tc, (uint64_t)d, dB};
  const Operand Wop{W, (uint64_t)V, (uint64_t)d, dB};
  const Operand dZop{dz_blk, (uint64_t)tc, (uint64_t)V, vB};
  auto dH_product = [&]() {
    StoreBf16Epi::Params p2{static_cast<__nv_bfloat16*>(d_hidden_blk), d, (int)tc, d};
    return run_gemm<StoreBf16Epi, false, true>(env, dZop, Wop, 0, p2, s);
  };
  auto dW_product = [&]() {
    StoreF32TransposedEpi::Params p3{d_W, d, d, V, accumulate_dW ? 1 : 0};
    return run_gemm<StoreF32TransposedEpi, true, true>(
        env, Hblk, dZop, logprob_pick_splits((int64_t)d, (int32_t)tc, V, ctx->sm_count, env.pair, 0, 0), p3, s);
  };
  // With a "d_W ready" event registered, the last block runs its dW product first and records the
  // event behind it: d_W is complete from there on, and whoever waits on the event (a gradient
  // all-reduce on another stream) overlaps with the block's dH product and whatever follows.
  if (last_block && ctx->dw_ready) {
    af_status st = dW_product();
    if (st != AF_OK) return st;
    if (cudaEventRecord(ctx->dw_ready, s) != cudaSuccess) return AF_ERR_CUDA;
    return dH_product();
  }
  af_status st = dH_product();
  if (st != AF_OK) return st;
  return dW_product();
}

// Token block of the backward (and of the fused update): a multiple of 128 rows.
int64_t backward_token_block(const af_ctx* ctx, int64_t T) {
  int64_t Tc = ctx->bwd_token_block > 0 ? ctx->bwd_token_block : kDefaultTokenBlock;
  const int64_t T_round = ((T + 127) / 128) * 128;
  if (Tc > T_round) Tc = T_round > 0 ? T_round : 128;
  return Tc;
}

af_status launch_backward(af_ctx* ctx, const void* hidden, const void* W, const int32_t* target,
                          const float* lse, const float* dlogp, int64_t T, int32_t d, int32_t V,
                          void* d_hidden, float* d_W, int32_t accumulate_dW, cudaStream_t s, int32_t v_offset) {
  const int64_t Tc = backward_token_block(ctx, T);
  const GemmEnv env = gemm_env(ctx);
  af_status st;
  if ((st = ws_grow(ctx->dz, (size_t)Tc * V * 2)) != AF_OK) return st;
  if (accumulate_dW < 0) return AF_OK;  // reserve only

  if (T == 0) {
    if (!accumulate_dW && cudaMemsetAsync(d_W, 0, (size_t)V * d * sizeof(float), s) != cudaSuccess) return AF_ERR_CUDA;
    if (ctx->dw_ready && cudaEventRecord(ctx->dw_ready, s) != cudaSuccess) return AF_ERR_CUDA;
    return AF_OK;
  }
  const __nv_bfloat16* H = static_cast<const __nv_bfloat16*>(hidden);
  __nv_bfloat16* dz = static_cast<__nv_bfloat16*>(ctx->dz.p);
  const uint64_t dB = (uint64_t)d * 2;

  bool first = true;
  for (int64_t t0 = 0; t0 < T; t0 += Tc, first = false) {
    const uint64_t tc = (uint64_t)((T - t0) < Tc ? (T - t0) : Tc);
    const Operand Hblk{H + t0 * d, tc, (uint64_t)d, dB};
    const Operand Wop{W, (uint64_t)V, (uint64_t)d, dB};
    // 1. dZ block:  Z = H_blk W^T, both K-major
    DzEpi::Params p1{target + t0, lse + t0, dlogp + t0, dz, (int)tc, V, v_offset};
    st = run_gemm<DzEpi, false, false>(env, Hblk, Wop,
                                       logprob_pick_splits((int64_t)tc, d, V, ctx->sm_count, env.pair, ctx->v_splits, env.die0_pairs), p1, s);
    if (st != AF_OK) return st;
    st = launch_backward_products(ctx, H + t0 * d, W, dz, (int64_t)tc, d, V,
                                  static_cast<__nv_bfloat16*>(d_hidden) + t0 * d, d_W,
                                  (!first || accumulate_dW) ? 1 : 0, t0 + Tc >= T, s);
    if (st != AF_OK) return st;
  }
  return AF_OK;
}

}  // namespace af
