// af_policy_loss_backward: gradient of the policy loss through log-softmax and the LM head.
//
// Tokens are processed in blocks of Tc rows.  Per block, three tensor-core GEMMs built on the
// same tcgen05 main loop:
//   1. recompute  Z = H_blk W^T  and turn it, in the epilogue, into
//        dZ = g_t (1{v = y_t} - exp(z - lse_t))   (bf16), written as dZ [Tc,V] and dZ^T [V,Tc];
//   2. dH_blk = dZ  * W      ([Tc,V] x [V,d], K = V)  -> bf16, using W^T  [d,V] as the K-major B;
//   3. dW    += dZ^T * H_blk ([V,Tc] x [Tc,d], K = Tc) -> fp32, using H^T [d,T] as the K-major B.
// The scratch is one block of dZ (both orientations) plus transposed copies of W and H; [T,V] is
// never materialised and the scratch does not grow with T (beyond the H^T copy).
#include "common.cuh"
#include "umma.cuh"

namespace af {
namespace {

constexpr float kLog2e = 1.4426950408889634f;
constexpr int kDefaultTokenBlock = 74 * 128;  // 74 row tiles x 14 column tiles of d = 3584 fill 7 waves of 148 SMs

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}

// ---- bf16 transpose: out[c, r] = in[r, c]; in [R, C] pitch ldi, out [C, R] pitch ldo ----------
__global__ void __launch_bounds__(256) transpose_bf16_kernel(const __nv_bfloat16* __restrict__ in,
                                                             __nv_bfloat16* __restrict__ out, int R,
                                                             int C, int64_t ldi, int64_t ldo) {
  __shared__ __nv_bfloat16 tile[64][66];
  const int r0 = blockIdx.x * 64, c0 = blockIdx.y * 64;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;  // 32 x 8
  for (int i = ty; i < 64; i += 8) {
    const int r = r0 + i, c = c0 + tx * 2;
    __nv_bfloat16 a = __float2bfloat16(0.f), b = a;
    if (r < R) {
      if (c + 1 < C) {
        const __nv_bfloat162 v = *reinterpret_cast<const __nv_bfloat162*>(in + (int64_t)r * ldi + c);
        a = v.x; b = v.y;
      } else if (c < C) {
        a = in[(int64_t)r * ldi + c];
      }
    }
    tile[i][tx * 2] = a; tile[i][tx * 2 + 1] = b;
  }
  __syncthreads();
  for (int i = ty; i < 64; i += 8) {
    const int c = c0 + i, r = r0 + tx * 2;
    if (c < C) {
      if (r + 1 < R) {
        __nv_bfloat162 v; v.x = tile[tx * 2][i]; v.y = tile[tx * 2 + 1][i];
        *reinterpret_cast<__nv_bfloat162*>(out + (int64_t)c * ldo + r) = v;
      } else if (r < R) {
        out[(int64_t)c * ldo + r] = tile[tx * 2][i];
      }
    }
  }
}

// ---- epilogue 1: logits tile -> dZ (both orientations) ----------------------------------------
struct DzEpi {
  struct Params {
    const int32_t* target;  // [rows] of this block
    const float* lse;       // [rows]
    const float* g;         // [rows] dL/dlogp
    __nv_bfloat16* dz;      // [rows, V]
    __nv_bfloat16* dzt;     // [V, ldzt]
    int rows, V;
    int64_t ldzt;
  };
  struct State {
    float g, nl;
    int y;
  };
  static __device__ __forceinline__ void unit_begin(State& st, const Params& p, int row, int, int) {
    if (row < p.rows) {
      st.g = __ldg(p.g + row);
      st.nl = -__ldg(p.lse + row) * kLog2e;
      st.y = __ldg(p.target + row);
    } else {
      st.g = 0.f; st.nl = 0.f; st.y = -1;
    }
  }
  static __device__ __forceinline__ void chunk(State& st, const Params& p, int row, int col0,
                                               const uint32_t (&v)[32]) {
    if (row >= p.rows || col0 >= p.V) return;
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
    __nv_bfloat16* drow = p.dz + (size_t)row * p.V + col0;
    if (col0 + 32 <= p.V) {
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        uint4 w;
        w.x = pack_bf16x2(dzv[q * 8 + 0], dzv[q * 8 + 1]);
        w.y = pack_bf16x2(dzv[q * 8 + 2], dzv[q * 8 + 3]);
        w.z = pack_bf16x2(dzv[q * 8 + 4], dzv[q * 8 + 5]);
        w.w = pack_bf16x2(dzv[q * 8 + 6], dzv[q * 8 + 7]);
        *reinterpret_cast<uint4*>(drow + q * 8) = w;
      }
#pragma unroll
      for (int j = 0; j < 32; ++j) p.dzt[(size_t)(col0 + j) * p.ldzt + row] = __float2bfloat16_rn(dzv[j]);
    } else {
#pragma unroll
      for (int j = 0; j < 32; ++j) {
        if (col0 + j < p.V) {
          const __nv_bfloat16 b = __float2bfloat16_rn(dzv[j]);
          drow[j] = b;
          p.dzt[(size_t)(col0 + j) * p.ldzt + row] = b;
        }
      }
    }
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
  static __device__ __forceinline__ void unit_begin(State&, const Params&, int, int, int) {}
  static __device__ __forceinline__ void chunk(State&, const Params& p, int row, int col0,
                                               const uint32_t (&v)[32]) {
    if (row >= p.M || col0 >= p.N) return;
    __nv_bfloat16* c = p.C + (size_t)row * p.ldc + col0;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      if (col0 + q * 8 + 8 <= p.N) {
        uint4 w;
        w.x = pack_bf16x2(__uint_as_float(v[q * 8 + 0]), __uint_as_float(v[q * 8 + 1]));
        w.y = pack_bf16x2(__uint_as_float(v[q * 8 + 2]), __uint_as_float(v[q * 8 + 3]));
        w.z = pack_bf16x2(__uint_as_float(v[q * 8 + 4]), __uint_as_float(v[q * 8 + 5]));
        w.w = pack_bf16x2(__uint_as_float(v[q * 8 + 6]), __uint_as_float(v[q * 8 + 7]));
        *reinterpret_cast<uint4*>(c + q * 8) = w;
      }
    }
  }
  static __device__ __forceinline__ void unit_end(State&, const Params&, int, int) {}
};

// ---- epilogue 3: accumulator tile -> fp32 matrix (store or add) ---------------------------------
struct StoreF32Epi {
  struct Params {
    float* C;
    int64_t ldc;
    int M, N;
    int accumulate;
  };
  struct State {};
  static __device__ __forceinline__ void unit_begin(State&, const Params&, int, int, int) {}
  static __device__ __forceinline__ void chunk(State&, const Params& p, int row, int col0,
                                               const uint32_t (&v)[32]) {
    if (row >= p.M || col0 >= p.N) return;
    float* c = p.C + (size_t)row * p.ldc + col0;
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      if (col0 + q * 4 + 4 <= p.N) {
        float4 w = make_float4(__uint_as_float(v[q * 4 + 0]), __uint_as_float(v[q * 4 + 1]),
                               __uint_as_float(v[q * 4 + 2]), __uint_as_float(v[q * 4 + 3]));
        if (p.accumulate) {
          const float4 o = *reinterpret_cast<const float4*>(c + q * 4);
          w.x += o.x; w.y += o.y; w.z += o.z; w.w += o.w;
        }
        *reinterpret_cast<float4*>(c + q * 4) = w;
      }
    }
  }
  static __device__ __forceinline__ void unit_end(State&, const Params&, int, int) {}
};

template <class E>
af_status run_gemm(af_ctx* ctx, const void* A, uint64_t a_rows, uint64_t a_pitch, const void* B,
                   uint64_t b_rows, uint64_t b_pitch, uint64_t K, int splits,
                   const typename E::Params& ep, cudaStream_t s) {
  CUtensorMap ta, tb;
  af_status st = encode_bf16_2d(ctx, &ta, A, a_rows, K, a_pitch, umma::kBM);
  if (st != AF_OK) return st;
  st = encode_bf16_2d(ctx, &tb, B, b_rows, K, b_pitch, umma::kBN);
  if (st != AF_OK) return st;
  umma::GemmShape g;
  g.M = (int)a_rows; g.N = (int)b_rows; g.K = (int)K;
  g.m_tiles = (int)((a_rows + umma::kBM - 1) / umma::kBM);
  g.n_tiles = (int)((b_rows + umma::kBN - 1) / umma::kBN);
  g.splits = splits > 0 && splits < g.n_tiles ? splits : g.n_tiles;
  g.k_blocks = (int)((K + umma::kBK - 1) / umma::kBK);
  if (cudaFuncSetAttribute(umma::gemm_kernel<E>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           umma::kSmemBytes) != cudaSuccess) return AF_ERR_CUDA;
  const int64_t units = (int64_t)g.m_tiles * g.splits;
  const int grid = (int)(units < ctx->sm_count ? units : ctx->sm_count);
  umma::gemm_kernel<E><<<grid, umma::kThreads, umma::kSmemBytes, s>>>(ta, tb, g, ep, ctx->d_err);
  return cudaGetLastError() == cudaSuccess ? AF_OK : AF_ERR_CUDA;
}

}  // namespace

af_status launch_backward(af_ctx* ctx, const void* hidden, const void* W, const int32_t* target,
                          const float* lse, const float* dlogp, int64_t T, int32_t d, int32_t V,
                          void* d_hidden, float* d_W, int32_t accumulate_dW, cudaStream_t s) {
  int64_t Tc = ctx->bwd_token_block > 0 ? ctx->bwd_token_block : kDefaultTokenBlock;
  const int64_t T_round = ((T + 127) / 128) * 128;
  if (Tc > T_round) Tc = T_round > 0 ? T_round : 128;
  const int64_t T_pad = (T + 7) & ~(int64_t)7;

  af_status st;
  if ((st = ws_grow(ctx->wt, (size_t)d * V * 2)) != AF_OK) return st;
  if ((st = ws_grow(ctx->ht, (size_t)d * (T_pad > 0 ? T_pad : 8) * 2)) != AF_OK) return st;
  if ((st = ws_grow(ctx->dz, (size_t)Tc * V * 2)) != AF_OK) return st;
  if ((st = ws_grow(ctx->dzt, (size_t)V * Tc * 2)) != AF_OK) return st;
  if (accumulate_dW < 0) return AF_OK;  // reserve only

  if (T == 0) {
    if (!accumulate_dW && cudaMemsetAsync(d_W, 0, (size_t)V * d * sizeof(float), s) != cudaSuccess) return AF_ERR_CUDA;
    return AF_OK;
  }
  const __nv_bfloat16* H = static_cast<const __nv_bfloat16*>(hidden);
  __nv_bfloat16* wt = static_cast<__nv_bfloat16*>(ctx->wt.p);
  __nv_bfloat16* ht = static_cast<__nv_bfloat16*>(ctx->ht.p);
  __nv_bfloat16* dz = static_cast<__nv_bfloat16*>(ctx->dz.p);
  __nv_bfloat16* dzt = static_cast<__nv_bfloat16*>(ctx->dzt.p);

  {  // K-major copies of the two B operands
    dim3 gw((V + 63) / 64, (d + 63) / 64);
    transpose_bf16_kernel<<<gw, 256, 0, s>>>(static_cast<const __nv_bfloat16*>(W), wt, V, d, d, V);
    dim3 gh((unsigned)((T + 63) / 64), (d + 63) / 64);
    transpose_bf16_kernel<<<gh, 256, 0, s>>>(H, ht, (int)T, d, d, T_pad);
    if (cudaGetLastError() != cudaSuccess) return AF_ERR_CUDA;
  }

  bool first = true;
  for (int64_t t0 = 0; t0 < T; t0 += Tc, first = false) {
    const int64_t tc = (T - t0) < Tc ? (T - t0) : Tc;
    // 1. dZ block
    DzEpi::Params p1{target + t0, lse + t0, dlogp + t0, dz, dzt, (int)tc, V, Tc};
    st = run_gemm<DzEpi>(ctx, H + t0 * d, (uint64_t)tc, (uint64_t)d * 2, W, (uint64_t)V, (uint64_t)d * 2,
                         (uint64_t)d, logprob_pick_splits(tc, V, ctx->sm_count, ctx->v_splits), p1, s);
    if (st != AF_OK) return st;
    // 2. dH block = dZ * W
    StoreBf16Epi::Params p2{static_cast<__nv_bfloat16*>(d_hidden) + t0 * d, d, (int)tc, d};
    st = run_gemm<StoreBf16Epi>(ctx, dz, (uint64_t)tc, (uint64_t)V * 2, wt, (uint64_t)d, (uint64_t)V * 2,
                                (uint64_t)V, 0, p2, s);
    if (st != AF_OK) return st;
    // 3. dW += dZ^T * H block
    StoreF32Epi::Params p3{d_W, d, V, d, (!first || accumulate_dW) ? 1 : 0};
    st = run_gemm<StoreF32Epi>(ctx, dzt, (uint64_t)V, (uint64_t)Tc * 2, ht + t0, (uint64_t)d,
                               (uint64_t)T_pad * 2, (uint64_t)tc, 0, p3, s);
    if (st != AF_OK) return st;
  }
  return AF_OK;
}

}  // namespace af
