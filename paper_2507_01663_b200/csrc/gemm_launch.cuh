// Host side of the tensor-core GEMMs: tensor-map encoding, work decomposition and the launch of
// either variant of the main loop (one CTA per 128 x 256 tile, or a CTA pair per 256 x 256 tile).
#pragma once

#include "common.cuh"
#include "umma.cuh"

namespace af {

// One operand of a GEMM launch: the matrix as it sits in memory.
struct Operand {
  const void* base;
  uint64_t rows, cols;   // memory rows and (contiguous) columns
  uint64_t pitch_bytes;
};

// What a launch needs from its surroundings (a context, or the context-free entry point).
struct GemmEnv {
  EncodeTiledFn encode;
  int sm_count;
  unsigned int* d_err;
  bool pair;             // CTA-pair variant (cta_group::2)
  unsigned int* tile_clock;  // device word the pair variant paces itself with (zeroed per launch), or null
  TmapCache* cache;          // tensor maps encoded earlier (a context's), or null
  const unsigned char* die_of_sm;  // measured die of every SM id, or null
  int die0_pairs;            // > 0: deal row tiles to pairs by die; CTA pairs the first die hosts
};

// Die-aware dealing of a pair GEMM's units (see umma::PairWork): can the first rows0 row tiles go to
// the n0 pairs of one die and the rest to the others without any pair needing more rounds of units
// than plain dealing would?  rows0 is looked for near m_tiles * n0 / pairs.  Returns 0 if not.
inline int die_split_rows(int64_t m_tiles, int64_t splits, int64_t pairs, int64_t n0) {
  const int64_t n1 = pairs - n0, units = m_tiles * splits;
  if (n0 <= 0 || n1 <= 0 || units < pairs || m_tiles < 2) return 0;
  const int64_t plain_rounds = (units + pairs - 1) / pairs;
  const int64_t guess = (m_tiles * n0 + pairs / 2) / pairs;
  int64_t best_rows = 0, best_rounds = INT64_MAX;
  for (int64_t r0 = guess - 2; r0 <= guess + 2; ++r0) {
    if (r0 < 1 || r0 >= m_tiles) continue;
    const int64_t a = (r0 * splits + n0 - 1) / n0, b = ((m_tiles - r0) * splits + n1 - 1) / n1;
    const int64_t rounds = a > b ? a : b;
    if (rounds < best_rounds) { best_rounds = rounds; best_rows = r0; }
  }
  return best_rows > 0 && best_rounds <= plain_rounds ? (int)best_rows : 0;
}

// Tiles, vocabulary ranges and K blocks of C[M,N] = sum_k A(m,k) B(n,k); `splits` <= 0 means one unit
// per B tile.  Dealt plainly until deal_by_die says otherwise.
inline umma::GemmShape gemm_shape(uint64_t M, uint64_t N, uint64_t K, int splits, bool pair) {
  const int tile_rows = pair ? umma::kPairBM : umma::kBM;
  umma::GemmShape g;
  g.M = (int)M; g.N = (int)N; g.K = (int)K;
  g.m_tiles = (int)((M + tile_rows - 1) / tile_rows);
  g.n_tiles = (int)((N + umma::kBN - 1) / umma::kBN);
  g.splits = splits > 0 && splits < g.n_tiles ? splits : g.n_tiles;
  g.k_blocks = (int)((K + umma::kBK - 1) / umma::kBK);
  g.die0_pairs = 0;
  g.die0_rows = 0;
  return g;
}
// Die-aware dealing of a pair launch: only when every SM pair gets a CTA pair and it costs no extra
// round of units.  Fills g.die0_pairs / g.die0_rows and returns true if so.
inline bool deal_by_die(umma::GemmShape& g, int pairs, int die0_pairs) {
  const int64_t units = (int64_t)g.m_tiles * g.splits;
  const int rows0 = die0_pairs > 0 && units >= pairs ? die_split_rows(g.m_tiles, g.splits, pairs, die0_pairs) : 0;
  if (rows0 <= 0) return false;
  g.die0_pairs = die0_pairs;
  g.die0_rows = rows0;
  return true;
}

inline af_status encode_operand(const GemmEnv& env, CUtensorMap* map, const Operand& op, uint32_t box_rows) {
  TmapCache::Entry* slot = nullptr;
  if (env.cache) {
    for (TmapCache::Entry& c : env.cache->e)
      if (c.base == op.base && c.rows == op.rows && c.cols == op.cols && c.pitch == op.pitch_bytes &&
          c.box_rows == box_rows) { *map = c.map; return AF_OK; }
    slot = &env.cache->e[env.cache->next];
    env.cache->next = (env.cache->next + 1) % TmapCache::kEntries;
  }
  cuuint64_t dims[2] = {op.cols, op.rows};
  cuuint64_t strides[1] = {op.pitch_bytes};
  cuuint32_t box[2] = {64, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = env.encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(op.base), dims, strides,
                          box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) { if (slot) slot->base = nullptr; return AF_ERR_CUDA; }
  if (slot) {
    slot->base = op.base; slot->rows = op.rows; slot->cols = op.cols; slot->pitch = op.pitch_bytes;
    slot->box_rows = box_rows; slot->map = *map;
  }
  return AF_OK;
}

// C[M,N] = sum_k A(m,k) B(n,k).  A K-major operand is stored [M or N, K]; an MN-major operand is
// stored [K, M or N].  TMA box: 64 contiguous elements wide; K-major A 128 rows, K-major B 256
// rows (128 per CTA of a pair), MN-major 64 K-rows.  `splits` <= 0 means one unit per B tile.
template <class E, bool kAMN, bool kBMN>
af_status run_gemm(const GemmEnv& env, const Operand& A, const Operand& B, int splits,
                   const typename E::Params& ep, cudaStream_t s) {
  CUtensorMap ta, tb;
  af_status st = encode_operand(env, &ta, A, kAMN ? 64 : umma::kBM);
  if (st != AF_OK) return st;
  st = encode_operand(env, &tb, B, kBMN ? 64 : (env.pair ? umma::kBN / 2 : umma::kBN));
  if (st != AF_OK) return st;
  const uint64_t M = kAMN ? A.cols : A.rows, K = kAMN ? A.rows : A.cols;
  const uint64_t N = kBMN ? B.cols : B.rows;
  umma::GemmShape g = gemm_shape(M, N, K, splits, env.pair);
  const int64_t units = (int64_t)g.m_tiles * g.splits;
  if (env.pair) {
    constexpr int smem = E::kStaged ? umma::kPairSmemBytesStaged : umma::kPairSmemBytes;
    static SmemAttrOnce once;
    if (set_smem_once(once, umma::gemm_pair_kernel<E, kAMN, kBMN>, smem) != cudaSuccess) return AF_ERR_CUDA;
    const int pairs = env.sm_count / 2;
    const int grid = 2 * (int)(units < pairs ? units : pairs);
    unsigned int* clock = env.tile_clock;
    const bool by_die = env.die_of_sm && clock && deal_by_die(g, pairs, env.die0_pairs);
    if (clock && cudaMemsetAsync(clock, 0, (by_die ? 3 : 1) * sizeof(unsigned int), s) != cudaSuccess) return AF_ERR_CUDA;
    umma::gemm_pair_kernel<E, kAMN, kBMN><<<grid, umma::kThreads, smem, s>>>(ta, tb, g, ep, env.d_err, clock,
                                                                             by_die ? clock + 1 : nullptr, env.die_of_sm);
  } else {
    constexpr int smem = E::kStaged ? umma::kSmemBytesStaged : umma::kSmemBytes;
    static SmemAttrOnce once;
    if (set_smem_once(once, umma::gemm_kernel<E, kAMN, kBMN>, smem) != cudaSuccess) return AF_ERR_CUDA;
    const int grid = (int)(units < env.sm_count ? units : env.sm_count);
    umma::gemm_kernel<E, kAMN, kBMN><<<grid, umma::kThreads, smem, s>>>(ta, tb, g, ep, env.d_err);
  }
  return cudaGetLastError() == cudaSuccess ? AF_OK : AF_ERR_CUDA;
}

inline GemmEnv gemm_env(af_ctx* ctx) {
  return GemmEnv{ctx->encode, ctx->sm_count, ctx->d_err, ctx->gemm_pair != 0, ctx->d_err + kTileClockWord,
                 &ctx->tmaps, reinterpret_cast<const unsigned char*>(ctx->d_err) + kDieTableByte,
                 ctx->die_aware && ctx->die0_sms > 0 ? ctx->die0_sms / 2 : 0};
}

}  // namespace af
