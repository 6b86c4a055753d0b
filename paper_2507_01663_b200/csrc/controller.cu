// Controller side of the streaming store: the per-sample status table and one read request
// against it, plus the token-balancing step the controller runs on a selected batch.
//
// Status table (device): ready[i] has bit c set once column c of sample i has been written;
// consumed[i] has bit t set once sample i has been handed to RL task t.
//
//   put    ready[idx[j]] |= column_bits                          (one atomic OR per entry)
//   get    eligible(i) = (ready[i] & mask) == mask && !(consumed[i] & task_bit); the request
//          takes the longest prefix of the eligible samples, in index order, within a sample
//          count and an optional token budget, writes their indices in order and marks them
//          consumed.  An ordered, bounded stream compaction: 8-12 bytes read per sample.
//
// A launch of `get` is two passes.  Pass 1: every block reduces its contiguous segment of the
// table to (eligible count, eligible tokens, first tile holding an eligible sample).  Pass 2: a
// block sums the aggregates of the blocks before it, and only if the prefix can still reach into
// its segment re-reads the segment from that first tile on (a table whose head has been consumed
// already is the normal case), ranks its eligible samples with a block-wide scan and emits those
// inside the limits.  Small tables
// (one segment) run pass 2 alone.  All integer arithmetic; the result is unique.
//
// Balancing (host): the k-way largest differencing method of Karmarkar and Karp on token counts,
// with or without equal sample counts per group.  A sequential heap algorithm over a few thousand
// integers: it runs on the host, where the index lists live.
#include <algorithm>
#include <climits>
#include <queue>
#include <vector>

#include "common.cuh"

namespace af {
namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kQuad = 4;                       // samples per thread per tile (one 128-bit load per column)
constexpr int kTile = kThreads * kQuad;        // samples per block tile
constexpr int64_t kSingleBlockMax = 16384;     // tables up to this size are served by one block

struct Agg {                                   // per-block aggregate of pass 1
  int count;
  int first_tile;                              // first tile of the segment that holds an eligible sample
  long long tokens;
};

struct Quad {
  int elig[kQuad];
  int len[kQuad];
};

// Status of samples i0 .. i0+3 (i0 a multiple of 4): eligibility flags and lengths, zero past N.
__device__ __forceinline__ Quad load_quad(const uint32_t* __restrict__ ready, const uint32_t* __restrict__ consumed,
                                          const int32_t* __restrict__ length, int64_t i0, int64_t N,
                                          uint32_t mask, uint32_t task_bit, bool vec_ok) {
  Quad q;
  uint32_t r[kQuad], c[kQuad];
  if (vec_ok && i0 + kQuad <= N) {
    const uint4 rv = __ldg(reinterpret_cast<const uint4*>(ready + i0));
    const uint4 cv = __ldcv(reinterpret_cast<const uint4*>(consumed + i0));
    r[0] = rv.x; r[1] = rv.y; r[2] = rv.z; r[3] = rv.w;
    c[0] = cv.x; c[1] = cv.y; c[2] = cv.z; c[3] = cv.w;
    if (length) {
      const int4 lv = __ldg(reinterpret_cast<const int4*>(length + i0));
      q.len[0] = lv.x; q.len[1] = lv.y; q.len[2] = lv.z; q.len[3] = lv.w;
    }
  } else {
#pragma unroll
    for (int k = 0; k < kQuad; ++k) {
      const bool in = i0 + k < N;
      r[k] = in ? __ldg(ready + i0 + k) : 0u;
      c[k] = in ? __ldcv(consumed + i0 + k) : 0u;
      if (length) q.len[k] = in ? __ldg(length + i0 + k) : 0;
    }
  }
#pragma unroll
  for (int k = 0; k < kQuad; ++k) {
    q.elig[k] = (i0 + k < N) && ((r[k] & mask) == mask) && ((c[k] & task_bit) == 0u);
    if (!length) q.len[k] = 0;
    if (!q.elig[k]) q.len[k] = 0;
    if (q.len[k] < 0) q.len[k] = 0;
  }
  return q;
}

// Block-wide exclusive scan of (count, tokens) pairs in thread order; also returns the totals.
__device__ __forceinline__ void block_scan(int c, long long t, int& c_ex, long long& t_ex, int& c_tot,
                                           long long& t_tot, int* s_c, long long* s_t) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int ci = c;
  long long ti = t;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int cu = __shfl_up_sync(0xffffffffu, ci, o);
    const long long tu = __shfl_up_sync(0xffffffffu, ti, o);
    if (lane >= o) { ci += cu; ti += tu; }
  }
  __syncthreads();                    // the arrays may still be read from the previous call
  if (lane == 31) { s_c[warp] = ci; s_t[warp] = ti; }
  __syncthreads();
  int cb = 0; long long tb = 0; c_tot = 0; t_tot = 0;
#pragma unroll
  for (int w = 0; w < kWarps; ++w) {
    if (w < warp) { cb += s_c[w]; tb += s_t[w]; }
    c_tot += s_c[w]; t_tot += s_t[w];
  }
  c_ex = cb + ci - c;
  t_ex = tb + ti - t;
}

__device__ __forceinline__ void segment_of(int64_t N, int block, int grid, int64_t& q0, int64_t& q1) {
  const int64_t Q = (N + kQuad - 1) / kQuad;              // quads in the table
  const int64_t per = (Q + grid - 1) / grid;
  q0 = per * block < Q ? per * block : Q;
  q1 = q0 + per < Q ? q0 + per : Q;
}

// Pass 1: aggregate of each block's segment.  Block 0 also clears the result record.
__global__ void __launch_bounds__(kThreads) controller_count_kernel(
    const uint32_t* __restrict__ ready, const uint32_t* __restrict__ consumed, const int32_t* __restrict__ length,
    int64_t N, uint32_t mask, uint32_t task_bit, int vec_ok, Agg* __restrict__ agg, af_get_result* __restrict__ out) {
  __shared__ int s_c[kWarps];
  __shared__ long long s_t[kWarps];
  __shared__ int s_first;
  if (threadIdx.x == 0) s_first = INT_MAX;
  __syncthreads();
  int64_t q0, q1;
  segment_of(N, blockIdx.x, gridDim.x, q0, q1);
  int c = 0; long long t = 0;
  int tile = 0, first = INT_MAX;                          // tile index within the segment (fits: N < 2^31)
  int64_t q = q0 + threadIdx.x;
  for (; q + kThreads < q1; q += 2 * kThreads, tile += 2) {   // two independent quads in flight per thread
    const Quad v0 = load_quad(ready, consumed, length, q * kQuad, N, mask, task_bit, vec_ok != 0);
    const Quad v1 = load_quad(ready, consumed, length, (q + kThreads) * kQuad, N, mask, task_bit, vec_ok != 0);
    int c0 = 0, c1 = 0;
#pragma unroll
    for (int k = 0; k < kQuad; ++k) { c0 += v0.elig[k]; c1 += v1.elig[k]; t += v0.len[k] + v1.len[k]; }
    if (first == INT_MAX && (c0 | c1)) first = c0 ? tile : tile + 1;
    c += c0 + c1;
  }
  for (; q < q1; q += kThreads, ++tile) {
    const Quad v = load_quad(ready, consumed, length, q * kQuad, N, mask, task_bit, vec_ok != 0);
    int c0 = 0;
#pragma unroll
    for (int k = 0; k < kQuad; ++k) { c0 += v.elig[k]; t += v.len[k]; }
    if (first == INT_MAX && c0) first = tile;
    c += c0;
  }
  if (first != INT_MAX) atomicMin(&s_first, first);
  int c_ex, c_tot; long long t_ex, t_tot;
  block_scan(c, t, c_ex, t_ex, c_tot, t_tot, s_c, s_t);   // its barriers also order s_first
  if (threadIdx.x == 0) {
    agg[blockIdx.x] = Agg{c_tot, s_first == INT_MAX ? 0 : s_first, t_tot};
    if (blockIdx.x == 0) { out->count = 0; out->eligible = 0; out->tokens = 0; }
  }
}

// Pass 2 (or the only pass when the grid is one block): ordered selection.
__global__ void __launch_bounds__(kThreads) controller_select_kernel(
    const uint32_t* __restrict__ ready, uint32_t* __restrict__ consumed, const int32_t* __restrict__ length,
    int64_t N, uint32_t mask, uint32_t task_bit, int vec_ok, int max_samples, long long token_budget,
    const Agg* __restrict__ agg, int32_t* __restrict__ out_idx, af_get_result* __restrict__ out) {
  __shared__ int s_c[kWarps];
  __shared__ long long s_t[kWarps];
  const bool single = gridDim.x == 1;
  // rank and tokens of the eligible samples before this block's segment; block 0 also totals
  int base_c = 0; long long base_t = 0;
  if (!single) {
    int c = 0; long long t = 0, all_c = 0;
    const int upto = blockIdx.x == 0 ? gridDim.x : blockIdx.x;
    for (int b = threadIdx.x; b < upto; b += kThreads) {
      const Agg a = agg[b];
      if (b < (int)blockIdx.x) { c += a.count; t += a.tokens; }
      all_c += a.count;
    }
    int c_ex, c_tot; long long t_ex, t_tot;
    block_scan(c, t, c_ex, t_ex, c_tot, t_tot, s_c, s_t);
    base_c = c_tot; base_t = t_tot;
    if (blockIdx.x == 0) {
      int d0, all_tot; long long d1, d2;
      block_scan((int)all_c, 0, d0, d1, all_tot, d2, s_c, s_t);
      if (threadIdx.x == 0) out->eligible = all_tot;
    }
    // the prefix has ended before this segment, or the segment holds no eligible sample:
    // nothing here can be selected (block-uniform)
    if (base_c >= max_samples || (token_budget > 0 && base_c > 0 && base_t > token_budget)) return;
    if (agg[blockIdx.x].count == 0) return;
  }
  int64_t q0, q1;
  segment_of(N, blockIdx.x, gridDim.x, q0, q1);
  int run_c = base_c; long long run_t = base_t;          // eligible seen so far, in index order
  int sel_c = 0; long long sel_t = 0;                    // selected by this thread
  int elig_c = 0;
  // tiles before the segment's first eligible sample need no visit (pass 1 recorded where it is)
  const int64_t q_start = single ? q0 : q0 + (int64_t)agg[blockIdx.x].first_tile * kThreads;
  for (int64_t qb = q_start; qb < q1; qb += kThreads) {   // block-uniform trip count
    const int64_t q = qb + threadIdx.x;
    Quad v;
    if (q < q1) {
      v = load_quad(ready, consumed, length, q * kQuad, N, mask, task_bit, vec_ok != 0);
    } else {
#pragma unroll
      for (int k = 0; k < kQuad; ++k) { v.elig[k] = 0; v.len[k] = 0; }
    }
    int c = 0; long long t = 0;
#pragma unroll
    for (int k = 0; k < kQuad; ++k) { c += v.elig[k]; t += v.len[k]; }
    int c_ex, c_tot; long long t_ex, t_tot;
    block_scan(c, t, c_ex, t_ex, c_tot, t_tot, s_c, s_t);
    int rank = run_c + c_ex; long long tok = run_t + t_ex;
#pragma unroll
    for (int k = 0; k < kQuad; ++k) {
      if (v.elig[k]) {
        tok += v.len[k];                                  // inclusive token prefix
        const bool take = rank < max_samples && (token_budget <= 0 || tok <= token_budget || rank == 0);
        if (take) {
          const int64_t i = q * kQuad + k;
          out_idx[rank] = (int32_t)i;
          consumed[i] |= task_bit;                        // only this thread touches sample i in this launch
          ++sel_c; sel_t += v.len[k];
        }
        ++rank;
      }
    }
    elig_c += c;
    run_c += c_tot; run_t += t_tot;
    if (run_c >= max_samples || (token_budget > 0 && run_t > token_budget && run_c > 0)) {
      if (!single) break;                                 // block-uniform: the prefix ends in this tile
    }
  }
  // block totals of what was selected
  int d0, c_tot; long long d1, t_tot;
  block_scan(sel_c, sel_t, d0, d1, c_tot, t_tot, s_c, s_t);
  if (single) {
    int e0, e_tot; long long e1, e2;
    block_scan(elig_c, 0, e0, e1, e_tot, e2, s_c, s_t);
    if (threadIdx.x == 0) { out->count = c_tot; out->eligible = e_tot; out->tokens = t_tot; }
  } else if (threadIdx.x == 0 && c_tot > 0) {
    atomicAdd(&out->count, c_tot);
    atomicAdd(reinterpret_cast<unsigned long long*>(&out->tokens), (unsigned long long)t_tot);
  }
}

__global__ void __launch_bounds__(kThreads) controller_put_kernel(uint32_t* __restrict__ ready,
                                                                 const int32_t* __restrict__ idx, int64_t n,
                                                                 int64_t N, uint32_t bits, unsigned int* d_err) {
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; j < n; j += stride) {
    const int64_t i = __ldg(idx + j);
    if (i < 0 || i >= N) { atomicOr(d_err, AF_DEVERR_SAMPLE_INDEX); continue; }
    atomicOr(ready + i, bits);
  }
}

// Four samples per thread with 128-bit accesses (tail and unaligned tables: one sample per thread),
// one block per 4 KB run of the table in address order.
__global__ void __launch_bounds__(kThreads) controller_clear_kernel(uint32_t* __restrict__ ready,
                                                                   uint32_t* __restrict__ consumed, int64_t N,
                                                                   uint32_t column_bits, uint32_t task_bits, int vec_ok) {
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  const int64_t n_vec = vec_ok ? N / 4 : 0;
  const uint32_t keep_r = ~column_bits, keep_c = ~task_bits;
  for (int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; v < n_vec; v += stride) {
    if (column_bits) {
      uint4 r = __ldcs(reinterpret_cast<const uint4*>(ready) + v);
      r.x &= keep_r; r.y &= keep_r; r.z &= keep_r; r.w &= keep_r;
      __stcs(reinterpret_cast<uint4*>(ready) + v, r);
    }
    if (task_bits) {
      uint4 c = __ldcs(reinterpret_cast<const uint4*>(consumed) + v);
      c.x &= keep_c; c.y &= keep_c; c.z &= keep_c; c.w &= keep_c;
      __stcs(reinterpret_cast<uint4*>(consumed) + v, c);
    }
  }
  for (int64_t i = n_vec * 4 + (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < N; i += stride) {
    if (column_bits) ready[i] &= keep_r;
    if (task_bits) consumed[i] &= keep_c;
  }
}

inline int grid_for(int64_t items, int sm_count) {
  int64_t b = (items + kThreads - 1) / kThreads;
  if (b < 1) b = 1;
  if (b > (int64_t)sm_count * 8) b = (int64_t)sm_count * 8;
  return (int)b;
}

}  // namespace

size_t controller_workspace_bytes(int sm_count) { return (size_t)sm_count * 8 * sizeof(Agg); }

cudaError_t launch_controller_put(const af_controller_view& v, const int32_t* idx, int64_t n, uint32_t bits,
                                  unsigned int* d_err, int sm_count, cudaStream_t s) {
  if (n == 0 || bits == 0) return cudaSuccess;
  controller_put_kernel<<<grid_for(n, sm_count), kThreads, 0, s>>>(v.ready, idx, n, v.n_samples, bits, d_err);
  return cudaGetLastError();
}

cudaError_t launch_controller_clear(const af_controller_view& v, uint32_t column_bits, uint32_t task_bits,
                                    int sm_count, cudaStream_t s) {
  if (v.n_samples == 0 || (column_bits == 0 && task_bits == 0)) return cudaSuccess;
  const int vec_ok = ((reinterpret_cast<uintptr_t>(v.ready) | reinterpret_cast<uintptr_t>(v.consumed)) & 15) == 0;
  int64_t blocks = ((vec_ok ? v.n_samples / 4 : v.n_samples) + kThreads - 1) / kThreads;
  if (blocks < 1) blocks = 1;
  if (blocks > (int64_t)1 << 30) blocks = (int64_t)1 << 30;
  (void)sm_count;
  controller_clear_kernel<<<(int)blocks, kThreads, 0, s>>>(v.ready, v.consumed, v.n_samples, column_bits, task_bits,
                                                          vec_ok);
  return cudaGetLastError();
}

cudaError_t launch_controller_get(const af_controller_view& v, uint32_t mask, uint32_t task_bit, int32_t max_samples,
                                  int64_t token_budget, int32_t* out_idx, af_get_result* out, void* ws,
                                  int sm_count, cudaStream_t s) {
  const int64_t N = v.n_samples;
  auto al = [](const void* q) { return (reinterpret_cast<uintptr_t>(q) & 15) == 0; };
  const int vec_ok = al(v.ready) && al(v.consumed) && (v.length == nullptr || al(v.length));
  int grid = 1;
  if (N > kSingleBlockMax) {
    const int64_t tiles = (N + kTile - 1) / kTile;
    grid = (int)(tiles < (int64_t)sm_count * 8 ? tiles : (int64_t)sm_count * 8);
    controller_count_kernel<<<grid, kThreads, 0, s>>>(v.ready, v.consumed, v.length, N, mask, task_bit, vec_ok,
                                                      static_cast<Agg*>(ws), out);
  }
  controller_select_kernel<<<grid, kThreads, 0, s>>>(v.ready, v.consumed, v.length, N, mask, task_bit, vec_ok,
                                                     max_samples, token_budget, static_cast<const Agg*>(ws),
                                                     out_idx, out);
  return cudaGetLastError();
}

}  // namespace af

// ---------------------------------------------------------------------------------------------
// af_balance_partitions (host): k-way largest differencing method.
// ---------------------------------------------------------------------------------------------
namespace {

struct Group {          // one group of a partial solution: token sum and a linked list of its items
  int64_t sum;
  int32_t head, tail;   // -1 when empty
};
struct Partial {        // k groups in decreasing order of sum
  int64_t spread;
  int64_t id;           // creation order, breaks ties between equal spreads
  std::vector<Group> g;
};
struct BySpread {
  bool operator()(const Partial* a, const Partial* b) const {   // priority queue: "less" = comes later
    if (a->spread != b->spread) return a->spread < b->spread;
    return a->id > b->id;
  }
};

}  // namespace

extern "C" af_status af_balance_partitions(const int32_t* length_host, int32_t n, int32_t k, int32_t equal_size,
                                           int32_t* part_host, int64_t* group_tokens_host) {
  if (n < 0 || k < 1 || (n > 0 && (!length_host || !part_host))) return AF_ERR_INVALID_ARG;
  if (group_tokens_host) std::fill(group_tokens_host, group_tokens_host + k, (int64_t)0);
  if (n == 0) return AF_OK;
  for (int32_t i = 0; i < n; ++i) if (length_host[i] < 0) return AF_ERR_INVALID_ARG;
  try {
    std::vector<int32_t> order(n), next(n, -1);
    for (int32_t i = 0; i < n; ++i) order[i] = i;
    std::stable_sort(order.begin(), order.end(),
                     [&](int32_t a, int32_t b) { return length_host[a] > length_host[b]; });  // ties: index ascending
    std::vector<Partial> pool;
    pool.reserve((size_t)2 * n + 2);
    auto single = [&](int32_t item) { return Group{(int64_t)length_host[item], item, item}; };
    const Group empty{0, -1, -1};
    int64_t next_id = 0;
    if (equal_size) {
      for (int32_t s = 0; s < n; s += k) {
        Partial p; p.id = next_id++; p.g.assign(k, empty);
        for (int32_t j = 0; j < k && s + j < n; ++j) p.g[j] = single(order[s + j]);
        p.spread = p.g.front().sum - p.g.back().sum;
        pool.push_back(std::move(p));
      }
    } else {
      for (int32_t q = 0; q < n; ++q) {
        Partial p; p.id = next_id++; p.g.assign(k, empty);
        p.g[0] = single(order[q]);
        p.spread = p.g.front().sum - p.g.back().sum;
        pool.push_back(std::move(p));
      }
    }
    std::priority_queue<Partial*, std::vector<Partial*>, BySpread> heap;
    for (Partial& p : pool) heap.push(&p);
    while (heap.size() > 1) {
      Partial* a = heap.top(); heap.pop();
      Partial* b = heap.top(); heap.pop();
      Partial m; m.id = next_id++; m.g.resize(k);
      for (int32_t j = 0; j < k; ++j) {           // j-th largest of a with j-th smallest of b
        const Group& x = a->g[j];
        const Group& y = b->g[k - 1 - j];
        Group z{x.sum + y.sum, x.head, x.tail};
        if (x.head < 0) { z.head = y.head; z.tail = y.tail; }
        else if (y.head >= 0) { next[x.tail] = y.head; z.tail = y.tail; }
        m.g[j] = z;
      }
      std::stable_sort(m.g.begin(), m.g.end(), [](const Group& p, const Group& q) { return p.sum > q.sum; });
      m.spread = m.g.front().sum - m.g.back().sum;
      a->g.clear(); a->g.shrink_to_fit(); b->g.clear(); b->g.shrink_to_fit();
      pool.push_back(std::move(m));               // reserved: pointers into the pool stay valid
      heap.push(&pool.back());
    }
    const Partial* fin = heap.top();
    for (int32_t gi = 0; gi < k; ++gi) {
      for (int32_t i = fin->g[gi].head; i >= 0; i = next[i]) part_host[i] = gi;
      if (group_tokens_host) group_tokens_host[gi] = fin->g[gi].sum;
    }
  } catch (const std::bad_alloc&) {
    return AF_ERR_WORKSPACE;
  }
  return AF_OK;
}
