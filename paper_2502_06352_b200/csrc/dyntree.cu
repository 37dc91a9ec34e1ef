// Dynamic-tree drafting (Sec. 2.1, the dynamic variant of tree drafting; Sec. 3 "Shallow draft trees"):
// every draft node carries log V = sum of the logs of the drafter's confidences along its path.
//   expand_rows_kernel   one CTA per frontier node: the K most confident tokens of its drafter row
//                        become candidates (token, parent, log V, depth) in the sequence's pool;
//   select_frontier_kernel  one CTA per sequence: the E candidates of this depth with the largest
//                        log V form the next frontier;
//   trim_tree_kernel     one CTA per sequence: the m - 1 pool entries with the largest log V and
//                        the root, renumbered breadth first (the numbering lantern_tree_create wants).
// Orders of equal values: tokens of a row by (z descending, token ascending), candidates by
// (log V descending, pool index ascending); a parent therefore always ranks before its children.
#include <cmath>

#include "common.cuh"

namespace lantern {

template <typename T> __device__ __forceinline__ float dyn_widen(T x);
template <> __device__ __forceinline__ float dyn_widen<float>(float x) { return x; }
template <> __device__ __forceinline__ float dyn_widen<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }

constexpr int kDynThreads = 256;
constexpr int kDynMaxPool = 2048;

struct ExpandArgs {
  const void *dc, *du;
  long long row_stride, seq_stride;
  int B, F, K, E, V, allow_lo, allow_hi;
  float g, inv_tau;
  const int32_t* frontier;           // [B][F] pool index of the node in each slot, -1: empty slot
  int P, pool_off, depth;
  int32_t *pool_parent, *pool_token, *pool_depth;
  double* pool_logv;
  int32_t* next_frontier;            // [B][E]
};

// (value, index) maximum with ties to the lower index, over the CTA; result in every thread
__device__ __forceinline__ void block_best(float& z, int& j, float* sz, int* sj) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float oz = __shfl_xor_sync(0xffffffffu, z, o);
    const int oj = __shfl_xor_sync(0xffffffffu, j, o);
    if (oz > z || (oz == z && oj < j)) { z = oz; j = oj; }
  }
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane == 0) { sz[warp] = z; sj[warp] = j; }
  __syncthreads();
  z = sz[0]; j = sj[0];
  for (int w = 1; w < kDynThreads / 32; ++w)
    if (sz[w] > z || (sz[w] == z && sj[w] < j)) { z = sz[w]; j = sj[w]; }
  __syncthreads();
}

template <typename T>
__global__ void __launch_bounds__(kDynThreads) expand_rows_kernel(const ExpandArgs a) {
  __shared__ float sz[kDynThreads / 32];
  __shared__ int sj[kDynThreads / 32];
  __shared__ double sd[kDynThreads / 32];
  const int f = blockIdx.x, b = blockIdx.y, tid = threadIdx.x;
  const int node = a.frontier[b * a.F + f];
  const long long pbase = static_cast<long long>(b) * a.P + a.pool_off + f * a.K;
  if (node < 0) {                                   // empty slot: candidates that can never be chosen
    for (int r = tid; r < a.K; r += kDynThreads) {
      a.pool_parent[pbase + r] = -1;
      a.pool_token[pbase + r] = -1;
      a.pool_depth[pbase + r] = a.depth;
      a.pool_logv[pbase + r] = -INFINITY;
    }
    return;
  }
  const T* c = static_cast<const T*>(a.dc) + b * a.seq_stride + f * a.row_stride;
  const T* u = a.du ? static_cast<const T*>(a.du) + b * a.seq_stride + f * a.row_stride : nullptr;
  // the float32 pre-softmax value of a token: the row post-processing of every other entry point
  auto zof = [&](int j) {
    const float cc = dyn_widen<T>(c[j]);
    if (u) { const float uu = dyn_widen<T>(u[j]); return __fmul_rn(__fmaf_rn(a.g, __fsub_rn(cc, uu), uu), a.inv_tau); }
    return __fmul_rn(cc, a.inv_tau);
  };
  // maximum, then the softmax denominator (terms in float32, sum in double)
  float m = -INFINITY;
  int mj = 0x7fffffff;
  for (int j = a.allow_lo + tid; j < a.allow_hi; j += kDynThreads) {
    const float z = zof(j);
    if (z > m) { m = z; mj = j; }
  }
  block_best(m, mj, sz, sj);
  double s = 0.0;
  for (int j = a.allow_lo + tid; j < a.allow_hi; j += kDynThreads) s += static_cast<double>(expf(zof(j) - m));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  if ((tid & 31) == 0) sd[tid >> 5] = s;
  __syncthreads();
  s = 0.0;
  for (int w = 0; w < kDynThreads / 32; ++w) s += sd[w];
  const double ln_s = log(s);
  const double parent_logv = a.pool_logv[static_cast<long long>(b) * a.P + node];
  // K rounds: the best token that comes after the last pick in the order (z descending, id ascending)
  float pz = INFINITY;
  int pj = -1;
  for (int r = 0; r < a.K; ++r) {
    float bz = -INFINITY;
    int bj = 0x7fffffff;
    for (int j = a.allow_lo + tid; j < a.allow_hi; j += kDynThreads) {
      const float z = zof(j);
      const bool after = z < pz || (z == pz && j > pj);
      if (after && (z > bz || (z == bz && j < bj))) { bz = z; bj = j; }
    }
    block_best(bz, bj, sz, sj);
    if (tid == 0) {
      const bool found = bj != 0x7fffffff;          // fewer than K allowed tokens: the rest can never be chosen
      a.pool_parent[pbase + r] = found ? node : -1;
      a.pool_token[pbase + r] = found ? bj : -1;
      a.pool_depth[pbase + r] = a.depth;
      a.pool_logv[pbase + r] = found ? parent_logv + ((static_cast<double>(bz) - static_cast<double>(m)) - ln_s) : -INFINITY;
    }
    pz = bz;
    pj = bj;
  }
}

// rank of entry i among n entries by (value descending, index ascending); -inf entries rank last
__device__ __forceinline__ int rank_desc(const double* v, int n, int i) {
  const double vi = v[i];
  int r = 0;
  for (int j = 0; j < n; ++j) {
    const double vj = v[j];
    r += (vj > vi || (vj == vi && j < i)) ? 1 : 0;
  }
  return r;
}

__global__ void __launch_bounds__(kDynThreads) select_frontier_kernel(const ExpandArgs a) {
  extern __shared__ double dyn_lv[];
  const int b = blockIdx.x, tid = threadIdx.x, T = a.F * a.K;
  const double* lv = a.pool_logv + static_cast<long long>(b) * a.P + a.pool_off;
  for (int i = tid; i < T; i += kDynThreads) dyn_lv[i] = lv[i];
  for (int e = tid; e < a.E; e += kDynThreads) a.next_frontier[b * a.E + e] = -1;
  __syncthreads();
  for (int i = tid; i < T; i += kDynThreads) {
    if (dyn_lv[i] == -INFINITY) continue;
    const int r = rank_desc(dyn_lv, T, i);
    if (r < a.E) a.next_frontier[b * a.E + r] = a.pool_off + i;
  }
}

struct TrimArgs {
  int B, P, used, m, max_depth;
  const int32_t *pool_parent, *pool_token, *pool_depth;
  const double* pool_logv;
  int32_t *n_nodes, *parent, *token, *pool_index;
  double* logv;
};

__global__ void __launch_bounds__(kDynThreads) trim_tree_kernel(const TrimArgs a) {
  extern __shared__ double dyn_lv[];                 // [used] log V | new id [used] | selected [used]
  int* newid = reinterpret_cast<int*>(dyn_lv + a.used);
  int* sel = newid + a.used;
  __shared__ int count, level_n;
  const int b = blockIdx.x, tid = threadIdx.x, n = a.used;
  const long long base = static_cast<long long>(b) * a.P;
  for (int i = tid; i < n; i += kDynThreads) {
    dyn_lv[i] = i == 0 ? INFINITY : a.pool_logv[base + i];      // the root ranks first
    newid[i] = -1;
  }
  __syncthreads();
  for (int i = tid; i < n; i += kDynThreads)
    sel[i] = (i == 0 || (dyn_lv[i] != -INFINITY && rank_desc(dyn_lv, n, i) < a.m)) ? 1 : 0;
  if (tid == 0) { count = 1; newid[0] = 0; }
  __syncthreads();
  // breadth-first numbering: a level is ordered by (new id of the parent, pool index)
  for (int dep = 1; dep <= a.max_depth; ++dep) {
    if (tid == 0) level_n = 0;
    __syncthreads();
    const int start = count;
    for (int i = tid; i < n; i += kDynThreads) {
      if (!sel[i] || a.pool_depth[base + i] != dep) continue;
      const int pi = newid[a.pool_parent[base + i]];
      int pos = 0;
      for (int j = 1; j < n; ++j) {
        if (!sel[j] || j == i || a.pool_depth[base + j] != dep) continue;
        const int pj = newid[a.pool_parent[base + j]];
        pos += (pj < pi || (pj == pi && j < i)) ? 1 : 0;
      }
      const int id = start + pos;
      const long long o = static_cast<long long>(b) * a.m + id;
      a.parent[o] = pi;
      a.token[o] = a.pool_token[base + i];
      a.pool_index[o] = i;
      a.logv[o] = a.pool_logv[base + i];
      atomicAdd(&level_n, 1);
      // the id is published after the level is complete (below), so this level's reads see parents only
      sel[i] = 2 + id;
    }
    __syncthreads();
    for (int i = tid; i < n; i += kDynThreads)
      if (sel[i] >= 2) { newid[i] = sel[i] - 2; sel[i] = 1; }
    if (tid == 0) count = start + level_n;
    __syncthreads();
  }
  if (tid == 0) {
    const long long o = static_cast<long long>(b) * a.m;
    a.parent[o] = -1; a.token[o] = -1; a.pool_index[o] = 0; a.logv[o] = 0.0;
    a.n_nodes[b] = count;
  }
  for (int i = count + tid; i < a.m; i += kDynThreads) {       // unused tail of the outputs
    const long long o = static_cast<long long>(b) * a.m + i;
    a.parent[o] = -1; a.token[o] = -1; a.pool_index[o] = -1; a.logv[o] = -INFINITY;
  }
}

}  // namespace lantern

using namespace lantern;

extern "C" lantern_status lantern_expand_frontier(const lantern_params* p, const void* draft_cond, const void* draft_uncond,
                                                  lantern_dtype dt, int64_t row_stride, int64_t seq_stride, int32_t batch,
                                                  int32_t n_frontier, int32_t n_children, int32_t n_expand,
                                                  const int32_t* frontier, int32_t pool_size, int32_t pool_offset,
                                                  int32_t depth, int32_t* pool_parent, int32_t* pool_token,
                                                  double* pool_logv, int32_t* pool_depth, int32_t* next_frontier,
                                                  void* stream) {
  if (!p || !draft_cond || !frontier || !pool_parent || !pool_token || !pool_logv || !pool_depth || !next_frontier)
    return LANTERN_ERR_INVALID_ARG;
  if (dt != LANTERN_F32 && dt != LANTERN_BF16) return LANTERN_ERR_INVALID_ARG;
  if (batch <= 0 || n_frontier <= 0 || p->vocab <= 0 || !(p->temperature > 0.f) || depth < 1) return LANTERN_ERR_INVALID_ARG;
  if (n_children < 1 || n_children > LANTERN_MAX_CHILDREN || n_expand < 1) return LANTERN_ERR_INVALID_ARG;
  if (p->top_k_draft != 0) return LANTERN_ERR_UNSUPPORTED;          // confidences of truncated rows: not built
  const long long T = static_cast<long long>(n_frontier) * n_children;
  if (T > kDynMaxPool || pool_size > kDynMaxPool) return LANTERN_ERR_UNSUPPORTED;
  if (pool_offset < 1 || pool_offset + T > pool_size) return LANTERN_ERR_INVALID_ARG;
  const int V = p->vocab, lo = p->allowed_begin, hi = p->allowed_end == 0 ? V : p->allowed_end;
  if (lo < 0 || hi > V || lo >= hi) return LANTERN_ERR_INVALID_ARG;
  if (row_stride < V || seq_stride < 0) return LANTERN_ERR_INVALID_ARG;
  ExpandArgs a;
  a.dc = draft_cond; a.du = draft_uncond; a.row_stride = row_stride; a.seq_stride = seq_stride;
  a.B = batch; a.F = n_frontier; a.K = n_children; a.E = n_expand; a.V = V; a.allow_lo = lo; a.allow_hi = hi;
  a.g = p->cfg_scale; a.inv_tau = 1.0f / p->temperature;
  a.frontier = frontier; a.P = pool_size; a.pool_off = pool_offset; a.depth = depth;
  a.pool_parent = pool_parent; a.pool_token = pool_token; a.pool_depth = pool_depth; a.pool_logv = pool_logv;
  a.next_frontier = next_frontier;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const dim3 grid(n_frontier, batch);
  if (dt == LANTERN_F32) expand_rows_kernel<float><<<grid, kDynThreads, 0, st>>>(a);
  else expand_rows_kernel<__nv_bfloat16><<<grid, kDynThreads, 0, st>>>(a);
  if (cudaGetLastError() != cudaSuccess) return LANTERN_ERR_CUDA;
  select_frontier_kernel<<<batch, kDynThreads, static_cast<size_t>(T) * sizeof(double), st>>>(a);
  return cudaGetLastError() == cudaSuccess ? LANTERN_OK : LANTERN_ERR_CUDA;
}

extern "C" lantern_status lantern_trim_tree(int32_t batch, int32_t pool_size, int32_t pool_used, int32_t max_depth,
                                            const int32_t* pool_parent, const int32_t* pool_token, const double* pool_logv,
                                            const int32_t* pool_depth, int32_t max_nodes, int32_t* n_nodes, int32_t* parent,
                                            int32_t* token, int32_t* pool_index, double* logv, void* stream) {
  if (!pool_parent || !pool_token || !pool_logv || !pool_depth || !n_nodes || !parent || !token || !pool_index || !logv)
    return LANTERN_ERR_INVALID_ARG;
  if (batch <= 0 || pool_used < 1 || pool_used > pool_size || max_nodes < 1 || max_depth < 0) return LANTERN_ERR_INVALID_ARG;
  if (pool_size > kDynMaxPool || max_nodes > LANTERN_MAX_NODES) return LANTERN_ERR_UNSUPPORTED;
  TrimArgs a;
  a.B = batch; a.P = pool_size; a.used = pool_used; a.m = max_nodes; a.max_depth = max_depth;
  a.pool_parent = pool_parent; a.pool_token = pool_token; a.pool_depth = pool_depth; a.pool_logv = pool_logv;
  a.n_nodes = n_nodes; a.parent = parent; a.token = token; a.pool_index = pool_index; a.logv = logv;
  trim_tree_kernel<<<batch, kDynThreads, static_cast<size_t>(pool_used) * 16, static_cast<cudaStream_t>(stream)>>>(a);
  return cudaGetLastError() == cudaSuccess ? LANTERN_OK : LANTERN_ERR_CUDA;
}
