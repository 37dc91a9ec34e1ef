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

#include "rowops.cuh"

namespace lantern {

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

constexpr int kDynList = 1024;          // tokens at or above the row's selection threshold

// Visits every allowed token of a row once: 16-byte vector loads over the aligned middle (when the
// row pointers allow it), scalar loads at the ragged ends.  fn(j, z) per token; fold() after every
// vector and after every scalar token.
template <typename T, bool CFG, typename F, typename G>
__device__ __forceinline__ void for_each_z(const T* c, const T* u, float g, float inv_tau, int lo, int hi, F&& fn, G&& fold) {
  constexpr int VN = Vec<T>::N;
  auto z1 = [&](float cc, float uu) { return combine<CFG>(cc, uu, g, inv_tau); };
  const bool aligned = (reinterpret_cast<uintptr_t>(c) % 16 == 0) && (!CFG || reinterpret_cast<uintptr_t>(u) % 16 == 0);
  int v0 = lo, v1 = lo;                                 // vector part [v0, v1)
  if (aligned) {
    v0 = (lo + VN - 1) / VN * VN;
    v1 = hi / VN * VN;
    if (v1 < v0) v1 = v0;
  }
  const int tid = threadIdx.x;
  for (int j = lo + tid; j < (aligned ? min(v0, hi) : hi); j += kDynThreads) {
    fn(j, z1(Vec<T>::widen(c[j]), CFG ? Vec<T>::widen(u[j]) : 0.f));
    fold();
  }
  if (!aligned) return;
  constexpr int UV = 4;                                 // vectors a thread keeps in flight (more would only grow the code)
  for (int j0 = v0 + tid * VN; j0 < v1; j0 += kDynThreads * VN * UV) {
    uint4 rc[UV], ru[UV];
#pragma unroll
    for (int q = 0; q < UV; ++q) {
      const int j = j0 + q * kDynThreads * VN;
      if (j < v1) {
        rc[q] = ldg_stream_u128(c + j);
        if (CFG) ru[q] = ldg_stream_u128(u + j);
      }
    }
#pragma unroll
    for (int q = 0; q < UV; ++q) {
      const int j = j0 + q * kDynThreads * VN;
      if (j < v1) {
        float cf[VN], uf[VN];
        Vec<T>::unpack_raw(rc[q], cf);
        if (CFG) Vec<T>::unpack_raw(ru[q], uf);
#pragma unroll
        for (int e = 0; e < VN; ++e) fn(j + e, z1(cf[e], CFG ? uf[e] : 0.f));
        fold();
      }
    }
  }
  for (int j = max(v1, v0) + tid; j < hi; j += kDynThreads) {
    fn(j, z1(Vec<T>::widen(c[j]), CFG ? Vec<T>::widen(u[j]) : 0.f));
    fold();
  }
}

// The round of the fallback path: best token after (pz, pj) over the whole row, scalar loads.  Kept out
// of line so that this rarely used scan does not grow the kernel's main loops.
template <typename T>
__device__ __noinline__ void scan_row_after(const T* c, const T* u, float g, float inv_tau, int lo, int hi, float pz, int pj,
                                            float& bz, int& bj) {
  for (int j = lo + threadIdx.x; j < hi; j += kDynThreads) {
    const float z = u ? combine<true>(Vec<T>::widen(c[j]), Vec<T>::widen(u[j]), g, inv_tau)
                      : combine<false>(Vec<T>::widen(c[j]), 0.f, g, inv_tau);
    const bool after = z < pz || (z == pz && j > pj);
    if (after && (z > bz || (z == bz && j < bj))) { bz = z; bj = j; }
  }
}

// One frontier row.  Pass 1 (from HBM): every thread's maximum; the K-th largest of the warps' two
// largest thread maxima each is a lower bound tau of the row's K-th largest value.  Pass 2 (the row is in L2 now): the
// softmax denominator, and the tokens with z >= tau go to a short list in shared memory, from which
// K rounds pick the children in the order (z descending, token ascending).  A list that overflows
// (thousands of equal values) falls back to K rounds over the row.
template <typename T, bool CFG>
__global__ void __launch_bounds__(kDynThreads) expand_rows_kernel(const ExpandArgs a) {
  __shared__ float sz[kDynThreads / 32];
  __shared__ int sj[kDynThreads / 32];
  __shared__ double sd[kDynThreads / 32];
  __shared__ float tmax[2 * (kDynThreads / 32)];
  __shared__ float lz[kDynList];
  __shared__ int lj[kDynList];
  __shared__ int lcount;
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
  const T* u = CFG ? static_cast<const T*>(a.du) + b * a.seq_stride + f * a.row_stride : nullptr;
  // pass 1 (from HBM): maxima only
  float m = -INFINITY;
  for_each_z<T, CFG>(c, u, a.g, a.inv_tau, a.allow_lo, a.allow_hi, [&](int, float z) { m = fmaxf(m, z); }, [] {});
  // the two largest thread maxima of every warp: 16 values of distinct tokens, whose K-th largest
  // (K <= 8) is a lower bound tau of the row's K-th largest value; every warp ranks them for itself
  {
    const int lane = tid & 31, warp = tid >> 5;
    const float w1 = warp_max(m);
    const int wl = __ffs(__ballot_sync(0xffffffffu, m == w1)) - 1;
    const float w2 = warp_max(lane == wl ? -INFINITY : m);
    if (lane == 0) { tmax[2 * warp] = w1; tmax[2 * warp + 1] = w2; }
  }
  if (tid == 0) lcount = 0;
  float bm = m;
  int bj = tid;
  block_best(bm, bj, sz, sj);                       // bm: the row's maximum (the barriers inside publish tmax and lcount too)
  float tau = -INFINITY;
  {
    const int lane = tid & 31;
    constexpr int NV = 2 * (kDynThreads / 32);
    const float v = lane < NV ? tmax[lane] : -INFINITY;
    int r = 0;
#pragma unroll
    for (int i = 0; i < NV; ++i) {
      const float o = __shfl_sync(0xffffffffu, v, i);
      r += (o > v || (o == v && i < lane)) ? 1 : 0;
    }
    const uint32_t hit = __ballot_sync(0xffffffffu, lane < NV && r == min(a.K, NV) - 1);
    tau = __shfl_sync(0xffffffffu, v, __ffs(hit) - 1);
  }
  // pass 2 (the row is in L2 now): softmax denominator relative to the row maximum, terms in float32,
  // a vector's terms summed in float32 and folded into a double (double-precision work is slow on this
  // part, so it stays at one addition per vector); tokens at or above tau go to the list
  double s = 0.0;
  float part = 0.f;
  for_each_z<T, CFG>(c, u, a.g, a.inv_tau, a.allow_lo, a.allow_hi,
                [&](int j, float z) {
                  part += ex2_approx(__fmul_rn(__fsub_rn(z, bm), kLog2e));   // exp(z - max): the argument's rounding costs
                                                                             // |z - max| 2^-24 relative on a term of weight exp(z - max)
                  if (z >= tau) {
                    const int pos = atomicAdd(&lcount, 1);
                    if (pos < kDynList) { lz[pos] = z; lj[pos] = j; }
                  }
                },
                [&] { s += static_cast<double>(part); part = 0.f; });
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  if ((tid & 31) == 0) sd[tid >> 5] = s;
  __syncthreads();
  s = 0.0;
  for (int w = 0; w < kDynThreads / 32; ++w) s += sd[w];
  const double ln_s = log(s);
  const double parent_logv = a.pool_logv[static_cast<long long>(b) * a.P + node];
  __syncthreads();
  const int n = lcount;
  const bool listed = n <= kDynList;
  float pz = INFINITY;
  int pj = -1;
  for (int r = 0; r < a.K; ++r) {
    float bz = -INFINITY;
    int bjj = 0x7fffffff;
    if (listed) {
      for (int i = tid; i < n; i += kDynThreads) {
        const float z = lz[i];
        const int j = lj[i];
        const bool after = z < pz || (z == pz && j > pj);
        if (after && (z > bz || (z == bz && j < bjj))) { bz = z; bjj = j; }
      }
    } else {
      scan_row_after<T>(c, u, a.g, a.inv_tau, a.allow_lo, a.allow_hi, pz, pj, bz, bjj);
    }
    block_best(bz, bjj, sz, sj);
    if (tid == 0) {
      const bool found = bjj != 0x7fffffff;         // fewer than K allowed tokens: the rest can never be chosen
      a.pool_parent[pbase + r] = found ? node : -1;
      a.pool_token[pbase + r] = found ? bjj : -1;
      a.pool_depth[pbase + r] = a.depth;
      a.pool_logv[pbase + r] = found ? parent_logv + ((static_cast<double>(bz) - static_cast<double>(bm)) - ln_s) : -INFINITY;
    }
    pz = bz;
    pj = bjj;
  }
}

// order-preserving map of a double to an unsigned 64-bit integer (compares then run on the integer pipe)
__device__ __forceinline__ unsigned long long mono64(double x) {
  const unsigned long long b = static_cast<unsigned long long>(__double_as_longlong(x));
  return (b >> 63) ? ~b : (b | 0x8000000000000000ull);
}

// rank of entry i among n entries by (value descending, index ascending); v holds mono64 keys
__device__ __forceinline__ int rank_desc(const unsigned long long* v, int n, int i) {
  const unsigned long long vi = v[i];
  int r = 0;
  for (int j = 0; j < n; ++j) {
    const unsigned long long vj = v[j];
    r += (vj > vi || (vj == vi && j < i)) ? 1 : 0;
  }
  return r;
}

__global__ void __launch_bounds__(kDynThreads) select_frontier_kernel(const ExpandArgs a) {
  extern __shared__ unsigned long long dyn_lv[];
  const int b = blockIdx.x, tid = threadIdx.x, T = a.F * a.K;
  const double* lv = a.pool_logv + static_cast<long long>(b) * a.P + a.pool_off;
  for (int i = tid; i < T; i += kDynThreads) dyn_lv[i] = mono64(lv[i]);
  for (int e = tid; e < a.E; e += kDynThreads) a.next_frontier[b * a.E + e] = -1;
  __syncthreads();
  for (int i = tid; i < T; i += kDynThreads) {
    if (dyn_lv[i] == mono64(-INFINITY)) continue;
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
  extern __shared__ unsigned long long dyn_lv[];     // [used] keys of log V | new id | selected | depth | parent, [used] each
  int* newid = reinterpret_cast<int*>(dyn_lv + a.used);
  int* sel = newid + a.used;
  int* dep_s = sel + a.used;
  int* par_s = dep_s + a.used;
  __shared__ int count, level_n;
  const int b = blockIdx.x, tid = threadIdx.x, n = a.used;
  const long long base = static_cast<long long>(b) * a.P;
  for (int i = tid; i < n; i += kDynThreads) {
    dyn_lv[i] = mono64(i == 0 ? INFINITY : a.pool_logv[base + i]);      // the root ranks first
    newid[i] = -1;
    dep_s[i] = a.pool_depth[base + i];
    par_s[i] = a.pool_parent[base + i];
  }
  __syncthreads();
  for (int i = tid; i < n; i += kDynThreads)
    sel[i] = (i == 0 || (dyn_lv[i] != mono64(-INFINITY) && rank_desc(dyn_lv, n, i) < a.m)) ? 1 : 0;
  if (tid == 0) { count = 1; newid[0] = 0; }
  __syncthreads();
  // the selected entries, compacted (order irrelevant); at most m of them
  int* lst = reinterpret_cast<int*>(dyn_lv);        // the keys are no longer needed
  __shared__ int nsel;
  if (tid == 0) nsel = 0;
  __syncthreads();
  for (int i = 1 + tid; i < n; i += kDynThreads)
    if (sel[i]) lst[atomicAdd(&nsel, 1)] = i;
  __syncthreads();
  const int ns = nsel;
  // breadth-first numbering: a level is ordered by (new id of the parent, pool index)
  for (int dep = 1; dep <= a.max_depth; ++dep) {
    if (tid == 0) level_n = 0;
    __syncthreads();
    const int start = count;
    for (int t = tid; t < ns; t += kDynThreads) {
      const int i = lst[t];
      if (dep_s[i] != dep) continue;
      const int pi = newid[par_s[i]];
      int pos = 0;
      for (int t2 = 0; t2 < ns; ++t2) {
        const int j = lst[t2];
        if (j == i || dep_s[j] != dep) continue;
        const int pj = newid[par_s[j]];
        pos += (pj < pi || (pj == pi && j < i)) ? 1 : 0;
      }
      const int id = start + pos;
      const long long o = static_cast<long long>(b) * a.m + id;
      a.parent[o] = pi;
      a.token[o] = a.pool_token[base + i];
      a.pool_index[o] = i;
      a.logv[o] = a.pool_logv[base + i];
      atomicAdd(&level_n, 1);
      sel[i] = 2 + id;                               // the id is published once the level is complete (below)
    }
    __syncthreads();
    for (int t = tid; t < ns; t += kDynThreads) {
      const int i = lst[t];
      if (sel[i] >= 2) { newid[i] = sel[i] - 2; sel[i] = 1; }
    }
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
  const bool cfg = draft_uncond != nullptr;
  if (dt == LANTERN_F32) {
    if (cfg) expand_rows_kernel<float, true><<<grid, kDynThreads, 0, st>>>(a);
    else expand_rows_kernel<float, false><<<grid, kDynThreads, 0, st>>>(a);
  } else {
    if (cfg) expand_rows_kernel<__nv_bfloat16, true><<<grid, kDynThreads, 0, st>>>(a);
    else expand_rows_kernel<__nv_bfloat16, false><<<grid, kDynThreads, 0, st>>>(a);
  }
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
  trim_tree_kernel<<<batch, kDynThreads, static_cast<size_t>(pool_used) * 24, static_cast<cudaStream_t>(stream)>>>(a);
  return cudaGetLastError() == cudaSuccess ? LANTERN_OK : LANTERN_ERR_CUDA;
}
