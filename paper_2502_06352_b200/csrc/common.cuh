// Shared device helpers: thread-block-cluster primitives, reductions, Philox.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "lantern.h"

namespace lantern {

constexpr int kThreads = 256;           // threads per CTA of the row kernels
constexpr int kWarps = kThreads / 32;
constexpr int kMaxCluster = 16;         // CTAs one logit row may be split over

// Host-side tree handle (the C ABI's opaque lantern_tree).
struct TreeDev {
  int32_t n_nodes;
  int32_t max_depth;
  int32_t max_children;
  int32_t n_internal;
  int32_t per_seq;          // 0: one tree for every sequence.  B > 0: a forest of B trees padded to n_nodes, arrays [B][N]
  int32_t* d_first_child;   // [N] first child id, or -1
  int32_t* d_n_child;       // [N]
  int32_t* d_order;         // [N] node ids, internal nodes first (launch order)
  void* d_block;            // the one allocation behind the arrays above
  int32_t* h_first_child;
  int32_t* h_n_child;
};

// ---------------------------------------------------------------- cluster primitives
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t cluster_nctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
  return r;
}
// Barrier over every thread of the cluster; release/acquire at cluster scope.
__device__ __forceinline__ void cluster_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;"
               ::: "memory");
}
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
// Address of the same shared-memory location in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t dsmem_addr(uint32_t local_saddr, uint32_t rank) {
  uint32_t d;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(d) : "r"(local_saddr), "r"(rank));
  return d;
}
__device__ __forceinline__ float dsmem_ld_f32(uint32_t addr) {
  float v;
  asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ uint32_t dsmem_ld_u32(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared::cluster.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
  return v;
}

// ---------------------------------------------------------------- programmatic dependent launch
// Every kernel of a decode step starts with this: wait until the kernel launched before it on the
// stream has finished and its writes are visible, then let the kernel launched after it be set up
// early (its CTAs start as SMs drain and wait at the same place).  Launched with
// launch_after_previous() below, consecutive kernels lose the launch gap between them; launched
// any other way, both instructions do nothing.
__device__ __forceinline__ void grid_dependency_sync() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// ---------------------------------------------------------------- warp / block reductions
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_incl_scan(float v, int lane) {
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    float t = __shfl_up_sync(0xffffffffu, v, o);
    if (lane >= o) v += t;
  }
  return v;
}

// Monotone map float -> uint32 (larger float, larger key; -0 < +0).
__device__ __forceinline__ uint32_t float_key(float f) {
  uint32_t b = __float_as_uint(f);
  return b ^ ((b >> 31) ? 0xffffffffu : 0x80000000u);
}
__device__ __forceinline__ float key_float(uint32_t k) {
  uint32_t b = (k >> 31) ? (k ^ 0x80000000u) : ~k;
  return __uint_as_float(b);
}

// ---------------------------------------------------------------- Philox-4x32-10
// Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3" (SC 2011).
struct Philox4 { uint32_t x, y, z, w; };
__host__ __device__ __forceinline__ Philox4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2,
                                                          uint32_t c3, uint32_t k0, uint32_t k1) {
  const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u, W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    uint64_t p0 = static_cast<uint64_t>(M0) * c0;
    uint64_t p1 = static_cast<uint64_t>(M1) * c2;
    uint32_t n0 = static_cast<uint32_t>(p1 >> 32) ^ c1 ^ k0;
    uint32_t n2 = static_cast<uint32_t>(p0 >> 32) ^ c3 ^ k1;
    c1 = static_cast<uint32_t>(p1);
    c3 = static_cast<uint32_t>(p0);
    c0 = n0;
    c2 = n2;
    k0 += W0;
    k1 += W1;
  }
  return Philox4{c0, c1, c2, c3};
}
// The same generator with the ten round keys k + r * W precomputed (kernel arguments: they feed
// the xor straight from the constant bank, so a round is two wide multiplies and two xors).
__device__ __forceinline__ Philox4 philox4x32_10_keys(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                                      const uint32_t (&rk0)[10], const uint32_t (&rk1)[10]) {
  const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint64_t p0 = static_cast<uint64_t>(M0) * c0;
    const uint64_t p1 = static_cast<uint64_t>(M1) * c2;
    const uint32_t n0 = static_cast<uint32_t>(p1 >> 32) ^ c1 ^ rk0[r];
    const uint32_t n2 = static_cast<uint32_t>(p0 >> 32) ^ c3 ^ rk1[r];
    c1 = static_cast<uint32_t>(p1);
    c3 = static_cast<uint32_t>(p0);
    c0 = n0;
    c2 = n2;
  }
  return Philox4{c0, c1, c2, c3};
}
enum { kStreamGumbel = 0, kStreamAccept = 1, kStreamResample = 2 };
// counter = (block, row, step_lo, step_hi << 2 | stream), key = seed
__device__ __forceinline__ Philox4 philox_stream(uint64_t seed, uint64_t step, uint32_t row,
                                                 uint32_t stream, uint32_t block) {
  return philox4x32_10(block, row, static_cast<uint32_t>(step),
                       (static_cast<uint32_t>(step >> 32) << 2) | stream,
                       static_cast<uint32_t>(seed), static_cast<uint32_t>(seed >> 32));
}
__device__ __forceinline__ float uniform_halfopen(uint32_t x) {   // [0,1)
  return static_cast<float>(x >> 8) * 5.9604644775390625e-8f;
}
__device__ __forceinline__ float uniform_open(uint32_t x) {       // (0,1), exact in float32
  return (static_cast<float>(x >> 9) + 0.5f) * 1.1920928955078125e-7f;
}

// ---------------------------------------------------------------- asynchronous 16-byte copies
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, uint32_t src_bytes = 16u) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ uint4 lds_u128(const void* p) {       // ordered shared-memory load
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(smem_u32(p)) : "memory");
  return v;
}

// Arguments of the verify kernels (all thread-count variants).
struct VerifyArgs {
  const void *tc, *tu, *dc, *du;
  long long row_stride, seq_stride;
  const int32_t* tokens;
  const float *u_acc, *u_res;
  const int32_t* nbr;
  int k_table, use_bulk;
  const int32_t *first_child, *n_child, *order;
  int B, N, V, kpad, n_internal, max_children;
  float g, inv_tau, lambda, delta;
  int skip, det;           // greedy-skip subset rule; deterministic drafts (p(x) = 1, no drafter rows)
  int topk_t, topk_d, k, code_offset, n_codes, allow_lo, allow_hi;
  unsigned long long seed, step;
  int32_t *node_next, *node_token;
  float *node_mass, *node_thresh;
  int32_t* status;
  const int32_t* only;     // [B*N] or NULL: process only the nodes whose entry is non-zero
  // set together with `only`: the last CTA to finish also walks the trees (no separate launch)
  int lazy;                // non-zero: one cluster per sequence walks the accepted path (no `only`, no `done`)
  int32_t* done;           // one counter, zero before the launch and again after it
  int32_t *accept_len, *out_tokens, *out_nodes;
  int D1;
  int tree_stride;         // 0: the tree arrays are shared by all sequences; N: sequence b's arrays start at b * N (a forest)
};

// ---- walk (Sec. 2.1): follow accepted children from the root of one sequence.  nx / nt are the
// sequence's node_next / node_token rows (staged in shared memory by the callers: the walk is a
// chain of dependent reads), tk its draft tokens, ot / on its output rows.
__device__ __forceinline__ void walk_rows(const int32_t* nx, const int32_t* nt, const int32_t* __restrict__ tk,
                                          int N, int D1, int32_t* __restrict__ accept_len,
                                          int32_t* __restrict__ ot, int32_t* __restrict__ on) {
  int cur = 0, len = 0;
  while (len < D1 - 1) {
    const int nxt = nx[cur];
    if (nxt <= cur || nxt >= N) break;      // -1, or anything that is not a forward edge
    cur = nxt;
    ot[len] = tk[cur];
    on[len] = cur;
    ++len;
  }
  ot[len] = nt[cur];
  on[len] = cur;
  *accept_len = len;
  for (int i = len + 1; i < D1; ++i) { ot[i] = -1; on[i] = -1; }
}

// Walks of sequences [b0, b0 + nb) by the calling CTA: both per-node arrays are first copied to
// `stage` (2 * nb * N ints of shared memory) with coalesced L2 loads (other CTAs of the same launch
// may have written them), then thread i walks sequence b0 + i.
__device__ __forceinline__ void walk_staged(const int32_t* __restrict__ node_next, const int32_t* __restrict__ node_token,
                                            const int32_t* __restrict__ tokens, int b0, int nb, int N, int D1,
                                            int32_t* __restrict__ accept_len, int32_t* __restrict__ out_tokens,
                                            int32_t* __restrict__ out_nodes, int32_t* stage) {
  const long long off = static_cast<long long>(b0) * N;
  const int cnt = nb * N;
  for (int i = threadIdx.x; i < cnt; i += blockDim.x) {
    stage[i] = __ldcg(node_next + off + i);
    stage[cnt + i] = __ldcg(node_token + off + i);
  }
  __syncthreads();
  for (int i = threadIdx.x; i < nb; i += blockDim.x) {
    const int b = b0 + i;
    walk_rows(stage + i * N, stage + cnt + i * N, tokens + static_cast<long long>(b) * N, N, D1, accept_len + b,
              out_tokens + static_cast<long long>(b) * D1, out_nodes + static_cast<long long>(b) * D1);
  }
  __syncthreads();
}

// Host side: launch `kern` with programmatic stream serialisation (and, when cluster > 1, that
// cluster size).  The kernel must call grid_dependency_sync() before it touches global memory.
template <typename... KArgs, typename... Args>
static inline cudaError_t launch_after_previous(void (*kern)(KArgs...), unsigned grid, unsigned block, size_t smem,
                                                cudaStream_t st, int cluster, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid, 1, 1);
  cfg.blockDim = dim3(block, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  int na = 0;
  attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[na].val.programmaticStreamSerializationAllowed = 1;
  ++na;
  if (cluster > 1) {
    attr[na].id = cudaLaunchAttributeClusterDimension;
    attr[na].val.clusterDim.x = static_cast<unsigned>(cluster);
    attr[na].val.clusterDim.y = 1;
    attr[na].val.clusterDim.z = 1;
    ++na;
  }
  cfg.attrs = attr;
  cfg.numAttrs = na;
  return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

}  // namespace lantern
