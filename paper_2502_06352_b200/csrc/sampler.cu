// Stochastic static-tree drafting (Sec. 2.1): s children of a node are drawn from the drafter
// distribution p without replacement.  Gumbel-top-s: key_j = log p_j - log(-log U_j); since
// log p_j = z_j - const over the row, ranking z_j + G_j gives the same children.
//
// Same row machinery as the verify kernel: one CTA (a cluster for rows wider than 16384) per
// expanded parent, the drafter row read once into shared memory, exact top-k threshold, then
// one sweep that forms the keys (Philox-4x32-10, four uniforms per counter) and the softmax
// denominator.  Every thread keeps the best key of its own entries in registers; a round picks
// the row-wide best (ties: lower token id) and only the winner's owner rescans its entries.
#include "common.cuh"
#define LANTERN_VT 1024
#define LANTERN_VNS v1024
#include "verify_kernel.cuh"

namespace lantern {
using namespace v1024;

struct SampleArgs {
  const void *dc, *du;
  long long row_stride, seq_stride;
  const float* gumbel;
  const int32_t *first_child, *n_child, *order;
  int order_begin;
  int B, N, V;
  float g, inv_tau;
  int topk_d, allow_lo, allow_hi;
  unsigned long long seed, step;
  int32_t* tokens;
  float* draft_prob;
  int32_t* status;
  int n_parents;       // parents per sequence in this launch
  int repair;          // non-zero: draw only the parents whose first child's token is the redo marker
  uint32_t rk0[10], rk1[10];   // Philox round keys of `seed`
};

}  // namespace lantern
#include "sampler_sparse.cuh"
#include "sampler_stream.cuh"
namespace lantern {

constexpr float kDenseKeyErr = 2e-5f;     // bound on |float32 key - exact key| (|key| < 64)

__device__ __forceinline__ bool better(float ka, int ia, float kb, int ib) {   // a beats b
  return ka > kb || (ka == kb && ia < ib);
}

__device__ __forceinline__ void warp_argbest(float& k, int& i) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ok = __shfl_xor_sync(0xffffffffu, k, o);
    const int oi = __shfl_xor_sync(0xffffffffu, i, o);
    if (better(ok, oi, k, i)) { k = ok; i = oi; }
  }
}

// best key among this thread's entries of the key slice
template <int E>
__device__ __forceinline__ void thread_best(const float* __restrict__ K, int lo, float& bk, int& bi) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  bk = -INFINITY;
  bi = 0x7fffffff;
#pragma unroll
  for (int v = 0; v < E / 4; ++v) {
    const int j = warp * 32 * E + v * 128 + lane * 4;
    const float4 k4 = *reinterpret_cast<const float4*>(K + j);
    const float kv[4] = {k4.x, k4.y, k4.z, k4.w};
#pragma unroll
    for (int e = 0; e < 4; ++e)
      if (kv[e] > bk) { bk = kv[e]; bi = lo + j + e; }     // ascending ids: strict > keeps the lower id
  }
}

// One parent: drafter row into shared memory, keys, s selection rounds.
template <typename T, bool CFG, int E>
__device__ __forceinline__ void sample_node(const SampleArgs& a, const int idx, VCtx& c, const TopkSmem& tk,
                                            float* __restrict__ Z, float* __restrict__ K) {
  constexpr int SL = VT * E;
  constexpr int NV4 = E / 4;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int b = idx % a.B;
  const int n = a.order[a.order_begin + idx / a.B];
  const int fc = a.first_child[n], nc = a.n_child[n];
  const int lo = c.rank * SL;
  const int len = max(0, min(a.V - lo, SL));
  const long long row_off = static_cast<long long>(b) * a.seq_stride + static_cast<long long>(n) * a.row_stride;
  const long long out_b = static_cast<long long>(b) * a.N;
  const bool single = c.nrank == 1;

  const bool masked = a.allow_lo > 0 || a.allow_hi < a.V;
  float mx[2];
  const T* dcp = static_cast<const T*>(a.dc) + row_off;
  const T* dup = CFG ? static_cast<const T*>(a.du) + row_off : nullptr;
  issue_row<T, E>(dcp, lo, len, Z);
  if (CFG) issue_row<T, E>(dup, lo, len, K);
  cp_async_commit();
  cp_async_wait<0>();
  mx[0] = finish_row<T, CFG, E>(dcp, dup, a.g, a.inv_tau, lo, len, a.allow_lo, a.allow_hi, masked, Z, K);
  mx[1] = -INFINITY;
  row_reduce<2, true>(c, mx);
  if (mx[0] == -INFINITY) {
    if (tid == 0 && c.rank == 0) vflag(a.status, LANTERN_DEV_EMPTY_ROW);
    mx[0] = 0.f;
  }
  mx[1] = 0.f;
  float theta[2] = {-INFINITY, -INFINITY};
  const int kth[2] = {(a.topk_d > 0 && a.topk_d < a.V) ? a.topk_d : 0, 0};
  const bool has_topk = kth[0] > 0;
  if (has_topk) topk_thresholds<E>(c, tk, Z, Z, mx, kth, theta);

  // (the top-k routine's candidate scratch is dead from here on: it holds the rounds' winners and
  // the near-tied tokens of the exact re-ranking)
  float* fx_key = tk.all;                                   // [8]
  int* fx_tok = reinterpret_cast<int*>(tk.all + 8);         // [8]
  int* fx_cand = fx_tok + 8;                                // [32]
  int* fx_cnt = fx_cand + 32;
  // ---- keys z + G, G = -log(-log U), and the softmax denominator, in one sweep
  const uint32_t row_id = static_cast<uint32_t>(out_b + n);
  const float* gum = a.gumbel ? a.gumbel + (static_cast<long long>(row_id) * a.V + lo) : nullptr;
  const float c0 = -mx[0] * kLog2e;
  float sm[2] = {0.f, 0.f};
  float bk = -INFINITY;
  int bi = 0x7fffffff;
#pragma unroll 2
  for (int v = 0; v < NV4; ++v) {
    const int j = warp * 32 * E + v * 128 + lane * 4;
    const float4 z4 = *reinterpret_cast<const float4*>(Z + j);
    const float zv[4] = {z4.x, z4.y, z4.z, z4.w};
    float u4[4];
    if (gum) {
#pragma unroll
      for (int e = 0; e < 4; ++e) u4[e] = (j + e < len) ? __ldcs(gum + j + e) : 0.5f;
    } else {
      const Philox4 r = philox_stream(a.seed, a.step, row_id, kStreamGumbel, static_cast<uint32_t>((lo + j) >> 2));
      u4[0] = uniform_open(r.x); u4[1] = uniform_open(r.y); u4[2] = uniform_open(r.z); u4[3] = uniform_open(r.w);
    }
    float kv[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const bool keep = zv[e] >= theta[0] && zv[e] != -INFINITY;
      kv[e] = keep ? zv[e] - __logf(-logf(u4[e])) : -INFINITY;
      if (keep) sm[0] += ex2_approx(fmaf(zv[e], kLog2e, c0));
      if (kv[e] > bk) { bk = kv[e]; bi = lo + j + e; }
    }
    *reinterpret_cast<float4*>(K + j) = make_float4(kv[0], kv[1], kv[2], kv[3]);
  }
  row_reduce<2, false>(c, sm);
  const float inv_sum = sm[0] > 0.f ? 1.f / sm[0] : 0.f;

  // ---- s rounds: row-wide best key; the owner of the winner retires it and rescans
  float* pk = c.red + 2 * VW * 4 - 2 * VW;     // [VW] keys and [VW] ids of the warps' best (tail of red[1])
  for (int round = 0; round < nc; ++round) {
    float wk = bk;
    int wi = bi;
    warp_argbest(wk, wi);
    __syncthreads();                            // pk of the previous round has been consumed
    if (lane == 0) { pk[warp] = wk; pk[VW + warp] = __int_as_float(wi); }
    __syncthreads();
    float ck = lane < VW ? pk[lane] : -INFINITY;
    int ci = lane < VW ? __float_as_int(pk[VW + lane]) : 0x7fffffff;
    warp_argbest(ck, ci);
    if (!single) {
      if (tid == 0) { c.xch[c.parity * 4] = ck; c.xch[c.parity * 4 + 1] = __int_as_float(ci); }
      cluster_sync();
      float rk = -INFINITY;
      int ri = 0x7fffffff;
      if (lane < static_cast<int>(c.nrank)) {
        rk = dsmem_ld_f32(dsmem_addr(smem_u32(&c.xch[c.parity * 4]), lane));
        ri = __float_as_int(dsmem_ld_f32(dsmem_addr(smem_u32(&c.xch[c.parity * 4 + 1]), lane)));
      }
      warp_argbest(rk, ri);
      ck = rk;
      ci = ri;
      c.parity ^= 1;
    }
    const bool valid = ck != -INFINITY;
    if (tid == 0) { fx_key[round] = ck; fx_tok[round] = valid ? ci : -1; }
    if (valid && ci == bi) {                    // exactly one thread of the row owns the winner
      const int jl = ci - lo;
      K[jl] = -INFINITY;
      a.tokens[out_b + fc + round] = ci;
      if (a.draft_prob) a.draft_prob[out_b + fc + round] = ex2_approx(fmaf(Z[jl], kLog2e, c0)) * inv_sum;
      thread_best<E>(K, lo, bk, bi);           // this thread's own writes are visible to it
    }
    if (!valid && c.rank == 0 && tid == 0) {
      a.tokens[out_b + fc + round] = -1;
      if (a.draft_prob) a.draft_prob[out_b + fc + round] = 0.f;
    }
  }

  // ---- exact order.  The rounds ranked float32 keys (error below kDenseKeyErr each).  Where two
  // of the chosen keys, or a chosen key and one left out, are closer than twice that, the
  // entries involved are ranked again by keys evaluated in double precision (ties: lower token
  // id) by CTA 0 of the row, which reads the other CTAs' near-tied tokens through DSMEM.
  __syncthreads();
  int nv = 0;
  while (nv < nc && fx_tok[nv] >= 0) ++nv;
  const float k_last = nv > 0 ? fx_key[nv - 1] : 0.f;
  bool need = false;
  for (int r = 1; r < nv; ++r) need |= fx_key[r - 1] - fx_key[r] <= 2.f * kDenseKeyErr;
  if (tid == 0) *fx_cnt = 0;
  __syncthreads();
  if (nv > 0) {
#pragma unroll
    for (int v = 0; v < NV4; ++v) {
      const int j = warp * 32 * E + v * 128 + lane * 4;
      const float4 k4 = *reinterpret_cast<const float4*>(K + j);
      const float kv[4] = {k4.x, k4.y, k4.z, k4.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        if (kv[e] != -INFINITY && kv[e] >= k_last - 2.f * kDenseKeyErr) {
          const int at = atomicAdd(fx_cnt, 1);
          if (at < 32) fx_cand[at] = lo + j + e;
        }
      }
    }
  }
  csync(c);                                     // every CTA's list of near-tied tokens is complete
  if (c.rank == 0 && warp == 0 && nv > 0) {
    int ncand = nv, extra = 0;
    int t = lane < nv ? fx_tok[lane] : 0x7fffffff;
    for (uint32_t q = 0; q < c.nrank; ++q) {
      const int nq = single ? *fx_cnt : static_cast<int>(dsmem_ld_u32(dsmem_addr(smem_u32(fx_cnt), q)));
      extra += nq;
      for (int i = 0; i < nq && i < 32; ++i) {
        const int tq = single ? fx_cand[i] : static_cast<int>(dsmem_ld_u32(dsmem_addr(smem_u32(&fx_cand[i]), q)));
        if (ncand < 32 && lane == ncand) t = tq;
        ++ncand;
      }
    }
    if (extra > 0 || need) {
      if (ncand > 32) {
        if (lane == 0) vflag(a.status, LANTERN_DEV_KEY_TIES);     // more near-ties than one warp ranks
      } else {
        double key = -INFINITY;
        float z = 0.f;
        if (lane < ncand) {
          z = combine<CFG>(Vec<T>::widen(dcp[t]), CFG ? Vec<T>::widen(dup[t]) : 0.f, a.g, a.inv_tau);
          float u;
          if (a.gumbel) {
            u = __ldcs(a.gumbel + static_cast<long long>(row_id) * a.V + t);
          } else {
            const Philox4 r = philox_stream(a.seed, a.step, row_id, kStreamGumbel, static_cast<uint32_t>(t >> 2));
            const uint32_t w = (t & 3) == 0 ? r.x : ((t & 3) == 1 ? r.y : ((t & 3) == 2 ? r.z : r.w));
            u = uniform_open(w);
          }
          key = static_cast<double>(z) - log(-log(static_cast<double>(u)));
        }
        int rank = 0;
        for (int o = 0; o < ncand; ++o) {
          const double ko = __shfl_sync(0xffffffffu, key, o);
          const int to = __shfl_sync(0xffffffffu, t, o);
          rank += (ko > key || (ko == key && to < t)) ? 1 : 0;
        }
        if (lane < ncand && rank < nv) {
          a.tokens[out_b + fc + rank] = t;
          if (a.draft_prob) a.draft_prob[out_b + fc + rank] = ex2_approx(fmaf(z, kLog2e, c0)) * inv_sum;
        }
      }
    }
  }
}

template <typename T, bool CFG, int E>
__global__ void __launch_bounds__(VT, 1) sample_children_kernel(const SampleArgs a) {
  grid_dependency_sync();
  constexpr int SL = VT * E;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  float* Z = reinterpret_cast<float*>(smem_raw);
  float* K = Z + SL;                                    // keys; first the uncond staging buffer
  unsigned char* nxt = reinterpret_cast<unsigned char*>(K + SL);
  TopkSmem tk;
  tk.gbins = reinterpret_cast<uint32_t*>(nxt);
  tk.comp = reinterpret_cast<float*>(tk.gbins + 2 * kBins);
  tk.all = tk.comp + 2 * kCandLocal;
  nxt += kScratchBytes;
  tk.bins = reinterpret_cast<uint32_t*>(nxt);
  tk.wl = reinterpret_cast<float*>(tk.bins + 2 * kBins);
  tk.wcnt = reinterpret_cast<int*>(tk.wl + 2 * kCandLocal);
  tk.wtot = reinterpret_cast<uint32_t*>(tk.wcnt + 2 * VW);
  VCtx c;
  c.red = reinterpret_cast<float*>(tk.wtot + 2 * (kBins / 32));
  c.xch = c.red + 2 * VW * 4;
  c.gath = c.xch + 8;
  tk.sel = reinterpret_cast<int*>(c.gath + kMaxCluster * 4);
  tk.cnts = tk.sel + 8;
  c.rank = cluster_ctarank();
  c.nrank = cluster_nctarank();
  c.parity = 0;
  c.last_red = c.red;

  // A regular launch has one CTA (cluster) per parent.  A repair launch has fewer: cluster g of
  // G takes the marked parents idx = g (mod G) one after another, and leaves at once when none of
  // them is marked.
  const int tid = threadIdx.x;
  const int np = static_cast<int>(a.n_parents), rows = a.B * np;
  const int G = gridDim.x / c.nrank, g0 = blockIdx.x / c.nrank;
  auto marked = [&](int idx) {
    const int n = a.order[a.order_begin + idx / a.B];
    return a.tokens[static_cast<long long>(idx % a.B) * a.N + a.first_child[n]] == sparse::kRedoToken;
  };
  if (a.repair) {
    bool any = false;
    for (long long i = g0 + static_cast<long long>(tid) * G; i < rows; i += static_cast<long long>(VT) * G)
      any |= marked(static_cast<int>(i));
    if (!__syncthreads_or(any)) return;      // the same marks, hence the same decision, in every CTA of a cluster
  }
  for (int idx = g0; idx < rows; idx += G) {
    if (a.repair && !marked(idx)) continue;
    csync(c);     // every CTA of the row has read the mark before the row's first token is rewritten
    sample_node<T, CFG, E>(a, idx, c, tk, Z, K);
    csync(c);     // peers may still be reading this CTA's shared memory; the next parent overwrites it
  }
}

}  // namespace lantern

namespace lantern {

// Choose E (row entries per thread; a CTA's slice is VT*E entries) and the cluster size.
static bool sampler_shape(int V, int rows, int min_e, int override_cs, int* cs_out, int* e_out, size_t* smem_out) {
  constexpr int kMaxE = 16384 / VT;
  auto cs_for = [&](int e) { int cs = (V + VT * e - 1) / (VT * e); return cs > 8 ? (cs > 16 ? 0 : 16) : cs; };
  int e = 0;
  if (override_cs > 0) {
    for (int cand = min_e; cand <= kMaxE; cand *= 2)
      if (static_cast<long long>(VT) * cand * override_cs >= V) { e = cand; break; }
    if (e == 0) return false;
    *cs_out = override_cs;
  } else {
    for (int cand = min_e; cand <= kMaxE; cand *= 2)
      if (VT * cand >= V) { e = cand; break; }
    if (e == 0) e = kMaxE;
    if (cs_for(e) == 0) return false;
    while (e > min_e && static_cast<long long>(rows) * cs_for(e) < 74 && cs_for(e / 2) != 0 && cs_for(e / 2) <= 8) e /= 2;
    *cs_out = cs_for(e);
  }
  *e_out = e;
  *smem_out = static_cast<size_t>(2) * VT * e * 4 + kScratchBytes + kSmallSmem;
  return *smem_out <= 227 * 1024;
}

template <typename T, bool CFG, int E>
static cudaError_t launch_sampler_e(const SampleArgs& a, int n_parents, int cs, size_t smem, cudaStream_t st) {
  auto kern = sample_children_kernel<T, CFG, E>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (e != cudaSuccess) return e;
  if (cs > 8) {
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
    if (e != cudaSuccess) return e;
  }
  unsigned clusters = static_cast<unsigned>(a.B) * n_parents;
  if (a.repair) {        // about one cluster per SM; each walks its share of the marked parents
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
      sms = 148;
    const unsigned per_wave = static_cast<unsigned>(sms / cs > 0 ? sms / cs : 1);
    if (clusters > per_wave) clusters = per_wave;
  }
  return launch_after_previous(kern, clusters * cs, VT, smem, st, cs, a);
}

template <typename T, bool CFG>
static cudaError_t launch_sampler(const SampleArgs& a, int n_parents, int cs, int e, size_t smem, cudaStream_t st) {
  if constexpr (16384 / VT >= 32) {
    if (e == 32) return launch_sampler_e<T, CFG, 32>(a, n_parents, cs, smem, st);
  }
  if (e == 16) return launch_sampler_e<T, CFG, 16>(a, n_parents, cs, smem, st);
  if (e == 8) return launch_sampler_e<T, CFG, 8>(a, n_parents, cs, smem, st);
  if constexpr (Vec<T>::N <= 4) {
    if (e == 4) return launch_sampler_e<T, CFG, 4>(a, n_parents, cs, smem, st);
  }
  return cudaErrorInvalidValue;
}

// ---- launch of the list-based kernel: one CTA per parent
template <typename T, bool CFG, int E>
static cudaError_t launch_sample_sparse_e(const SampleArgs& a, cudaStream_t st) {
  auto kern = sparse::sample_sparse_kernel<T, CFG, E>;
  const size_t smem = sparse::sampler_smem_bytes(E);
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (e != cudaSuccess) return e;
  return launch_after_previous(kern, static_cast<unsigned>(a.B) * a.n_parents, sparse::ST, smem, st, 1, a);
}
template <typename T, bool CFG>
static cudaError_t launch_sample_sparse(const SampleArgs& a, int V, cudaStream_t st) {
  if (V <= sparse::ST * 8) return launch_sample_sparse_e<T, CFG, 8>(a, st);
  if (V <= sparse::ST * 16) return launch_sample_sparse_e<T, CFG, 16>(a, st);
  return launch_sample_sparse_e<T, CFG, 32>(a, st);
}


// ---- launch of the streaming kernel (rows without top-k): one CTA, or a cluster, per parent
template <typename T, bool CFG, bool TAU1>
static cudaError_t launch_sample_stream_t(const SampleArgs& a, int cs, cudaStream_t st) {
  auto kern = stream::sample_stream_kernel<T, CFG, TAU1>;
  const size_t smem = stream::sampler_stream_smem();
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (e != cudaSuccess) return e;
  if (cs > 8) {
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
    if (e != cudaSuccess) return e;
  }
  return launch_after_previous(kern, static_cast<unsigned>(a.B) * a.n_parents * cs, stream::ST, smem, st, cs, a);
}
static cudaError_t launch_sample_stream(const SampleArgs& a, int cs, bool f32, bool cfg, cudaStream_t st) {
  const bool tau1 = a.inv_tau == 1.0f;
  if (f32) {
    if (cfg) return launch_sample_stream_t<float, true, false>(a, cs, st);
    return tau1 ? launch_sample_stream_t<float, false, true>(a, cs, st) : launch_sample_stream_t<float, false, false>(a, cs, st);
  }
  if (cfg) return launch_sample_stream_t<__nv_bfloat16, true, false>(a, cs, st);
  return tau1 ? launch_sample_stream_t<__nv_bfloat16, false, true>(a, cs, st)
              : launch_sample_stream_t<__nv_bfloat16, false, false>(a, cs, st);
}

}  // namespace lantern

using namespace lantern;

extern "C" int32_t lantern_get_cluster_size(void);

namespace {
// Rows truncated to a moderate top-k can take the list-based kernel.
bool sampler_uses_lists(const lantern_params* p) {
  const int V = p->vocab;
  const int ov = lantern_get_cluster_size();
  return ov == 0 && V <= sparse::kMaxV && p->top_k_draft > 0 && p->top_k_draft < V && p->top_k_draft <= sparse::kMaxTopK;
}
}  // namespace

// Rows that no top-k truncates can take the streaming kernel; it does when the call expands at
// least kStreamMinParents parents or kStreamMinLogits / V of them (fewer fit the dense kernel's one
// wave of CTAs, or of CTA clusters for wide rows, whose shared-memory row shortens the chain of
// dependent steps: the measured cross-over lies between 2.6 M and 5.2 M parents x V for V = 16384
// and 65536, whatever the allowed range), when the dense kernel cannot hold the row, or when asked to.
constexpr int kStreamMinParents = 256;
constexpr long long kStreamMinLogits = 4ll << 20;
static bool sampler_uses_stream(const lantern_params* p, long long parents, bool fits_dense) {
  if ((p->top_k_draft > 0 && p->top_k_draft < p->vocab) || p->vocab > stream::kMaxV) return false;
  if (p->kernels == 2) return !fits_dense;
  if (p->kernels == 1) return true;
  return parents >= kStreamMinParents || parents * p->vocab >= kStreamMinLogits || !fits_dense;
}

extern "C" int32_t lantern_sample_draft_tree_path(const lantern_params* p, const lantern_tree* tree, int32_t batch) {
  if (!p || !tree || batch <= 0) return -1;
  const TreeDev* t = reinterpret_cast<const TreeDev*>(tree);
  if (sampler_uses_stream(p, static_cast<long long>(batch) * t->n_internal, true)) return LANTERN_PATH_STREAM;
  return sampler_uses_lists(p) ? LANTERN_PATH_LISTS : LANTERN_PATH_DENSE;
}

extern "C" lantern_status lantern_sample_draft_tree(
    const lantern_params* p, const lantern_tree* tree, const void* draft_cond, const void* draft_uncond,
    lantern_dtype dt, int64_t row_stride, int64_t seq_stride, int32_t batch, int32_t parent_begin,
    int32_t parent_end, const float* gumbel_uniforms, int32_t* tokens, float* draft_prob,
    int32_t* device_status, void* stream) {
  if (!p || !tree || !draft_cond || !tokens) return LANTERN_ERR_INVALID_ARG;
  const TreeDev* t = reinterpret_cast<const TreeDev*>(tree);
  if (batch <= 0 || p->vocab <= 0 || !(p->temperature > 0.f) || p->top_k_draft < 0) return LANTERN_ERR_INVALID_ARG;
  if (dt != LANTERN_F32 && dt != LANTERN_BF16) return LANTERN_ERR_INVALID_ARG;
  if (parent_begin < 0 || parent_end > t->n_nodes || parent_begin > parent_end) return LANTERN_ERR_INVALID_ARG;
  if (t->per_seq) return LANTERN_ERR_UNSUPPORTED;      // a forest holds deterministically drafted trees: nothing to sample
  const int V = p->vocab;
  const int allow_lo = p->allowed_begin, allow_hi = p->allowed_end == 0 ? V : p->allowed_end;
  if (allow_lo < 0 || allow_hi > V || allow_lo >= allow_hi) return LANTERN_ERR_INVALID_ARG;
  if (p->step >> 62) return LANTERN_ERR_INVALID_ARG;
  const size_t esz = dt == LANTERN_F32 ? 4 : 2;
  if (row_stride < V || seq_stride < 0 || (row_stride * esz) % 16 || (seq_stride * esz) % 16) return LANTERN_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(draft_cond) % 16) || (draft_uncond && reinterpret_cast<uintptr_t>(draft_uncond) % 16))
    return LANTERN_ERR_INVALID_ARG;
  if (static_cast<int64_t>(batch) * t->n_nodes > (1 << 24)) return LANTERN_ERR_UNSUPPORTED;
  // internal nodes with id in [parent_begin, parent_end): a contiguous run of the launch order
  int i0 = 0, i1 = 0;
  for (int n = 0; n < t->n_nodes; ++n) {
    if (t->h_n_child[n] == 0) continue;
    if (n < parent_begin) ++i0;
    if (n < parent_end) ++i1;
  }
  if (i1 == i0) return LANTERN_OK;
  SampleArgs a;
  a.dc = draft_cond; a.du = draft_uncond;
  a.row_stride = row_stride; a.seq_stride = seq_stride;
  a.gumbel = gumbel_uniforms;
  a.first_child = t->d_first_child; a.n_child = t->d_n_child; a.order = t->d_order;
  a.order_begin = i0;
  a.B = batch; a.N = t->n_nodes; a.V = V;
  a.g = p->cfg_scale; a.inv_tau = 1.0f / p->temperature;
  a.topk_d = p->top_k_draft; a.allow_lo = allow_lo; a.allow_hi = allow_hi;
  a.seed = p->seed; a.step = p->step;
  a.tokens = tokens; a.draft_prob = draft_prob; a.status = device_status;
  a.n_parents = i1 - i0;
  a.repair = 0;
  for (int r = 0; r < 10; ++r) {
    a.rk0[r] = static_cast<uint32_t>(p->seed) + static_cast<uint32_t>(r) * 0x9E3779B9u;
    a.rk1[r] = static_cast<uint32_t>(p->seed >> 32) + static_cast<uint32_t>(r) * 0xBB67AE85u;
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const bool cfg = draft_uncond != nullptr;
  const int ov = lantern_get_cluster_size();
  int cs_d, e_d;
  size_t smem_d;
  const bool fits_dense = sampler_shape(V, batch * (i1 - i0), dt == LANTERN_F32 ? 4 : 8, ov, &cs_d, &e_d, &smem_d);
  if (p->kernels < 0 || p->kernels > 2) return LANTERN_ERR_INVALID_ARG;
  if (sampler_uses_stream(p, static_cast<long long>(batch) * (i1 - i0), fits_dense)) {
    // CTAs per parent: the smallest power of two that gives every SM a CTA (measured on rows of 65536 logits:
    // 80 and 100 parents run fastest split in two, 200 unsplit; wider clusters pay for their merge)
    int cs = ov;
    if (cs <= 0) {
      int dev = 0, sms = 0;
      if (cudaGetDevice(&dev) != cudaSuccess ||
          cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
        sms = 148;
      const int nvec = (allow_hi - allow_lo) / (dt == LANTERN_F32 ? 4 : 8);
      cs = 1;
      while (cs < 16 && static_cast<long long>(batch) * (i1 - i0) * cs < sms && nvec / (2 * cs * stream::SW) >= 32) cs *= 2;
    }
    return launch_sample_stream(a, cs, dt == LANTERN_F32, cfg, st) == cudaSuccess ? LANTERN_OK : LANTERN_ERR_CUDA;
  }
  int cs, e;
  size_t smem;
  if (!sampler_shape(V, batch * (i1 - i0), dt == LANTERN_F32 ? 4 : 8, ov, &cs, &e, &smem)) return LANTERN_ERR_UNSUPPORTED;
  cudaError_t err;
  // Rows truncated to a moderate top-k take the list-based kernel; the dense kernel then draws
  // the parents it marked as not fitting (usually none).
  if (sampler_uses_lists(p)) {
    if (dt == LANTERN_F32)
      err = cfg ? launch_sample_sparse<float, true>(a, V, st) : launch_sample_sparse<float, false>(a, V, st);
    else
      err = cfg ? launch_sample_sparse<__nv_bfloat16, true>(a, V, st) : launch_sample_sparse<__nv_bfloat16, false>(a, V, st);
    if (err != cudaSuccess) return LANTERN_ERR_CUDA;
    a.repair = 1;
  }
  if (dt == LANTERN_F32)
    err = cfg ? launch_sampler<float, true>(a, i1 - i0, cs, e, smem, st) : launch_sampler<float, false>(a, i1 - i0, cs, e, smem, st);
  else
    err = cfg ? launch_sampler<__nv_bfloat16, true>(a, i1 - i0, cs, e, smem, st)
              : launch_sampler<__nv_bfloat16, false>(a, i1 - i0, cs, e, smem, st);
  return err == cudaSuccess ? LANTERN_OK : LANTERN_ERR_CUDA;
}
