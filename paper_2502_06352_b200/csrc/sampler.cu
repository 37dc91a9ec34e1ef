// Stochastic static-tree drafting (Sec. 2.1): s children of a node are drawn from the drafter
// distribution p without replacement.  Gumbel-top-s: key_j = log p_j - log(-log U_j); since
// log p_j = z_j - const over the row, ranking z_j + G_j gives the same children.
//
// One thread-block cluster per expanded parent; the drafter row is read once, its
// post-processed logits stay in shared memory (slice per CTA), the s winners are found by s
// rounds of a cluster-wide arg-max.
#include "rowops.cuh"

namespace lantern {

struct SampleArgs {
  const void *dc, *du;
  long long row_stride, seq_stride;
  const float* gumbel;
  const int32_t *first_child, *n_child, *order;
  int order_begin;
  int B, N, V, SL;
  float g, inv_tau;
  int topk_d, allow_lo, allow_hi;
  unsigned long long seed, step;
  int32_t* tokens;
  float* draft_prob;
  int32_t* status;
};

constexpr int kSamplerFixedSmem = 2 * 2 * 256 * 4 + kWarps * 4 * 4 + 8 * 4 + kMaxCluster * 4 * 4 + 4 * 4 + 16;

__device__ __forceinline__ bool better(float ka, int ia, float kb, int ib) {   // a beats b
  return ka > kb || (ka == kb && ia < ib);
}

template <typename T, bool CFG>
__global__ void __launch_bounds__(kThreads) sample_children_kernel(const SampleArgs a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  float* Z = reinterpret_cast<float*>(smem_raw);
  float* K = Z + a.SL;
  ClusterCtx c;
  c.hist = reinterpret_cast<uint32_t*>(K + a.SL);
  c.red = reinterpret_cast<float*>(c.hist + 2 * 2 * 256);
  c.xch = c.red + kWarps * 4;
  c.gath = c.xch + 8;
  c.sel = reinterpret_cast<int*>(c.gath + kMaxCluster * 4);
  c.rank = cluster_ctarank();
  c.nrank = cluster_nctarank();
  c.parity = 0;
  c.hist_parity = 0;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int idx = blockIdx.x / c.nrank;
  const int b = idx % a.B;
  const int n = a.order[a.order_begin + idx / a.B];
  const int fc = a.first_child[n], nc = a.n_child[n];
  const int SL = a.SL;
  const int lo = c.rank * SL;
  const int len = max(0, min(a.V - lo, SL));
  const long long row_off = static_cast<long long>(b) * a.seq_stride + static_cast<long long>(n) * a.row_stride;
  const long long out_b = static_cast<long long>(b) * a.N;

  float mx[1];
  mx[0] = load_slice<T, CFG>(static_cast<const T*>(a.dc) + row_off,
                             CFG ? static_cast<const T*>(a.du) + row_off : nullptr, a.g, a.inv_tau, lo,
                             len, a.allow_lo, a.allow_hi, Z);
  cluster_reduce<1, true>(c, mx);
  if (mx[0] == -INFINITY) {
    if (tid == 0 && c.rank == 0 && a.status) atomicOr(a.status, LANTERN_DEV_EMPTY_ROW);
    mx[0] = 0.f;
  }
  float theta[1] = {-INFINITY};
  if (a.topk_d > 0 && a.topk_d < a.V) {
    float* const rows[1] = {Z};
    const int kth[1] = {a.topk_d};
    cluster_topk_threshold<1>(c, rows, len, kth, theta);
  }

  // keys and the softmax denominator in one sweep
  const uint32_t row_id = static_cast<uint32_t>(out_b + n);
  const float* gum = a.gumbel ? a.gumbel + (static_cast<long long>(row_id) * a.V + lo) : nullptr;
  float sm[1] = {0.f};
  for (int i = tid; i * 4 < len; i += kThreads) {
    const int j = i * 4;
    float u4[4];
    if (gum) {
#pragma unroll
      for (int e = 0; e < 4; ++e) u4[e] = (j + e < len) ? __ldcs(gum + j + e) : 0.5f;
    } else {
      Philox4 r = philox_stream(a.seed, a.step, row_id, kStreamGumbel, static_cast<uint32_t>((lo + j) >> 2));
      u4[0] = uniform_open(r.x); u4[1] = uniform_open(r.y); u4[2] = uniform_open(r.z); u4[3] = uniform_open(r.w);
    }
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      if (j + e < len) {
        const float z = Z[j + e];
        const bool keep = z >= theta[0] && z != -INFINITY;
        K[j + e] = keep ? z - logf(-logf(u4[e])) : -INFINITY;
        if (keep) sm[0] += expf(z - mx[0]);
      }
    }
  }
  cluster_reduce<1, false>(c, sm);
  const float inv_sum = sm[0] > 0.f ? 1.f / sm[0] : 0.f;

  for (int round = 0; round < nc; ++round) {
    float bk = -INFINITY;
    int bi = 0x7fffffff;
    for (int j = tid; j < len; j += kThreads) {
      const float kj = K[j];
      if (better(kj, lo + j, bk, bi)) { bk = kj; bi = lo + j; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float ok = __shfl_xor_sync(0xffffffffu, bk, o);
      const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
      if (better(ok, oi, bk, bi)) { bk = ok; bi = oi; }
    }
    if (lane == 0) { c.red[warp * 2] = bk; c.red[warp * 2 + 1] = __int_as_float(bi); }
    __syncthreads();
    if (tid == 0) {
      for (int w = 1; w < kWarps; ++w) {
        const float ok = c.red[w * 2];
        const int oi = __float_as_int(c.red[w * 2 + 1]);
        if (better(ok, oi, bk, bi)) { bk = ok; bi = oi; }
      }
      c.xch[c.parity * 4] = bk;
      c.xch[c.parity * 4 + 1] = __int_as_float(bi);
    }
    cluster_sync();
    if (tid < static_cast<int>(c.nrank) * 2)
      c.gath[tid] = dsmem_ld_f32(dsmem_addr(smem_u32(&c.xch[c.parity * 4 + (tid & 1)]), tid >> 1));
    __syncthreads();
    c.parity ^= 1;
    bk = c.gath[0];
    bi = __float_as_int(c.gath[1]);
    for (uint32_t r = 1; r < c.nrank; ++r) {
      const float ok = c.gath[r * 2];
      const int oi = __float_as_int(c.gath[r * 2 + 1]);
      if (better(ok, oi, bk, bi)) { bk = ok; bi = oi; }
    }
    const bool valid = bk != -INFINITY;
    if (valid && bi >= lo && bi < lo + len && tid == 0) {
      K[bi - lo] = -INFINITY;
      a.tokens[out_b + fc + round] = bi;
      if (a.draft_prob) a.draft_prob[out_b + fc + round] = expf(Z[bi - lo] - mx[0]) * inv_sum;
    }
    if (!valid && c.rank == 0 && tid == 0) {
      a.tokens[out_b + fc + round] = -1;
      if (a.draft_prob) a.draft_prob[out_b + fc + round] = 0.f;
    }
    __syncthreads();
  }
  cluster_sync();
}

static bool sampler_shape(int V, int rows, int* cs_out, int* sl_out, size_t* smem_out, int override_cs) {
  auto smem_for = [&](int sl) { return static_cast<size_t>(2) * sl * 4 + kSamplerFixedSmem; };
  int cs = 1;
  if (override_cs > 0) {
    cs = override_cs;
  } else {
    while (cs < kMaxCluster && (V + cs - 1) / cs > 4096) cs *= 2;
    while (cs < 8 && rows * cs < 296 && (V + cs - 1) / cs > 1024) cs *= 2;
  }
  int sl = (((V + cs - 1) / cs) + 7) & ~7;
  while (cs < kMaxCluster && smem_for(sl) > 227 * 1024) {
    cs *= 2;
    sl = (((V + cs - 1) / cs) + 7) & ~7;
  }
  if (smem_for(sl) > 227 * 1024) return false;
  *cs_out = cs; *sl_out = sl; *smem_out = smem_for(sl);
  return true;
}

template <typename T, bool CFG>
static cudaError_t launch_sampler(const SampleArgs& a, int n_parents, int cs, size_t smem, cudaStream_t st) {
  auto kern = sample_children_kernel<T, CFG>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (e != cudaSuccess) return e;
  if (cs > 8) {
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
    if (e != cudaSuccess) return e;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(a.B) * n_parents * cs, 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = cs;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, a);
}

}  // namespace lantern

using namespace lantern;

extern "C" int32_t lantern_set_cluster_size(int32_t);

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
  int cs, sl;
  size_t smem;
  int ov = lantern_set_cluster_size(-1);     // -1 is not a valid size: reads the current value
  if (!sampler_shape(V, batch * (i1 - i0), &cs, &sl, &smem, ov)) return LANTERN_ERR_UNSUPPORTED;
  a.SL = sl;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const bool cfg = draft_uncond != nullptr;
  cudaError_t e;
  if (dt == LANTERN_F32)
    e = cfg ? launch_sampler<float, true>(a, i1 - i0, cs, smem, st) : launch_sampler<float, false>(a, i1 - i0, cs, smem, st);
  else
    e = cfg ? launch_sampler<__nv_bfloat16, true>(a, i1 - i0, cs, smem, st)
            : launch_sampler<__nv_bfloat16, false>(a, i1 - i0, cs, smem, st);
  return e == cudaSuccess ? LANTERN_OK : LANTERN_ERR_CUDA;
}
