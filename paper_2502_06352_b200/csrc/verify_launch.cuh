// Host-side launch helpers of the verify kernels; compiled once per thread-count variant,
// right after verify_kernel.cuh, into the same namespace.
namespace lantern {
namespace LANTERN_VNS {

struct LaunchShape { int cs, e; size_t smem; };
constexpr int kMaxE = 16384 / VT;      // a CTA's slice holds at most 16384 row entries

// Choose E (row entries per thread; a CTA's slice is 1024*E entries) and the cluster size.
// `min_e` is 4 for float32 rows and 8 for bfloat16 rows (one 16-byte vector per thread).
static bool choose_shape(int V, int rows, int max_children, int kpad, int min_e, bool cfg, LaunchShape* out) {
  auto smem_for = [&](int e) {
    return row_smem_bytes(cfg, e) + static_cast<size_t>(max_children) * kpad * 4;
  };
  auto cs_for = [&](int e) { int cs = (V + VT * e - 1) / (VT * e); return cs > 8 ? (cs > 16 ? 0 : 16) : cs; };
  int e = 0;
  if (g_cluster_override > 0) {
    for (int cand = min_e; cand <= kMaxE; cand *= 2)
      if (static_cast<long long>(VT) * cand * g_cluster_override >= V) { e = cand; break; }
    if (e == 0) return false;
    out->cs = g_cluster_override;
  } else {
    // the smallest slice that holds the row in one CTA, else the largest slice
    for (int cand = min_e; cand <= kMaxE; cand *= 2)
      if (VT * cand >= V) { e = cand; break; }
    if (e == 0) e = kMaxE;
    if (cs_for(e) == 0) return false;
    // few rows: split each over more CTAs so that more SMs stream
    while (e > min_e && static_cast<long long>(rows) * cs_for(e) < 74 && cs_for(e / 2) != 0 && cs_for(e / 2) <= 8) e /= 2;
    // shared memory: halve the slice (more CTAs per row) until the CTA fits
    while (smem_for(e) > 227 * 1024 && e > min_e && cs_for(e / 2) != 0) e /= 2;
    out->cs = cs_for(e);
  }
  out->e = e;
  out->smem = smem_for(e);
  return out->smem <= 227 * 1024;
}

template <typename T, bool CFG, int E>
static cudaError_t launch_verify_e(const VerifyArgs& a, const LaunchShape& sh, cudaStream_t st) {
  auto kern = verify_nodes_kernel<T, CFG, E>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(sh.smem));
  if (e != cudaSuccess) return e;
  if (sh.cs > 8) {
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
    if (e != cudaSuccess) return e;
  }
  // one cluster per node; a repair launch (a.only) gets about one cluster per SM and lets each
  // walk its share of the flagged nodes
  unsigned clusters = static_cast<unsigned>(a.B) * a.N;
  if (a.lazy) clusters = static_cast<unsigned>(a.B);       // path walk: one cluster per sequence
  if (a.only) {
    const unsigned per_wave = static_cast<unsigned>(sm_count() / sh.cs > 0 ? sm_count() / sh.cs : 1);
    if (clusters > per_wave) clusters = per_wave;
  }
  return launch_after_previous(kern, clusters * sh.cs, VT, sh.smem, st, sh.cs, a);
}

template <typename T, bool CFG>
static cudaError_t launch_verify(const VerifyArgs& a, const LaunchShape& sh, cudaStream_t st) {
  if constexpr (kMaxE >= 32) {
    if (sh.e == 32) return launch_verify_e<T, CFG, 32>(a, sh, st);
  }
  if (sh.e == 16) return launch_verify_e<T, CFG, 16>(a, sh, st);
  if (sh.e == 8) return launch_verify_e<T, CFG, 8>(a, sh, st);
  if constexpr (Vec<T>::N <= 4) {
    if (sh.e == 4) return launch_verify_e<T, CFG, 4>(a, sh, st);
  }
  return cudaErrorInvalidValue;
}


static cudaError_t launch_any(const VerifyArgs& a, const LaunchShape& sh, bool f32, bool cfg, cudaStream_t st) {
  if (f32) return cfg ? launch_verify<float, true>(a, sh, st) : launch_verify<float, false>(a, sh, st);
  return cfg ? launch_verify<__nv_bfloat16, true>(a, sh, st) : launch_verify<__nv_bfloat16, false>(a, sh, st);
}

}  // namespace LANTERN_VNS
}  // namespace lantern
