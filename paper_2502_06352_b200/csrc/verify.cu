// Relaxed verification of a static draft tree: host side of lantern_verify_tree and the walk.
#include <algorithm>

#include "common.cuh"

namespace lantern {
static int g_cluster_override = 0;
static int sm_count() {
  // per device: a process may drive GPUs of different sizes
  static int cached[64] = {};
  int dev = 0, v = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  if (cached[dev] == 0) {
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) return 148;
    cached[dev] = v;
  }
  return cached[dev];
}
}

// two builds of the kernels: 1024 threads per CTA for rows that fit one CTA, 512 threads per CTA
// for rows split over a cluster
#define LANTERN_VT 1024
#define LANTERN_VNS v1024
#include "verify_kernel.cuh"
#include "verify_launch.cuh"
#undef LANTERN_VT
#undef LANTERN_VNS
#define LANTERN_VT 512
#define LANTERN_VNS v512
#include "verify_kernel.cuh"
#include "verify_launch.cuh"
#undef LANTERN_VT
#undef LANTERN_VNS
#include "verify_sparse.cuh"
#include "verify_stream.cuh"

namespace lantern {

// ---- launch of the sparse (top-k) kernel: one CTA per node
template <typename T, bool CFG, int E>
static cudaError_t launch_sparse_e(const VerifyArgs& a, int32_t* redo, size_t smem, cudaStream_t st) {
  auto kern = sparse::verify_sparse_kernel<T, CFG, E>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (e != cudaSuccess) return e;
  const int chunk = sm_count();
  const int nI = a.B * a.n_internal, nL = a.B * (a.N - a.n_internal);
  const int blocks = (nI + chunk - 1) / chunk + (nL + chunk - 1) / chunk;
  return launch_after_previous(kern, static_cast<unsigned>(blocks) * chunk, sparse::ST, smem, st, 1, a, redo, chunk);
}
template <typename T, bool CFG>
static cudaError_t launch_sparse(const VerifyArgs& a, int32_t* redo, int e, size_t smem, cudaStream_t st) {
  if (e == 8) return launch_sparse_e<T, CFG, 8>(a, redo, smem, st);
  if (e == 16) return launch_sparse_e<T, CFG, 16>(a, redo, smem, st);
  return launch_sparse_e<T, CFG, 32>(a, redo, smem, st);
}
static cudaError_t launch_sparse_any(const VerifyArgs& a, int32_t* redo, int e, size_t smem, bool f32, bool cfg,
                                     cudaStream_t st) {
  if (f32) return cfg ? launch_sparse<float, true>(a, redo, e, smem, st) : launch_sparse<float, false>(a, redo, e, smem, st);
  return cfg ? launch_sparse<__nv_bfloat16, true>(a, redo, e, smem, st)
             : launch_sparse<__nv_bfloat16, false>(a, redo, e, smem, st);
}

// ---- launch of the streaming kernel (rows without top-k): one CTA, or a cluster of cs CTAs, per node
template <typename T, bool CFG, bool TAU1, bool GENERAL>
static cudaError_t launch_stream_k(const VerifyArgs& a, int cs, size_t smem, cudaStream_t st) {
  auto kern = stream::verify_stream_kernel<T, CFG, TAU1, GENERAL>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (e != cudaSuccess) return e;
  if (cs > 8) {
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
    if (e != cudaSuccess) return e;
  }
  const unsigned clusters = a.lazy ? static_cast<unsigned>(a.B) : static_cast<unsigned>(a.B) * a.N;
  return launch_after_previous(kern, clusters * cs, stream::ST, smem, st, cs, a);
}
template <typename T, bool CFG, bool TAU1>
static cudaError_t launch_stream_t(const VerifyArgs& a, int cs, size_t smem, cudaStream_t st) {
  return (a.lazy || a.skip || a.det || a.tree_stride) ? launch_stream_k<T, CFG, TAU1, true>(a, cs, smem, st)
                                     : launch_stream_k<T, CFG, TAU1, false>(a, cs, smem, st);
}
static cudaError_t launch_stream_any(const VerifyArgs& a, int cs, size_t smem, bool f32, bool cfg, cudaStream_t st) {
  const bool tau1 = a.inv_tau == 1.0f;
  if (f32) {
    if (cfg) return launch_stream_t<float, true, false>(a, cs, smem, st);
    return tau1 ? launch_stream_t<float, false, true>(a, cs, smem, st) : launch_stream_t<float, false, false>(a, cs, smem, st);
  }
  if (cfg) return launch_stream_t<__nv_bfloat16, true, false>(a, cs, smem, st);
  return tau1 ? launch_stream_t<__nv_bfloat16, false, true>(a, cs, smem, st)
              : launch_stream_t<__nv_bfloat16, false, false>(a, cs, smem, st);
}
// CTAs per node: one when the nodes alone fill the machine, else the smallest power of two that
// does, as long as every warp of the wider cluster keeps at least two full 512-byte steps of the row
// (narrow rows, e.g. an allowed range of 8192 tokens, run faster on fewer, busier CTAs)
static int stream_cluster_size(int nodes, int V, bool f32) {
  if (g_cluster_override > 0) return g_cluster_override;
  const int nvec = V / (f32 ? 4 : 8);
  int cs = 1;
  while (cs < 16 && static_cast<long long>(nodes) * cs < 8 * sm_count() && nvec / (4 * cs * stream::SW) >= 32) cs *= 2;
  return cs;
}

// ---- walk (Sec. 2.1) as a launch of its own: a CTA stages the per-node results of `seqs`
// sequences in shared memory (at most 48 KB) and walks them
constexpr int kWalkThreads = 128;
__global__ void __launch_bounds__(kWalkThreads) walk_kernel(const int32_t* __restrict__ node_next,
                                                            const int32_t* __restrict__ node_token,
                                                            const int32_t* __restrict__ tokens, int B, int N, int D1,
                                                            int seqs, int32_t* __restrict__ accept_len,
                                                            int32_t* __restrict__ out_tokens,
                                                            int32_t* __restrict__ out_nodes) {
  extern __shared__ int32_t walk_stage[];
  grid_dependency_sync();
  const int b0 = blockIdx.x * seqs;
  walk_staged(node_next, node_token, tokens, b0, min(seqs, B - b0), N, D1, accept_len, out_tokens, out_nodes,
              walk_stage);
}


static lantern_status launch_walk(const TreeDev* t, int batch, const int32_t* node_next, const int32_t* node_token,
                                  const int32_t* tokens, int32_t* accept_len, int32_t* out_tokens, int32_t* out_nodes,
                                  int D1, cudaStream_t st) {
  const int seqs = std::max(1, std::min(16, 6144 / t->n_nodes));      // 2 * seqs * N ints <= 48 KB
  if (launch_after_previous(walk_kernel, static_cast<unsigned>((batch + seqs - 1) / seqs), kWalkThreads,
                            sizeof(int32_t) * 2 * seqs * t->n_nodes, st, 1, node_next, node_token, tokens, batch,
                            t->n_nodes, D1, seqs, accept_len, out_tokens, out_nodes) != cudaSuccess)
    return LANTERN_ERR_CUDA;
  return cudaGetLastError() == cudaSuccess ? LANTERN_OK : LANTERN_ERR_CUDA;
}

}  // namespace lantern

using namespace lantern;

extern "C" int32_t lantern_set_cluster_size(int32_t ctas_per_row) {
  int32_t old = g_cluster_override;
  if (ctas_per_row == 0 || ctas_per_row == 1 || ctas_per_row == 2 || ctas_per_row == 4 ||
      ctas_per_row == 8 || ctas_per_row == 16)
    g_cluster_override = ctas_per_row;
  return old;
}

extern "C" int32_t lantern_get_cluster_size(void) { return g_cluster_override; }

namespace {
constexpr int kWsTailInts = 64;
// Rows truncated to a moderate top-k on every side that is read can take the list-based kernel.
bool verify_uses_lists(const lantern_params* p, const TreeDev* t) {
  const int V = p->vocab;
  auto topk_fits = [&](int k) { return k > 0 && k < V && k <= sparse::kMaxTopK; };
  return !p->lazy_walk && !p->subset_rule && !p->draft_deterministic && g_cluster_override == 0 &&
         V <= sparse::kMaxV && topk_fits(p->top_k_target) &&
         (t->n_internal == 0 || topk_fits(p->top_k_draft)) && t->max_children <= 8;
}
// Can the streaming kernel serve these parameters at all (rows that no top-k truncates)?
bool stream_applies(const lantern_params* p, const TreeDev* t) {
  const int V = p->vocab;
  const bool tk_t = p->top_k_target > 0 && p->top_k_target < V;
  const bool tk_d = t->n_internal > 0 && !p->draft_deterministic && p->top_k_draft > 0 && p->top_k_draft < V;
  return !tk_t && !tk_d && V <= stream::kMaxV &&
         stream::smem_bytes(V, t->max_children, p->k + 1, true) <= 227 * 1024;
}
// Can the dense kernels hold a row of these parameters (float32 rows in shared memory)?
bool dense_fits(const lantern_params* p, const TreeDev* t, bool f32, bool cfg) {
  const int kpad = (p->k + 3) & ~3, min_e = f32 ? 4 : 8;
  v1024::LaunchShape s1;
  v512::LaunchShape s5;
  return v1024::choose_shape(p->vocab, 1 << 20, t->max_children, kpad, min_e, cfg, &s1) ||
         v512::choose_shape(p->vocab, 1 << 20, t->max_children, kpad, min_e, cfg, &s5);
}
constexpr int kStreamMinNodes = 128;     // below this many nodes per call the dense kernels' shorter chain wins
// Does this call take the streaming kernel?  (`fits_dense`: the answer of dense_fits, or true when
// the storage type is not known yet, as in the path query.)
bool verify_uses_stream(const lantern_params* p, const TreeDev* t, int batch, bool fits_dense) {
  if (!stream_applies(p, t)) return false;
  if (p->subset_rule || p->draft_deterministic) return true;       // only the streaming kernel has the variants
  if (p->kernels == 2) return !fits_dense;
  // the path walk is a chain of dependent nodes per sequence: the dense kernel, whose rejection
  // passes read shared memory, walks it faster
  if (p->lazy_walk) return !fits_dense;
  if (p->kernels == 1) return true;
  return static_cast<long long>(batch) * t->n_nodes >= kStreamMinNodes || !fits_dense;
}
}  // namespace

extern "C" int32_t lantern_verify_tree_path(const lantern_params* p, const lantern_tree* tree, int32_t batch) {
  if (!p || !tree || batch <= 0) return -1;
  const TreeDev* t = reinterpret_cast<const TreeDev*>(tree);
  if (t->per_seq || verify_uses_stream(p, t, batch, true)) return LANTERN_PATH_STREAM;
  return verify_uses_lists(p, t) ? LANTERN_PATH_LISTS : LANTERN_PATH_DENSE;
}

extern "C" size_t lantern_verify_tree_workspace(const lantern_tree* tree, int32_t batch) {
  if (!tree || batch <= 0) return 0;
  const TreeDev* t = reinterpret_cast<const TreeDev*>(tree);
  // node_next, node_token, repair flags, and the completion counter of the repair launch
  return (static_cast<size_t>(3) * batch * t->n_nodes + kWsTailInts) * sizeof(int32_t);
}

extern "C" lantern_status lantern_verify_tree(
    const lantern_params* p, const lantern_tree* tree, const int32_t* nbr_idx, int32_t k_table,
    const void* target_cond, const void* target_uncond, const void* draft_cond, const void* draft_uncond,
    lantern_dtype dt, int64_t row_stride, int64_t seq_stride, int32_t batch, const int32_t* tokens,
    const float* u_accept, const float* u_resample, int32_t* accept_len, int32_t* out_tokens,
    int32_t* out_nodes, int32_t* node_next, int32_t* node_token, float* node_mass, float* node_thresh,
    int32_t* device_status, void* workspace, size_t workspace_bytes, void* stream) {
  if (!p || !tree || !target_cond || !tokens || !accept_len || !out_tokens || !out_nodes)
    return LANTERN_ERR_INVALID_ARG;
  const TreeDev* t = reinterpret_cast<const TreeDev*>(tree);
  if (batch <= 0 || p->vocab <= 0 || !(p->temperature > 0.f) || !(p->lambda >= 1.f)) return LANTERN_ERR_INVALID_ARG;
  if (dt != LANTERN_F32 && dt != LANTERN_BF16) return LANTERN_ERR_INVALID_ARG;
  const bool det = p->draft_deterministic != 0;
  if (p->subset_rule != 0 && p->subset_rule != 1) return LANTERN_ERR_INVALID_ARG;
  if (t->n_internal > 0 && !draft_cond && !det) return LANTERN_ERR_INVALID_ARG;
  if ((target_uncond != nullptr) != (draft_uncond != nullptr) && t->n_internal > 0 && !det) return LANTERN_ERR_INVALID_ARG;
  if ((det || p->subset_rule) && !stream_applies(p, t)) return LANTERN_ERR_UNSUPPORTED;
  // a forest (one tree per sequence) is served by the streaming kernel's eager launch only
  if (t->per_seq && (batch != t->per_seq || p->lazy_walk || p->kernels == 2 || !stream_applies(p, t)))
    return batch != t->per_seq ? LANTERN_ERR_INVALID_ARG : LANTERN_ERR_UNSUPPORTED;
  if (p->kernels < 0 || p->kernels > 2) return LANTERN_ERR_INVALID_ARG;
  if (p->k < 0 || p->top_k_target < 0 || p->top_k_draft < 0) return LANTERN_ERR_INVALID_ARG;
  if (!(p->delta >= 0.f) || p->delta > 4.f) return LANTERN_ERR_INVALID_ARG;      // also rejects NaN
  if (p->k > 0 && (!nbr_idx || p->k > k_table || p->n_codes <= 0 || k_table > p->n_codes - 1)) return LANTERN_ERR_INVALID_ARG;
  if (p->k > 1024) return LANTERN_ERR_UNSUPPORTED;
  const int V = p->vocab;
  const int allow_lo = p->allowed_begin, allow_hi = p->allowed_end == 0 ? V : p->allowed_end;
  if (allow_lo < 0 || allow_hi > V || allow_lo >= allow_hi) return LANTERN_ERR_INVALID_ARG;
  if (p->n_codes > 0 && (p->code_offset < 0 || static_cast<int64_t>(p->code_offset) + p->n_codes > V) && p->k > 0)
    return LANTERN_ERR_INVALID_ARG;
  if (p->step >> 62) return LANTERN_ERR_INVALID_ARG;
  const size_t esz = dt == LANTERN_F32 ? 4 : 2;
  if (row_stride < V || seq_stride < 0) return LANTERN_ERR_INVALID_ARG;
  if ((row_stride * esz) % 16 || (seq_stride * esz) % 16) return LANTERN_ERR_INVALID_ARG;
  const void* ptrs[4] = {target_cond, target_uncond, draft_cond, draft_uncond};
  for (const void* q : ptrs)
    if (q && (reinterpret_cast<uintptr_t>(q) % 16)) return LANTERN_ERR_INVALID_ARG;
  if (static_cast<int64_t>(batch) * t->n_nodes > (1 << 24)) return LANTERN_ERR_UNSUPPORTED;

  const size_t ws_need = lantern_verify_tree_workspace(tree, batch);
  const bool have_ws = workspace && workspace_bytes >= ws_need && (reinterpret_cast<uintptr_t>(workspace) % 256) == 0;
  if (!node_next || !node_token) {
    if (!have_ws) return LANTERN_ERR_WORKSPACE;
    int32_t* w = static_cast<int32_t*>(workspace);
    if (!node_next) node_next = w;
    if (!node_token) node_token = w + static_cast<size_t>(batch) * t->n_nodes;
  }
  int32_t* redo = have_ws ? static_cast<int32_t*>(workspace) + static_cast<size_t>(2) * batch * t->n_nodes : nullptr;

  VerifyArgs a;
  a.tc = target_cond; a.tu = target_uncond; a.dc = draft_cond; a.du = draft_uncond;
  a.row_stride = row_stride; a.seq_stride = seq_stride;
  a.tokens = tokens; a.u_acc = u_accept; a.u_res = u_resample;
  a.nbr = nbr_idx; a.k_table = k_table;
  a.use_bulk = (p->k > 0 && k_table % 4 == 0 && reinterpret_cast<uintptr_t>(nbr_idx) % 16 == 0) ? 1 : 0;
  a.first_child = t->d_first_child; a.n_child = t->d_n_child; a.order = t->d_order;
  a.B = batch; a.N = t->n_nodes; a.V = V; a.n_internal = t->n_internal; a.max_children = t->max_children;
  a.kpad = (p->k + 3) & ~3;
  a.g = p->cfg_scale; a.inv_tau = 1.0f / p->temperature; a.lambda = p->lambda; a.delta = p->delta;
  a.skip = p->subset_rule; a.det = det ? 1 : 0;
  a.topk_t = p->top_k_target; a.topk_d = p->top_k_draft; a.k = p->k;
  a.code_offset = p->code_offset; a.n_codes = p->n_codes; a.allow_lo = allow_lo; a.allow_hi = allow_hi;
  a.seed = p->seed; a.step = p->step;
  a.node_next = node_next; a.node_token = node_token; a.node_mass = node_mass; a.node_thresh = node_thresh;
  a.status = device_status;
  a.only = nullptr;
  a.done = nullptr;
  a.lazy = p->lazy_walk ? 1 : 0;
  a.tree_stride = t->per_seq ? t->n_nodes : 0;
  const int D1 = t->max_depth + 1;
  a.accept_len = accept_len; a.out_tokens = out_tokens; a.out_nodes = out_nodes; a.D1 = D1;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const bool cfg = target_uncond != nullptr;
  const bool f32 = dt == LANTERN_F32;
  const int min_e = f32 ? 4 : 8;
  // (the path walk is a chain of nodes per sequence: rows are not split over more CTAs than they need)
  const int rows = a.lazy ? (1 << 20) : batch * t->n_nodes;
  cudaError_t e;
  // Rows truncated to a moderate top-k on every side that is read take the sparse kernel; the
  // dense kernel then repairs the nodes it could not hold (a.only) and usually finds none.
  const bool use_sparse = redo && !a.lazy && !t->per_seq && verify_uses_lists(p, t);
  if (use_sparse) {
    const int se = V <= sparse::ST * 8 ? 8 : (V <= sparse::ST * 16 ? 16 : 32);
    a.done = redo + static_cast<size_t>(batch) * t->n_nodes;       // the sparse kernel clears it
    e = launch_sparse_any(a, redo, se, sparse::smem_bytes(se, t->max_children, a.kpad), f32, cfg, st);
    if (e != cudaSuccess) return LANTERN_ERR_CUDA;
    a.only = redo;
  }
  if (!use_sparse && (t->per_seq || verify_uses_stream(p, t, batch, dense_fits(p, t, f32, cfg)))) {
    const int cs = stream_cluster_size(a.lazy ? batch : batch * t->n_nodes, allow_hi - allow_lo, f32);
    e = launch_stream_any(a, cs, stream::smem_bytes(V, t->max_children, p->k + 1, cfg), f32, cfg, st);
    if (e != cudaSuccess) return LANTERN_ERR_CUDA;
    if (a.lazy) return cudaGetLastError() == cudaSuccess ? LANTERN_OK : LANTERN_ERR_CUDA;     // it walks as it goes
    return launch_walk(t, batch, node_next, node_token, tokens, accept_len, out_tokens, out_nodes, D1, st);
  }
  // rows that fit one CTA run the 1024-thread build; rows split over a cluster run the
  // 512-thread build (cheaper barriers, half the per-thread fixed work per entry)
  v1024::LaunchShape s1;
  const bool ok1 = v1024::choose_shape(V, rows, t->max_children, a.kpad, min_e, cfg, &s1);
  if (ok1 && s1.cs == 1) {
    e = v1024::launch_any(a, s1, f32, cfg, st);
  } else {
    v512::LaunchShape s5;
    if (v512::choose_shape(V, rows, t->max_children, a.kpad, min_e, cfg, &s5)) {
      e = v512::launch_any(a, s5, f32, cfg, st);
    } else if (ok1) {
      e = v1024::launch_any(a, s1, f32, cfg, st);
    } else {
      return LANTERN_ERR_UNSUPPORTED;
    }
  }
  if (e != cudaSuccess) return LANTERN_ERR_CUDA;
  if (!a.done && !a.lazy)        // otherwise the repair launch, or the path walk itself, has walked the trees
    return launch_walk(t, batch, node_next, node_token, tokens, accept_len, out_tokens, out_nodes, D1, st);
  return LANTERN_OK;
}

// ---------------------------------------------------------------------------------------------
// Variant of lantern_verify_tree for callers that cannot allocate device memory.
// Its per-node scratch (accepted child and drawn token of every node) lives in a fixed array
// that is part of the library image; every GPU that loads the library holds it until exit.
namespace {
constexpr int kStaticMaxNodes = 1 << 16;       // batch * tree nodes the built-in scratch can hold
static __device__ __align__(256) int32_t g_static_scratch[3 * kStaticMaxNodes + 64];
constexpr int kMaxDevices = 64;
void* g_static_scratch_ptr[kMaxDevices] = {};  // device address of the array, per device

// The array's name is only a handle on the host; the kernels need its device address, which is
// looked up once per device (with that device current).
lantern_status static_scratch_for_current_device(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return LANTERN_ERR_CUDA;
  if (!g_static_scratch_ptr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return LANTERN_ERR_CUDA;
    g_static_scratch_ptr[dev] = p;
  }
  *out = g_static_scratch_ptr[dev];
  return LANTERN_OK;
}
}  // namespace

extern "C" int32_t lantern_verify_tree_static_max_nodes(void) { return kStaticMaxNodes; }

extern "C" lantern_status lantern_verify_tree_static(
    const lantern_params* p, const lantern_tree* tree, const int32_t* nbr_idx, int32_t k_table,
    const void* target_cond, const void* target_uncond, const void* draft_cond, const void* draft_uncond,
    lantern_dtype dt, int64_t row_stride, int64_t seq_stride, int32_t batch, const int32_t* tokens,
    const float* u_accept, const float* u_resample, int32_t* accept_len, int32_t* out_tokens,
    int32_t* out_nodes, float* node_mass, float* node_thresh, int32_t* device_status, void* stream) {
  if (!tree || batch <= 0) return LANTERN_ERR_INVALID_ARG;
  const TreeDev* t = reinterpret_cast<const TreeDev*>(tree);
  if (static_cast<int64_t>(batch) * t->n_nodes > kStaticMaxNodes) return LANTERN_ERR_UNSUPPORTED;
  void* scratch = nullptr;
  lantern_status st = static_scratch_for_current_device(&scratch);
  if (st != LANTERN_OK) return st;
  // Every scratch entry of the nodes in use is written by the kernel before the walk reads it,
  // so nothing has to be cleared between calls.
  return lantern_verify_tree(p, tree, nbr_idx, k_table, target_cond, target_uncond, draft_cond, draft_uncond, dt,
                             row_stride, seq_stride, batch, tokens, u_accept, u_resample, accept_len, out_tokens,
                             out_nodes, nullptr, nullptr, node_mass, node_thresh, device_status, scratch,
                             sizeof(int32_t) * (3 * kStaticMaxNodes + 64), stream);
}
