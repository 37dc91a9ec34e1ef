// Tree handle, status strings and the raw Philox entry point of the C ABI.
#include <stdlib.h>
#include <string.h>

#include "common.cuh"

using namespace lantern;

extern "C" const char* lantern_status_string(lantern_status s) {
  switch (s) {
    case LANTERN_OK: return "ok";
    case LANTERN_ERR_INVALID_ARG: return "invalid argument";
    case LANTERN_ERR_UNSUPPORTED: return "unsupported size";
    case LANTERN_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case LANTERN_ERR_CUDA: return "CUDA runtime error";
  }
  return "unknown status";
}

extern "C" lantern_status lantern_tree_create(const int32_t* parent, int32_t n_nodes, lantern_tree** out) {
  if (!parent || !out || n_nodes < 1) return LANTERN_ERR_INVALID_ARG;
  if (n_nodes > LANTERN_MAX_NODES) return LANTERN_ERR_UNSUPPORTED;
  if (parent[0] != -1) return LANTERN_ERR_INVALID_ARG;
  for (int i = 1; i < n_nodes; ++i) {
    if (parent[i] < 0 || parent[i] >= i) return LANTERN_ERR_INVALID_ARG;
    if (parent[i] < parent[i - 1]) return LANTERN_ERR_INVALID_ARG;   // breadth-first numbering
  }
  int32_t* host = static_cast<int32_t*>(malloc(sizeof(int32_t) * 4 * n_nodes));
  if (!host) return LANTERN_ERR_CUDA;
  int32_t* first_child = host;
  int32_t* n_child = host + n_nodes;
  int32_t* order = host + 2 * n_nodes;
  int32_t* depth = host + 3 * n_nodes;
  int max_children = 0, max_depth = 0, n_internal = 0;
  for (int i = 0; i < n_nodes; ++i) { first_child[i] = -1; n_child[i] = 0; depth[i] = 0; }
  for (int i = 1; i < n_nodes; ++i) {
    int p = parent[i];
    if (n_child[p] == 0) first_child[p] = i;
    ++n_child[p];
    depth[i] = depth[p] + 1;
    if (depth[i] > max_depth) max_depth = depth[i];
    if (n_child[p] > max_children) max_children = n_child[p];
  }
  if (max_children > LANTERN_MAX_CHILDREN) { free(host); return LANTERN_ERR_UNSUPPORTED; }
  int w = 0;
  for (int i = 0; i < n_nodes; ++i) if (n_child[i] > 0) { order[w++] = i; ++n_internal; }
  for (int i = 0; i < n_nodes; ++i) if (n_child[i] == 0) order[w++] = i;

  TreeDev* t = static_cast<TreeDev*>(calloc(1, sizeof(TreeDev)));
  if (!t) { free(host); return LANTERN_ERR_CUDA; }
  void* dev = nullptr;
  if (cudaMalloc(&dev, sizeof(int32_t) * 3 * n_nodes) != cudaSuccess ||
      cudaMemcpy(dev, host, sizeof(int32_t) * 3 * n_nodes, cudaMemcpyHostToDevice) != cudaSuccess) {
    if (dev) cudaFree(dev);
    free(host);
    free(t);
    return LANTERN_ERR_CUDA;
  }
  t->n_nodes = n_nodes;
  t->max_depth = max_depth;
  t->max_children = max_children;
  t->n_internal = n_internal;
  t->d_block = dev;
  t->d_first_child = static_cast<int32_t*>(dev);
  t->d_n_child = t->d_first_child + n_nodes;
  t->d_order = t->d_first_child + 2 * n_nodes;
  t->h_first_child = first_child;
  t->h_n_child = n_child;
  *out = reinterpret_cast<lantern_tree*>(t);
  return LANTERN_OK;
}

// A forest: one tree per sequence, all padded to max_nodes (Sec. 2.1, dynamic tree drafting: the
// shape of the draft tree depends on the sequence).  The device arrays are [batch][max_nodes];
// padding nodes have no children and an order entry of -1.
extern "C" lantern_status lantern_forest_create(const int32_t* parent, const int32_t* n_nodes, int32_t batch,
                                                int32_t max_nodes, lantern_tree** out) {
  if (!parent || !n_nodes || !out || batch < 1 || max_nodes < 1) return LANTERN_ERR_INVALID_ARG;
  if (max_nodes > LANTERN_MAX_NODES || static_cast<int64_t>(batch) * max_nodes > (1 << 24)) return LANTERN_ERR_UNSUPPORTED;
  const size_t BN = static_cast<size_t>(batch) * max_nodes;
  int32_t* host = static_cast<int32_t*>(malloc(sizeof(int32_t) * 4 * BN));
  if (!host) return LANTERN_ERR_CUDA;
  int32_t* first_child = host;
  int32_t* n_child = host + BN;
  int32_t* order = host + 2 * BN;
  int32_t* depth = host + 3 * BN;
  int max_children = 0, max_depth = 0, max_internal = 0;
  for (int b = 0; b < batch; ++b) {
    const int n = n_nodes[b];
    const int32_t* par = parent + static_cast<size_t>(b) * max_nodes;
    int32_t* fc = first_child + static_cast<size_t>(b) * max_nodes;
    int32_t* nc = n_child + static_cast<size_t>(b) * max_nodes;
    int32_t* od = order + static_cast<size_t>(b) * max_nodes;
    int32_t* dp = depth + static_cast<size_t>(b) * max_nodes;
    bool ok = n >= 1 && n <= max_nodes && par[0] == -1;
    for (int i = 1; ok && i < n; ++i) ok = par[i] >= 0 && par[i] < i && par[i] >= par[i - 1];   // breadth-first numbering
    if (!ok) { free(host); return LANTERN_ERR_INVALID_ARG; }
    for (int i = 0; i < max_nodes; ++i) { fc[i] = -1; nc[i] = 0; dp[i] = 0; od[i] = -1; }
    for (int i = 1; i < n; ++i) {
      const int p = par[i];
      if (nc[p] == 0) fc[p] = i;
      ++nc[p];
      dp[i] = dp[p] + 1;
      if (dp[i] > max_depth) max_depth = dp[i];
      if (nc[p] > max_children) max_children = nc[p];
    }
    int w = 0, internal = 0;
    for (int i = 0; i < n; ++i) if (nc[i] > 0) { od[w++] = i; ++internal; }
    for (int i = 0; i < n; ++i) if (nc[i] == 0) od[w++] = i;
    if (internal > max_internal) max_internal = internal;
  }
  if (max_children > LANTERN_MAX_CHILDREN) { free(host); return LANTERN_ERR_UNSUPPORTED; }
  TreeDev* t = static_cast<TreeDev*>(calloc(1, sizeof(TreeDev)));
  if (!t) { free(host); return LANTERN_ERR_CUDA; }
  void* dev = nullptr;
  if (cudaMalloc(&dev, sizeof(int32_t) * 3 * BN) != cudaSuccess ||
      cudaMemcpy(dev, host, sizeof(int32_t) * 3 * BN, cudaMemcpyHostToDevice) != cudaSuccess) {
    if (dev) cudaFree(dev);
    free(host);
    free(t);
    return LANTERN_ERR_CUDA;
  }
  t->n_nodes = max_nodes;
  t->max_depth = max_depth;
  t->max_children = max_children;
  t->n_internal = max_internal;
  t->per_seq = batch;
  t->d_block = dev;
  t->d_first_child = static_cast<int32_t*>(dev);
  t->d_n_child = t->d_first_child + BN;
  t->d_order = t->d_first_child + 2 * BN;
  t->h_first_child = first_child;
  t->h_n_child = n_child;
  *out = reinterpret_cast<lantern_tree*>(t);
  return LANTERN_OK;
}

extern "C" lantern_status lantern_tree_destroy(lantern_tree* tree) {
  if (!tree) return LANTERN_OK;
  TreeDev* t = reinterpret_cast<TreeDev*>(tree);
  cudaError_t e = cudaFree(t->d_block);
  free(t->h_first_child);   // base of the host block
  free(t);
  return e == cudaSuccess ? LANTERN_OK : LANTERN_ERR_CUDA;
}

extern "C" int32_t lantern_tree_max_depth(const lantern_tree* tree) {
  return tree ? reinterpret_cast<const TreeDev*>(tree)->max_depth : -1;
}

namespace {
__global__ void philox_raw_kernel(uint32_t k0, uint32_t k1, uint32_t first, uint32_t c1, uint32_t c2,
                                  uint32_t c3, int n, uint32_t* out) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  Philox4 r = philox4x32_10(first + static_cast<uint32_t>(i), c1, c2, c3, k0, k1);
  reinterpret_cast<uint4*>(out)[i] = make_uint4(r.x, r.y, r.z, r.w);
}
}  // namespace

extern "C" lantern_status lantern_philox_raw(uint64_t seed, uint32_t first, uint32_t c1, uint32_t c2,
                                             uint32_t c3, int32_t n, uint32_t* out, void* stream) {
  if (!out || n < 0 || (reinterpret_cast<uintptr_t>(out) % 16)) return LANTERN_ERR_INVALID_ARG;
  if (n == 0) return LANTERN_OK;
  philox_raw_kernel<<<(n + 255) / 256, 256, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<uint32_t>(seed), static_cast<uint32_t>(seed >> 32), first, c1, c2, c3, n, out);
  return cudaGetLastError() == cudaSuccess ? LANTERN_OK : LANTERN_ERR_CUDA;
}
