// Row-level building blocks shared by the verify and the draft-sampler kernels.
//
// A logit row of V entries is split over the CTAs of one thread-block cluster; CTA `rank`
// owns the contiguous slice [rank*SL, min(V, (rank+1)*SL)) and keeps its float32 values in
// its own shared memory.  Row-wide reductions go through distributed shared memory.
#pragma once

#include "common.cuh"

namespace lantern {

struct ClusterCtx {
  uint32_t rank, nrank;
  int parity;        // slot of xch used by the next reduction
  int hist_parity;   // histogram buffer used by the next radix pass
  float* xch;        // smem [2][4]  this CTA's partials, read by the peers
  float* gath;       // smem [kMaxCluster*4]
  float* red;        // smem [kWarps*4]
  uint32_t* hist;    // smem [2 buffers][2 rows][256]
  int* sel;          // smem [2 rows][2]  (digit, remaining rank) of a radix pass
};

// Row-wide sum or max of NV values per thread (NV <= 4).  Every thread of every CTA of the
// cluster gets the same result: partials are combined in warp order, then in rank order.
template <int NV, bool IS_MAX>
__device__ __forceinline__ void cluster_reduce(ClusterCtx& c, float (&v)[NV]) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int i = 0; i < NV; ++i) v[i] = IS_MAX ? warp_max(v[i]) : warp_sum(v[i]);
  if (lane == 0) {
#pragma unroll
    for (int i = 0; i < NV; ++i) c.red[warp * NV + i] = v[i];
  }
  __syncthreads();
  if (threadIdx.x < NV) {
    float a = c.red[threadIdx.x];
    for (int w = 1; w < kWarps; ++w) {
      float b = c.red[w * NV + threadIdx.x];
      a = IS_MAX ? fmaxf(a, b) : a + b;
    }
    c.xch[c.parity * 4 + threadIdx.x] = a;
  }
  cluster_sync();
  if (threadIdx.x < c.nrank * NV) {
    uint32_t r = threadIdx.x / NV, i = threadIdx.x % NV;
    c.gath[threadIdx.x] = dsmem_ld_f32(dsmem_addr(smem_u32(&c.xch[c.parity * 4 + i]), r));
  }
  __syncthreads();
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    float a = c.gath[i];
    for (uint32_t r = 1; r < c.nrank; ++r) {
      float b = c.gath[r * NV + i];
      a = IS_MAX ? fmaxf(a, b) : a + b;
    }
    v[i] = a;
  }
  c.parity ^= 1;
}

// ---------------------------------------------------------------- loading a slice
template <typename T> struct Vec;
template <> struct Vec<float> {
  static constexpr int N = 4;
  using V = float4;
  __device__ static __forceinline__ void unpack(const V& v, float (&f)[4]) {
    f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w;
  }
  __device__ static __forceinline__ float widen(float x) { return x; }
};
template <> struct Vec<__nv_bfloat16> {
  static constexpr int N = 8;
  using V = uint4;
  __device__ static __forceinline__ void unpack(const V& v, float (&f)[8]) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      f[2 * i] = __uint_as_float(w[i] << 16);
      f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
  __device__ static __forceinline__ float widen(__nv_bfloat16 x) { return __bfloat162float(x); }
};

// Pre-softmax value (App. B "Models"): guidance with one fused multiply-add, then 1/tau.
// Explicit intrinsics keep the compiler from contracting or reassociating.
template <bool CFG>
__device__ __forceinline__ float combine(float c, float u, float g, float inv_tau) {
  if (CFG) return __fmul_rn(__fmaf_rn(g, __fsub_rn(c, u), u), inv_tau);
  return __fmul_rn(c, inv_tau);
}

// z[0..len) = post-processed logits of row elements [lo, lo+len); returns this thread's max.
// cond/uncond point at element 0 of the row; lo is a multiple of 8 and rows are 16-byte
// aligned, so vector loads are aligned.  Streaming loads: every element is read once.
template <typename T, bool CFG>
__device__ __forceinline__ float load_slice(const T* __restrict__ cond, const T* __restrict__ uncond,
                                            float g, float inv_tau, int lo, int len, int allow_lo,
                                            int allow_hi, float* __restrict__ z) {
  using VT = Vec<T>;
  constexpr int VN = VT::N;
  constexpr int U = 4;
  const typename VT::V* cv = reinterpret_cast<const typename VT::V*>(cond + lo);
  const typename VT::V* uv = reinterpret_cast<const typename VT::V*>(CFG ? uncond + lo : cond + lo);
  const int nvec = len / VN;
  float mx = -INFINITY;
  for (int base = 0; base < nvec; base += kThreads * U) {
    typename VT::V cr[U], ur[U];
#pragma unroll
    for (int k = 0; k < U; ++k) {
      int i = base + k * kThreads + threadIdx.x;
      if (i < nvec) {
        cr[k] = __ldcs(cv + i);
        if (CFG) ur[k] = __ldcs(uv + i);
      }
    }
#pragma unroll
    for (int k = 0; k < U; ++k) {
      int i = base + k * kThreads + threadIdx.x;
      if (i < nvec) {
        float cf[VN], uf[VN], zf[VN];
        VT::unpack(cr[k], cf);
        if (CFG) VT::unpack(ur[k], uf);
        int j0 = lo + i * VN;
#pragma unroll
        for (int e = 0; e < VN; ++e) {
          float v = combine<CFG>(cf[e], CFG ? uf[e] : 0.f, g, inv_tau);
          int j = j0 + e;
          if (j < allow_lo || j >= allow_hi) v = -INFINITY;
          zf[e] = v;
          mx = fmaxf(mx, v);
        }
        float4* dst = reinterpret_cast<float4*>(z + i * VN);
#pragma unroll
        for (int e = 0; e < VN; e += 4) dst[e / 4] = make_float4(zf[e], zf[e + 1], zf[e + 2], zf[e + 3]);
      }
    }
  }
  for (int i = nvec * VN + threadIdx.x; i < len; i += kThreads) {   // ragged tail
    float c = VT::widen(cond[lo + i]);
    float u = CFG ? VT::widen(uncond[lo + i]) : 0.f;
    float v = combine<CFG>(c, u, g, inv_tau);
    int j = lo + i;
    if (j < allow_lo || j >= allow_hi) v = -INFINITY;
    z[i] = v;
    mx = fmaxf(mx, v);
  }
  // pad to a multiple of 4 so that later float4 sweeps may cover the padding
  if (threadIdx.x < 4 && len > 0) {
    int i = len + threadIdx.x;
    if (i < ((len + 3) & ~3)) z[i] = -INFINITY;
  }
  return mx;
}

// ---------------------------------------------------------------- exact top-k threshold
// theta[r] = the kth[r]-th largest value of row r (r < NR rows, each split over the cluster;
// this CTA holds z[r][0..len)).  Radix select on the monotone key, 4 passes of 8 bits; the
// rows are processed in lockstep so that they share the cluster barriers.  inactive rows
// (kth <= 0) get theta = -inf.
template <int NR>
__device__ __forceinline__ void cluster_topk_threshold(ClusterCtx& c, float* const (&z)[NR], int len,
                                                       const int (&kth)[NR], float (&theta)[NR]) {
  uint32_t prefix[NR];
  int remaining[NR];
#pragma unroll
  for (int r = 0; r < NR; ++r) { prefix[r] = 0; remaining[r] = kth[r]; }
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    uint32_t* hb = c.hist + c.hist_parity * (2 * 256);
#pragma unroll
    for (int r = 0; r < NR; ++r) hb[r * 256 + threadIdx.x] = 0;   // kThreads == 256
    __syncthreads();
#pragma unroll
    for (int r = 0; r < NR; ++r) {
      if (kth[r] <= 0) continue;
      for (int j = threadIdx.x; j < len; j += kThreads) {
        uint32_t key = float_key(z[r][j]);
        if (pass == 0 || (key >> (shift + 8)) == prefix[r]) atomicAdd(&hb[r * 256 + ((key >> shift) & 255u)], 1u);
      }
    }
    cluster_sync();
    // bin threadIdx.x summed over the cluster
    uint32_t g[NR];
#pragma unroll
    for (int r = 0; r < NR; ++r) {
      g[r] = 0;
      if (kth[r] > 0) {
        uint32_t a = smem_u32(&hb[r * 256 + threadIdx.x]);
        for (uint32_t q = 0; q < c.nrank; ++q) g[r] += dsmem_ld_u32(dsmem_addr(a, q));
      }
    }
    // warp r walks the 256 bins from the top: lane l covers bins 255-8l .. 248-8l
    // (the cluster-wide bins are staged in the histogram buffer of the other parity)
    uint32_t* gb = c.hist + (c.hist_parity ^ 1) * (2 * 256);
    __syncthreads();            // everyone has read its peers' bins of this pass
#pragma unroll
    for (int r = 0; r < NR; ++r) gb[r * 256 + threadIdx.x] = g[r];
    __syncthreads();
    if (warp < NR && kth[warp % NR] > 0) {
      const int r = warp;
      uint32_t cnt[8], s = 0;
#pragma unroll
      for (int i = 0; i < 8; ++i) { cnt[i] = gb[r * 256 + 255 - (8 * lane + i)]; s += cnt[i]; }
      uint32_t incl = s;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
      }
      uint32_t excl = incl - s;
      uint32_t need = static_cast<uint32_t>(remaining[r]);
      if (excl < need && need <= incl) {
        uint32_t run = excl;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          if (run < need && need <= run + cnt[i]) {
            c.sel[r * 2 + 0] = 255 - (8 * lane + i);
            c.sel[r * 2 + 1] = static_cast<int>(need - run);
          }
          run += cnt[i];
        }
      }
    }
    __syncthreads();
#pragma unroll
    for (int r = 0; r < NR; ++r) {
      if (kth[r] > 0) {
        prefix[r] = (prefix[r] << 8) | static_cast<uint32_t>(c.sel[r * 2 + 0]);
        remaining[r] = c.sel[r * 2 + 1];
      }
    }
    // The next pass zeroes the buffer that held the cluster-wide bins (gb); peers read only
    // hb of this pass, and they will have passed the next cluster barrier before hb is
    // zeroed again two passes from now.
    c.hist_parity ^= 1;
  }
#pragma unroll
  for (int r = 0; r < NR; ++r) theta[r] = kth[r] > 0 ? key_float(prefix[r]) : -INFINITY;
}

}  // namespace lantern
