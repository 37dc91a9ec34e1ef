// Register-resident row phases of the verify kernel: load -> max -> top-k threshold -> exp.
//
// A CTA of 256 threads owns a slice of SL = 256*E row entries; warp w owns the contiguous
// segment [w*32E, (w+1)*32E).  While a row is being post-processed each thread keeps its E
// values in registers (vector v of the thread covers entries seg + v*32*VN + lane*VN ..+VN, so
// every global load instruction of a warp reads one contiguous 512-byte run).  Only the
// softmax numerators are written to shared memory, once.
#pragma once

#include "rowops.cuh"

namespace lantern {

constexpr float kLog2e = 1.4426950408889634f;
constexpr int kCandLocal = 256;    // top-k candidates one CTA may contribute per row
constexpr int kCandTotal = 1024;   // and the whole cluster
constexpr int kBinBase = (127 - 9) << 4;

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Load E entries per thread of one row slice and apply guidance and temperature.
// Entries at or beyond `len` become -inf.
template <typename T, bool CFG, int E>
__device__ __forceinline__ void load_row_regs(const T* __restrict__ cond, const T* __restrict__ uncond,
                                              float g, float inv_tau, int lo, int len, float (&z)[E]) {
  using VT = Vec<T>;
  constexpr int VN = VT::N, NV = E / VN;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int wb = warp * 32 * E + lane * VN;
  typename VT::V cr[NV], ur[NV];
#pragma unroll
  for (int v = 0; v < NV; ++v) {
    const int j = wb + v * 32 * VN;
    if (j + VN <= len) {
      cr[v] = __ldcs(reinterpret_cast<const typename VT::V*>(cond + lo + j));
      if (CFG) ur[v] = __ldcs(reinterpret_cast<const typename VT::V*>(uncond + lo + j));
    }
  }
#pragma unroll
  for (int v = 0; v < NV; ++v) {
    const int j = wb + v * 32 * VN;
    if (j + VN <= len) {
      float cf[VN], uf[VN];
      VT::unpack(cr[v], cf);
      if (CFG) VT::unpack(ur[v], uf);
#pragma unroll
      for (int e = 0; e < VN; ++e) z[v * VN + e] = combine<CFG>(cf[e], CFG ? uf[e] : 0.f, g, inv_tau);
    } else {
#pragma unroll
      for (int e = 0; e < VN; ++e) {
        float val = -INFINITY;
        if (j + e < len) {
          const float cc = VT::widen(cond[lo + j + e]);
          const float uu = CFG ? VT::widen(uncond[lo + j + e]) : 0.f;
          val = combine<CFG>(cc, uu, g, inv_tau);
        }
        z[v * VN + e] = val;
      }
    }
  }
}

// Tokens outside [allow_lo, allow_hi) get -inf.
template <int E, int VN>
__device__ __forceinline__ void mask_regs(float (&z)[E], int lo, int allow_lo, int allow_hi) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int wb = lo + warp * 32 * E + lane * VN;
#pragma unroll
  for (int v = 0; v < E / VN; ++v)
#pragma unroll
    for (int e = 0; e < VN; ++e) {
      const int j = wb + v * 32 * VN + e;
      if (j < allow_lo || j >= allow_hi) z[v * VN + e] = -INFINITY;
    }
}

template <int E>
__device__ __forceinline__ float max_regs(const float (&z)[E]) {
  float m = z[0];
#pragma unroll
  for (int e = 1; e < E; ++e) m = fmaxf(m, z[e]);
  return m;
}

// Coarse position of an entry below the row maximum: a monotone function of z (16 bins per
// binade of d = max - z, covering d in [2^-9, 2^7), clamped at both ends).
__device__ __forceinline__ int dist_bin(float mx, float z) {
  const float d = mx - z;
  const int b = static_cast<int>(__float_as_uint(d) >> 19) - kBinBase;
  return min(max(b, 0), 255);
}

struct TopkSmem {
  uint32_t* bins;     // [2][256]
  float* candl;       // [2][kCandLocal]  (also staging of the cluster-wide bins)
  float* all;         // [2][kCandTotal]  (aliased by the radix fallback's histograms)
  int* candn;         // [2] local candidate counts, [2..] scratch
};

// Exact top-k thresholds of up to two rows held in registers (row r active iff kth[r] > 0):
// theta[r] = kth[r]-th largest entry.  One histogram over dist_bin locates the bin of the
// k-th entry; the few entries of that bin are gathered cluster-wide and ranked exactly.
// Returns false when the candidates do not fit (caller falls back to the radix select);
// the decision is the same in every CTA of the cluster.
template <int E>
__device__ __forceinline__ bool topk_regs(ClusterCtx& c, const TopkSmem& s, const float (&z0)[E],
                                          const float (&z1)[E], const float (&mx)[2], const int (&kth)[2],
                                          float (&theta)[2]) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  s.bins[tid] = 0;
  s.bins[256 + tid] = 0;
  if (tid < 2) s.candn[tid] = 0;
  __syncthreads();
  if (kth[0] > 0) {
#pragma unroll
    for (int e = 0; e < E; ++e) atomicAdd(&s.bins[dist_bin(mx[0], z0[e])], 1u);
  }
  if (kth[1] > 0) {
#pragma unroll
    for (int e = 0; e < E; ++e) atomicAdd(&s.bins[256 + dist_bin(mx[1], z1[e])], 1u);
  }
  cluster_sync();
  uint32_t* gb = reinterpret_cast<uint32_t*>(s.candl);     // [2][256] cluster-wide bins
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    uint32_t g = 0;
    if (kth[r] > 0) {
      const uint32_t addr = smem_u32(&s.bins[r * 256 + tid]);
      for (uint32_t q = 0; q < c.nrank; ++q) g += dsmem_ld_u32(dsmem_addr(addr, q));
    }
    gb[r * 256 + tid] = g;
  }
  __syncthreads();
  if (warp < 2 && kth[warp & 1] > 0) {
    // smallest bin whose cumulative count reaches k: lane l covers bins 8l .. 8l+7
    const int r = warp;
    uint32_t cnt[8], sum = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) { cnt[i] = gb[r * 256 + 8 * lane + i]; sum += cnt[i]; }
    uint32_t incl = sum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += t;
    }
    const uint32_t excl = incl - sum, need = static_cast<uint32_t>(kth[r]);
    if (excl < need && need <= incl) {
      uint32_t run = excl;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        if (run < need && need <= run + cnt[i]) {
          c.sel[r * 2 + 0] = 8 * lane + i;
          c.sel[r * 2 + 1] = static_cast<int>(need - run);
        }
        run += cnt[i];
      }
    }
  }
  __syncthreads();           // also: gb has been consumed, candl may be overwritten
  int bstar[2], krem[2];
#pragma unroll
  for (int r = 0; r < 2; ++r) { bstar[r] = kth[r] > 0 ? c.sel[r * 2] : -1; krem[r] = kth[r] > 0 ? c.sel[r * 2 + 1] : 0; }
  if (kth[0] > 0) {
#pragma unroll
    for (int e = 0; e < E; ++e)
      if (dist_bin(mx[0], z0[e]) == bstar[0]) {
        const int pos = atomicAdd(&s.candn[0], 1);
        if (pos < kCandLocal) s.candl[pos] = z0[e];
      }
  }
  if (kth[1] > 0) {
#pragma unroll
    for (int e = 0; e < E; ++e)
      if (dist_bin(mx[1], z1[e]) == bstar[1]) {
        const int pos = atomicAdd(&s.candn[1], 1);
        if (pos < kCandLocal) s.candl[kCandLocal + pos] = z1[e];
      }
  }
  cluster_sync();
  // counts of every rank -> scratch [4 + r*16 + rank]
  int* cnts = s.candn + 4;
  if (tid < 2 * static_cast<int>(c.nrank)) {
    const int r = tid / c.nrank, q = tid % c.nrank;
    cnts[r * kMaxCluster + q] = static_cast<int>(dsmem_ld_u32(dsmem_addr(smem_u32(&s.candn[r]), q)));
  }
  __syncthreads();
  bool fits = true;
  int total[2] = {0, 0};
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    if (kth[r] <= 0) continue;
    for (uint32_t q = 0; q < c.nrank; ++q) {
      const int n = cnts[r * kMaxCluster + q];
      if (n > kCandLocal) fits = false;
      total[r] += n;
    }
    if (total[r] > kCandTotal) fits = false;
  }
  if (!fits) return false;
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    if (kth[r] <= 0) continue;
    int off = 0;
    for (uint32_t q = 0; q < c.nrank; ++q) {
      const int n = cnts[r * kMaxCluster + q];
      const uint32_t base = dsmem_addr(smem_u32(&s.candl[r * kCandLocal]), q);
      for (int i = tid; i < n; i += kThreads) s.all[r * kCandTotal + off + i] = dsmem_ld_f32(base + 4u * i);
      off += n;
    }
  }
  __syncthreads();
  // exact rank by counting: theta = v with  #(> v) < k' <= #(>= v)
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    if (kth[r] <= 0) continue;
    const float* a = s.all + r * kCandTotal;
    for (int i = tid; i < total[r]; i += kThreads) {
      const float v = a[i];
      int gt = 0, ge = 0;
      for (int t = 0; t < total[r]; ++t) {
        const float w = a[t];
        gt += (w > v);
        ge += (w >= v);
      }
      if (gt < krem[r] && krem[r] <= ge) reinterpret_cast<float*>(c.sel)[r] = v;
    }
  }
  __syncthreads();
#pragma unroll
  for (int r = 0; r < 2; ++r) theta[r] = kth[r] > 0 ? reinterpret_cast<float*>(c.sel)[r] : -INFINITY;
  __syncthreads();
  return true;
}

// Softmax numerators 2^((z - max) * log2 e) of the entries at or above theta, written once
// to shared memory (entries below theta and the padding beyond the row end become 0).
// Returns this thread's partial sum.
template <int E, int VN, bool HAS_THETA>
__device__ __forceinline__ float exp_store_regs(const float (&z)[E], float mx, float theta, float* __restrict__ dst) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int wb = warp * 32 * E + lane * VN;
  const float c2 = -mx * kLog2e;
  float sum = 0.f;
#pragma unroll
  for (int v = 0; v < E / VN; ++v) {
    float ev[VN];
#pragma unroll
    for (int e = 0; e < VN; ++e) {
      const float zz = z[v * VN + e];
      float x = ex2_approx(fmaf(zz, kLog2e, c2));
      if (HAS_THETA) x = (zz >= theta) ? x : 0.f;
      ev[e] = x;
      sum += x;
    }
    float4* d4 = reinterpret_cast<float4*>(dst + wb + v * 32 * VN);
#pragma unroll
    for (int e = 0; e < VN; e += 4) d4[e / 4] = make_float4(ev[e], ev[e + 1], ev[e + 2], ev[e + 3]);
  }
  return sum;
}

template <int E, int VN>
__device__ __forceinline__ void store_regs(const float (&z)[E], float* __restrict__ dst) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int wb = warp * 32 * E + lane * VN;
#pragma unroll
  for (int v = 0; v < E / VN; ++v) {
    float4* d4 = reinterpret_cast<float4*>(dst + wb + v * 32 * VN);
#pragma unroll
    for (int e = 0; e < VN; e += 4)
      d4[e / 4] = make_float4(z[v * VN + e], z[v * VN + e + 1], z[v * VN + e + 2], z[v * VN + e + 3]);
  }
}

}  // namespace lantern
