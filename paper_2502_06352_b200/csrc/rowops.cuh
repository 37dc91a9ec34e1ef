// Element-level building blocks shared by the verify and the draft-sampler kernels: 16-byte
// vector loads of float32 / bfloat16 logits and the float32 definition of the pre-softmax value.
#pragma once

#include "common.cuh"

namespace lantern {

template <typename T> struct Vec;
template <> struct Vec<float> {
  static constexpr int N = 4;
  using V = float4;
  __device__ static __forceinline__ void unpack(const V& v, float (&f)[4]) {
    f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w;
  }
  __device__ static __forceinline__ void unpack_raw(const uint4& v, float (&f)[4]) {
    f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y); f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
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
  __device__ static __forceinline__ void unpack_raw(const uint4& v, float (&f)[8]) { unpack(v, f); }
  __device__ static __forceinline__ float widen(__nv_bfloat16 x) { return __bfloat162float(x); }
};

// Pre-softmax value (App. B "Models"): guidance with one fused multiply-add, then 1/tau.
// Explicit intrinsics keep the compiler from contracting or reassociating.
template <bool CFG>
__device__ __forceinline__ float combine(float c, float u, float g, float inv_tau) {
  if (CFG) return __fmul_rn(__fmaf_rn(g, __fsub_rn(c, u), u), inv_tau);
  return __fmul_rn(c, inv_tau);
}

constexpr float kLog2e = 1.4426950408889634f;

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ void vflag(int32_t* status, int bit) {
  if (status) atomicOr(status, bit);
}

// ---- histogram bins of the top-k locator: a monotone, coarse position of an entry below the
// row maximum (128 bins per binade of d = max - z, 16 binades: d in [2^-9, 2^7), clamped)
constexpr int kBins = 2048;
constexpr int kBinLog = 7;
constexpr int kBinShift = 23 - kBinLog;
constexpr int kBinBase = (127 - 9) << kBinLog;
__device__ __forceinline__ int dist_bin(float mx, float z) {
  const float d = mx - z;
  // max(min(bits - base, last), 0) in one instruction
  return __viaddmin_s32_relu(static_cast<int>(__float_as_uint(d) >> kBinShift), -kBinBase, kBins - 1);
}
// bit patterns of d that fall into bin b: [bin_lo_bits(b), bin_hi_bits(b)] (the end bins are open)
__device__ __forceinline__ uint32_t bin_lo_bits(int b) {
  return b == 0 ? 0u : static_cast<uint32_t>(b + kBinBase) << kBinShift;
}
__device__ __forceinline__ uint32_t bin_hi_bits(int b) {
  return b == kBins - 1 ? 0xffffffffu : (static_cast<uint32_t>(b + kBinBase + 1) << kBinShift) - 1u;
}

// ---- bounded wait on an mbarrier phase; false when the limit was reached
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t mbar, uint32_t phase) {
  for (int it = 0; it < (1 << 22); ++it) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(mbar), "r"(phase) : "memory");
    if (ok) return true;
  }
  return false;
}

// 16-byte streaming load (read once: no L1 allocation)
__device__ __forceinline__ uint4 ldg_stream_u128(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}

}  // namespace lantern
