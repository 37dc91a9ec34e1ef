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

}  // namespace lantern
