// Draft sampling for rows that are truncated to their top-k entries (Sec. 2.1; App. B "Models"),
// vocabularies of up to 16384 tokens.  Only the k (plus ties) survivors of a row can be drawn, so
// the row is compacted to a (token, z) list first, with the same routine as in the verify kernel,
// and the Gumbel keys, the softmax denominator and the s selection rounds touch ~k entries instead
// of V.  A CTA of 512 threads handles one parent; two CTAs share an SM.  A parent whose row does
// not fit the fixed buffers (massive ties) gets the marker kRedoToken in its first child's token
// slot; the dense kernel then draws exactly those parents.
#pragma once

#include "verify_sparse.cuh"

namespace lantern {
namespace sparse {

constexpr int kRedoToken = -2;
constexpr int kPerThread = kCap / ST;     // list entries per thread
constexpr float kKeyErr = 2e-5f;          // bound on |float32 key - exact key| (|key| < 64)

__host__ __device__ constexpr size_t sampler_smem_bytes(int e) {
  return static_cast<size_t>(ST) * e * 4 + 3 * kCap * 4 + kBins * 4 + kWords * 4 + kCand * 4 + 2 * SW * 2 * 4 +
         SW * 4 + kMisc * 4 + 2 * 2 * SW * 4 + (8 + 8 + 8 + 32 + 4) * 4;
}

__device__ __forceinline__ bool key_better(float ka, int ia, float kb, int ib) {   // a beats b
  return ka > kb || (ka == kb && ia < ib);
}
__device__ __forceinline__ void warp_key_best(float& k, int& i) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ok = __shfl_xor_sync(0xffffffffu, k, o);
    const int oi = __shfl_xor_sync(0xffffffffu, i, o);
    if (key_better(ok, oi, k, i)) { k = ok; i = oi; }
  }
}

template <typename T, bool CFG, int E>
__global__ void __launch_bounds__(ST, 2) sample_sparse_kernel(const SampleArgs a) {
  grid_dependency_sync();
  extern __shared__ __align__(16) unsigned char smem_raw[];
  Smem s;
  s.Z = reinterpret_cast<float*>(smem_raw);
  s.ltok[0] = reinterpret_cast<int*>(s.Z + ST * E);
  s.lval[0] = reinterpret_cast<float*>(s.ltok[0] + kCap);
  float* keys = s.lval[0] + kCap;                 // [kCap]
  s.ltok[1] = nullptr;
  s.lval[1] = nullptr;
  s.bins = reinterpret_cast<uint32_t*>(keys + kCap);
  s.bm[0] = s.bins + kBins;
  s.bm[1] = nullptr;
  s.rk = nullptr;
  s.cand = reinterpret_cast<float*>(s.bm[0] + kWords);
  Ctx c;
  c.red = s.cand + kCand;
  c.last_red = c.red;
  c.parity = 0;
  s.wtot = reinterpret_cast<uint32_t*>(c.red + 2 * SW * 2);
  s.misc = reinterpret_cast<int*>(s.wtot + SW);
  float* pk = reinterpret_cast<float*>(s.misc + kMisc);    // [2][2*SW] warps' best key and token, two buffers
  float* wkey = pk + 2 * 2 * SW;                           // [8] keys of the rounds' winners
  int* wtok = reinterpret_cast<int*>(wkey + 8);            // [8] their tokens (-1: none), [8] their list positions
  int* wpos = wtok + 8;
  int* cpos = wpos + 8;                                    // [32] list positions of the entries ranked exactly
  int* ccnt = cpos + 32;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int idx = blockIdx.x;
  const int b = idx % a.B;
  const int n = a.order[a.order_begin + idx / a.B];
  const int fc = a.first_child[n], nc = a.n_child[n];
  const int len = min(a.V, ST * E);
  const long long row_off = static_cast<long long>(b) * a.seq_stride + static_cast<long long>(n) * a.row_stride;
  const long long out_b = static_cast<long long>(b) * a.N;

  const bool masked = a.allow_lo > 0 || a.allow_hi < a.V;
  const T* cond = static_cast<const T*>(a.dc) + row_off;
  const T* uncond = CFG ? static_cast<const T*>(a.du) + row_off : nullptr;
  for (int i = tid; i < kBins; i += ST) s.bins[i] = 0;
  s.bm[0][tid] = 0;
  float mx[2];
  mx[0] = load_row<T, CFG, E>(cond, uncond, a.g, a.inv_tau, len, a.allow_lo, a.allow_hi, masked, s.Z);
  mx[1] = -INFINITY;
  block_reduce2<true>(c, mx);
  int n_list = 0;
  float theta = INFINITY;
  bool ok = mx[0] != -INFINITY;
  if (ok) ok = compact_topk<E, true>(s, 0, mx[0], a.topk_d, n_list, theta);
  if (!ok) {
    if (tid == 0) a.tokens[out_b + fc] = kRedoToken;
    return;
  }

  // ---- keys z + G, G = -log(-log U), of the survivors; softmax denominator
  const uint32_t row_id = static_cast<uint32_t>(out_b + n);
  const float* gum = a.gumbel ? a.gumbel + static_cast<long long>(row_id) * a.V : nullptr;
  const float c0 = -mx[0] * kLog2e;
  float sm[2] = {0.f, 0.f};
  float bk = -INFINITY;
  int bi = 0x7fffffff, bpos = -1;
#pragma unroll
  for (int m = 0; m < kPerThread; ++m) {
    const int i = tid + m * ST;
    if (i >= n_list) break;
    const int t = s.ltok[0][i];
    const float z = s.lval[0][i];
    float key = -INFINITY;
    if (z >= theta && z != -INFINITY) {
      float u;
      if (gum) {
        u = __ldcs(gum + t);
      } else {
        const Philox4 r = philox_stream(a.seed, a.step, row_id, kStreamGumbel, static_cast<uint32_t>(t >> 2));
        const uint32_t w = (t & 3) == 0 ? r.x : ((t & 3) == 1 ? r.y : ((t & 3) == 2 ? r.z : r.w));
        u = uniform_open(w);
      }
      key = z - __logf(-logf(u));
      sm[0] += ex2_approx(fmaf(z, kLog2e, c0));
    }
    keys[i] = key;
    if (key_better(key, t, bk, bi) && key != -INFINITY) { bk = key; bi = t; bpos = i; }
  }
  block_reduce2<false>(c, sm);
  const float inv_sum = sm[0] > 0.f ? 1.f / sm[0] : 0.f;

  // ---- s rounds: block-wide best key (ties: lower token); its owner retires it and rescans
  for (int round = 0; round < nc; ++round) {
    float wk = bk;
    int wi = bi;
    warp_key_best(wk, wi);
    float* buf = pk + (round & 1) * 2 * SW;
    if (lane == 0) { buf[warp] = wk; buf[SW + warp] = __int_as_float(wi); }
    __syncthreads();
    float ck = lane < SW ? buf[lane] : -INFINITY;
    int ci = lane < SW ? __float_as_int(buf[SW + lane]) : 0x7fffffff;
    warp_key_best(ck, ci);
    const bool valid = ck != -INFINITY;
    if (tid == 0) { wkey[round] = ck; wtok[round] = valid ? ci : -1; }
    if (valid && ci == bi) {                    // exactly one thread owns the winner
      wpos[round] = bpos;
      a.tokens[out_b + fc + round] = ci;
      if (a.draft_prob)
        a.draft_prob[out_b + fc + round] = ex2_approx(fmaf(s.lval[0][bpos], kLog2e, c0)) * inv_sum;
      keys[bpos] = -INFINITY;
      bk = -INFINITY;
      bi = 0x7fffffff;
      bpos = -1;
#pragma unroll
      for (int m = 0; m < kPerThread; ++m) {
        const int i = tid + m * ST;
        if (i >= n_list) break;
        const float key = keys[i];
        const int t = s.ltok[0][i];
        if (key != -INFINITY && key_better(key, t, bk, bi)) { bk = key; bi = t; bpos = i; }
      }
    }
    if (!valid && tid == 0) {
      a.tokens[out_b + fc + round] = -1;
      if (a.draft_prob) a.draft_prob[out_b + fc + round] = 0.f;
    }
  }

  // ---- exact order.  The rounds ranked float32 keys (error below kKeyErr each).  Where two of
  // the chosen keys, or a chosen key and one left out, are closer than 2 * kKeyErr, the entries
  // involved are ranked again by keys evaluated in double precision (ties: lower token id).
  __syncthreads();
  int nv = 0;
  while (nv < nc && wtok[nv] >= 0) ++nv;
  if (nv == 0) return;
  const float k_last = wkey[nv - 1];
  bool close = false;
  for (int r = 1; r < nv; ++r) close |= wkey[r - 1] - wkey[r] <= 2.f * kKeyErr;
  bool mine = false;
#pragma unroll
  for (int m = 0; m < kPerThread; ++m) {
    const int i = tid + m * ST;
    if (i >= n_list) break;
    mine |= keys[i] != -INFINITY && keys[i] >= k_last - 2.f * kKeyErr;
  }
  if (!__syncthreads_or((mine || close) ? 1 : 0)) return;
  if (tid < nv) { cpos[tid] = wpos[tid]; }
  if (tid == 0) *ccnt = nv;
  __syncthreads();
#pragma unroll
  for (int m = 0; m < kPerThread; ++m) {
    const int i = tid + m * ST;
    if (i >= n_list) break;
    if (keys[i] != -INFINITY && keys[i] >= k_last - 2.f * kKeyErr) {
      const int at = atomicAdd(ccnt, 1);
      if (at < 32) cpos[at] = i;
    }
  }
  __syncthreads();
  if (warp == 0) {
    const int ncand = *ccnt;
    if (ncand > 32) {                             // more near-ties than one warp ranks
      if (lane == 0) vflag(a.status, LANTERN_DEV_KEY_TIES);
      return;
    }
    double key = -INFINITY;
    int t = 0x7fffffff;
    float z = 0.f;
    if (lane < ncand) {
      const int i = cpos[lane];
      t = s.ltok[0][i];
      z = s.lval[0][i];
      float u;
      if (gum) {
        u = __ldcs(gum + t);
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

}  // namespace sparse
}  // namespace lantern
