// Tensor-core path of the latent-neighbour table for bfloat16 codebooks whose embedding dimension
// makes the distance matrix a real dense contraction (d a multiple of 16, 32 <= d <= 256).
//
//   approximate distance  f(i,j) = |c_i|^2 + |c_j|^2 - 2 <c_i, c_j>      (float32)
// with the inner products from bf16 tensor-core MMAs (products exact, float32 accumulation).
// |f - D| <= eps_i for the exact squared distance D, eps_i = (d+8) * 2^-21 * (|c_i|^2 + max_j |c_j|^2)
// (accumulation of d exact products, the two norms, two final roundings, factor 2 of slack).
// If tau is the k-th smallest f seen for a query, every true neighbour has f <= tau + 2 eps, so
// the streaming filter keeps candidates with f <= tau + 2 eps and nothing else; the survivors are
// then re-ranked exactly (double precision, ties by index) like in the brute-force kernel.
//
// A CTA owns 32 query rows (kept in shared memory for the whole kernel) and streams all rows
// as candidate tiles of 64 through a cp.async double buffer; 8 warps each own a 16 x 16 block of
// the 32 x 64 tile (mma.sync m16n8k16).  Rows are padded by 16 bytes in shared memory, which
// makes the 32-bit fragment loads bank-conflict free.
#pragma once

#include "common.cuh"

namespace lantern {

constexpr int kTcQT = 32;          // query rows per CTA
constexpr int kTcCT = 64;          // candidate rows per tile
constexpr int kTcPad = 8;          // bf16 elements of padding per shared-memory row
constexpr int kTcMaxD = 256;

struct KnnTcArgs {
  const __nv_bfloat16* cb;
  const float* nrm;        // [L] squared norms, nrm[L] = their maximum
  int L, d, k, CAP;
  int32_t* nbr_idx;
  float* nbr_dist;
};

// squared norms (float32) and their maximum
__global__ void knn_norms_kernel(const __nv_bfloat16* __restrict__ cb, int L, int d, float* __restrict__ nrm) {
  const int row = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (row >= L) return;
  float s = 0.f;
  for (int t = lane; t < d; t += 32) {
    const float v = __bfloat162float(cb[static_cast<long long>(row) * d + t]);
    s = fmaf(v, v, s);
  }
  s = warp_sum(s);
  if (lane == 0) {
    nrm[row] = s;
    atomicMax(reinterpret_cast<unsigned int*>(nrm + L), __float_as_uint(s));   // s >= 0: bit order = value order
  }
}

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// four 8 x 8 bf16 matrices from shared memory: lane l supplies the address of row l % 8 of matrix l / 8
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], const __nv_bfloat16* row_ptr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(smem_u32(row_ptr)) : "memory");
}

// stage rows [row0, row0 + rows) of the codebook into padded shared-memory rows (zero beyond L)
__device__ __forceinline__ void stage_rows(const __nv_bfloat16* __restrict__ cb, int L, int d, int row0, int rows,
                                           __nv_bfloat16* dst) {
  const int chunks = d / 8;                   // 16-byte chunks per row
  const int ld = d + kTcPad;
  // thread i starts at chunk i and advances by the thread count: (row, chunk) follow by addition
  int r = static_cast<int>(threadIdx.x) / chunks, ch = static_cast<int>(threadIdx.x) - r * chunks;
  const int dr = kKnnThreads / chunks, dch = kKnnThreads - dr * chunks;
  while (r < rows) {
    const int row = row0 + r;
    const bool in = row < L;
    const __nv_bfloat16* src = cb + static_cast<long long>(in ? row : 0) * d + ch * 8;
    cp_async16(smem_u32(dst + r * ld + ch * 8), src, in ? 16u : 0u);
    r += dr;
    ch += dch;
    if (ch >= chunks) { ch -= chunks; ++r; }
  }
}

// squared norms of the candidate rows [row0, row0 + kTcCT) into shared memory (zero beyond L)
__device__ __forceinline__ void stage_norms(const float* __restrict__ nrm, int L, int row0, float* dst) {
  if (threadIdx.x < kTcCT) {
    const int j = row0 + threadIdx.x;
    const bool in = j < L;
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(smem_u32(dst + threadIdx.x)),
                 "l"(nrm + (in ? j : 0)), "r"(in ? 4u : 0u) : "memory");
  }
}


__global__ void __launch_bounds__(kKnnThreads) knn_tc_kernel(const KnnTcArgs a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int d = a.d, L = a.L, k = a.k, CAP = a.CAP, ld = d + kTcPad;
  const __nv_bfloat16* cb = a.cb;
  unsigned long long* buf = reinterpret_cast<unsigned long long*>(smem_raw);            // [QT][CAP]
  __nv_bfloat16* As = reinterpret_cast<__nv_bfloat16*>(buf + static_cast<size_t>(kTcQT) * CAP);   // [QT][ld]
  __nv_bfloat16* Bs = As + kTcQT * ld;                                                  // [2][CT][ld]
  float* ncs = reinterpret_cast<float*>(Bs + 2 * kTcCT * ld);                           // [2][CT]
  float* nq = ncs + 2 * kTcCT;                                                          // [QT]
  float* thr = nq + kTcQT;
  float* eps2 = thr + kTcQT;
  int* cnt = reinterpret_cast<int*>(eps2 + kTcQT);
  int* ovf = cnt + kTcQT;
  uint32_t* hist = reinterpret_cast<uint32_t*>(ovf + kTcQT);                            // [256] radix-select histogram
  int* sel = reinterpret_cast<int*>(hist + 256);                                        // [4]
  unsigned long long* cut_tmp = reinterpret_cast<unsigned long long*>(sel + 4);         // [CAP]
  // after the main loop the tile buffers are reused by the exact ranking
  double* sortd = reinterpret_cast<double*>(Bs);
  double* redd = sortd + CAP;
  int* sorti = reinterpret_cast<int*>(redd + 8);
  int* redi = sorti + CAP;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int q0 = blockIdx.x * kTcQT;
  const int ntiles = (L + kTcCT - 1) / kTcCT;
  const float nmax = a.nrm[L];

  stage_rows(cb, L, d, q0, kTcQT, As);
  stage_rows(cb, L, d, 0, kTcCT, Bs);
  stage_norms(a.nrm, L, 0, ncs);
  cp_async_commit();
  if (tid < kTcQT) {
    const float n = q0 + tid < L ? a.nrm[q0 + tid] : 0.f;
    nq[tid] = n;
    eps2[tid] = 2.f * static_cast<float>(d + 8) * 4.76837158203125e-7f * (n + nmax);     // 2 * eps, 2^-21
    thr[tid] = INFINITY;
    cnt[tid] = 0;
    ovf[tid] = 0;
  }

  const int wq = warp & 1, wc = warp >> 1;
  const int r0 = wq * 16 + (lane >> 2), r1 = r0 + 8;
  const int kc = 2 * (lane & 3);

  for (int t = 0; t < ntiles; ++t) {
    const int cur = t & 1;
    if (t + 1 < ntiles) {
      stage_rows(cb, L, d, (t + 1) * kTcCT, kTcCT, Bs + (cur ^ 1) * kTcCT * ld);
      stage_norms(a.nrm, L, (t + 1) * kTcCT, ncs + (cur ^ 1) * kTcCT);
      cp_async_commit();
      cp_async_wait<1>();
    } else {
      cp_async_wait<0>();
    }
    __syncthreads();
    const __nv_bfloat16* Bt = Bs + cur * kTcCT * ld;
    float acc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
    // fragments by ldmatrix: A = query rows (matrices: rows 0-7 / 8-15 x k 0-7 / 8-15), B = candidate
    // rows of two 8-wide column tiles (matrices: tile 0 k 0-7, tile 0 k 8-15, tile 1 k 0-7, tile 1 k 8-15)
    const int mi = lane >> 3, mr = lane & 7;
    const __nv_bfloat16* a_ptr = As + (wq * 16 + (mi & 1) * 8 + mr) * ld + (mi >> 1) * 8;
    const __nv_bfloat16* b_ptr = Bt + (wc * 16 + (mi >> 1) * 8 + mr) * ld + (mi & 1) * 8;
    for (int kb = 0; kb < d; kb += 16) {
      uint32_t af[4], bf[4];
      ldmatrix_x4(af, a_ptr + kb);
      ldmatrix_x4(bf, b_ptr + kb);
      mma_bf16_16816(acc[0], af, bf[0], bf[1]);
      mma_bf16_16816(acc[1], af, bf[2], bf[3]);
    }
    // epilogue: approximate distances, filter, append
    const float thr0 = thr[r0], thr1 = thr[r1], nq0 = nq[r0], nq1 = nq[r1];
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int col = wc * 16 + nt * 8 + kc + (e & 1);
        const int r = (e < 2) ? r0 : r1;
        const int j = t * kTcCT + col;
        const float f = fmaf(-2.f, acc[nt][e], ((e < 2) ? nq0 : nq1) + ncs[cur * kTcCT + col]);
        if (j < L && q0 + r < L && j != q0 + r && f <= ((e < 2) ? thr0 : thr1)) {
          const int pos = atomicAdd(&cnt[r], 1);
          if (pos < CAP)
            buf[static_cast<size_t>(r) * CAP + pos] =
                (static_cast<unsigned long long>(float_key(f)) << 32) | static_cast<unsigned>(j);
        }
      }
    }
    __syncthreads();                                   // this tile's appends are counted
    // cut back buffers that might overflow during the next tile (usually none: one vote)
    const bool near_full = tid < kTcQT && cnt[tid] > CAP - kTcCT && !ovf[tid];
    if (!__syncthreads_or(near_full)) continue;
    for (int q = 0; q < kTcQT; ++q) {
      const int n = cnt[q];
      if (n <= CAP - kTcCT || ovf[q]) continue;            // uniform: shared values
      unsigned long long* bq = buf + static_cast<size_t>(q) * CAP;
      // keep everything within the error margin of the k-th smallest approximate distance
      uint32_t limit;
      const float e2 = eps2[q];
      const int kept = radix_cut(bq, min(n, CAP), k, cut_tmp, hist, sel,
                                 [&](uint32_t kth) { return float_key(key_float(kth) + e2); }, &limit);
      if (tid == 0) {
        thr[q] = key_float(limit);
        cnt[q] = kept;
        if (kept > CAP - kTcCT) ovf[q] = 1;                 // too many rows within the error margin
      }
      __syncthreads();
    }
  }
  __syncthreads();
  for (int q = 0; q < kTcQT; ++q) {
    const int qi = q0 + q;
    if (qi >= L) break;
    rank_query<__nv_bfloat16>(cb, L, d, k, qi, buf + static_cast<size_t>(q) * CAP, cnt[q], ovf[q] != 0, CAP, sortd, sorti,
                              redd, redi, a.nbr_idx + static_cast<long long>(qi) * k,
                              a.nbr_dist ? a.nbr_dist + static_cast<long long>(qi) * k : nullptr, As + q * ld);
  }
}

}  // namespace lantern
