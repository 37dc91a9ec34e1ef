// Latent-neighbour table (Sec. 2.2 / Sec. 4: B_k = k nearest codebook entries; App. A.1:
// codebook C = {c_1..c_L}, c_i in R^d).  Exact squared-Euclidean k-NN of every row, ordered
// by (distance, index), self excluded.
//
// Exact brute-force kernel.  A CTA owns a tile of QT query rows and streams over all L
// candidate rows; distances are accumulated in double precision (sum of squared differences,
// so duplicate rows give distance exactly 0 and equal distances to third rows).  Selection is
// streaming: per query a float32 threshold tau (the k-th smallest rounded distance seen so
// far) filters candidates into a shared-memory buffer; when the buffer fills it is sorted and
// cut back to the entries <= the new tau (rounding to float32 is monotone, so nothing that can
// belong to the exact top k is ever dropped).  The survivors are re-ranked by their double
// distances.  If ties at tau overflow the buffer the query falls back to k rounds of an exact
// arg-min over all candidates.
#include "common.cuh"

namespace lantern {

constexpr int kKnnThreads = 256;
constexpr int kDC = 32;             // embedding dims staged per step

struct KnnArgs {
  const void* cb;
  int L, d, k, QT, CAP, q_double;
  int f32acc;        // filter distances accumulated in float32 with an error margin (small d)
  float margin;      // 1 + 3 (d + 2) 2^-24: the filter keeps everything within this factor of tau
  int32_t* nbr_idx;
  float* nbr_dist;
};

template <typename T> __device__ __forceinline__ float widen(T x);
template <> __device__ __forceinline__ float widen<float>(float x) { return x; }
template <> __device__ __forceinline__ float widen<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }

// in-place ascending bitonic sort of n (power of two) 64-bit keys in shared memory
__device__ __forceinline__ void bitonic_u64(unsigned long long* a, int n) {
  for (int size = 2; size <= n; size <<= 1) {
    for (int stride = size >> 1; stride > 0; stride >>= 1) {
      for (int i = threadIdx.x; i < (n >> 1); i += kKnnThreads) {
        int lo = 2 * i - (i & (stride - 1));
        int hi = lo + stride;
        bool up = (lo & size) == 0;
        unsigned long long x = a[lo], y = a[hi];
        if ((x > y) == up) { a[lo] = y; a[hi] = x; }
      }
      __syncthreads();
    }
  }
}

// ascending bitonic sort of n (power of two) (dist, idx) pairs
__device__ __forceinline__ void bitonic_pair(double* dv, int* iv, int n) {
  for (int size = 2; size <= n; size <<= 1) {
    for (int stride = size >> 1; stride > 0; stride >>= 1) {
      for (int i = threadIdx.x; i < (n >> 1); i += kKnnThreads) {
        int lo = 2 * i - (i & (stride - 1));
        int hi = lo + stride;
        bool up = (lo & size) == 0;
        double dx = dv[lo], dy = dv[hi];
        int ix = iv[lo], iy = iv[hi];
        bool gt = dx > dy || (dx == dy && ix > iy);
        if (gt == up) { dv[lo] = dy; dv[hi] = dx; iv[lo] = iy; iv[hi] = ix; }
      }
      __syncthreads();
    }
  }
}

template <int NT, int BAR>
__device__ __forceinline__ void knn_bar() {
  if (BAR == 0) __syncthreads();
  else asm volatile("bar.sync %0, %1;" ::"n"(BAR), "n"(NT) : "memory");
}

// Cut-back of one query's candidate buffer without sorting it.  Entries are 64-bit words whose
// upper half is a monotone 32-bit key of the filter distance.  A most-significant-digit radix
// select (4 passes of 8 bits, shared-memory histogram) finds the k-th smallest key; `limit_of`
// turns it into the largest key that may stay (k-th key plus the caller's error margin); the
// entries up to that limit are compacted through `tmp` (order is irrelevant: the final ranking
// sorts).  Returns the number kept; *kth_key_out receives the k-th smallest key.  n >= k.
// NT threads (threadIdx.x < NT) take part and meet at hardware barrier BAR (0 = the whole CTA).
template <int NT = kKnnThreads, int BAR = 0, typename F>
__device__ __forceinline__ int radix_cut(unsigned long long* bq, int n, int k, unsigned long long* tmp, uint32_t* hist,
                                         int* sel, F&& limit_of, uint32_t* limit_out) {
  const int tid = threadIdx.x, lane = tid & 31;
  uint32_t prefix = 0;
  int rem = k;
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    for (int i = tid; i < 256; i += NT) hist[i] = 0;
    knn_bar<NT, BAR>();
    for (int i = tid; i < n; i += NT) {
      const uint32_t key = static_cast<uint32_t>(bq[i] >> 32);
      if (pass == 0 || (key >> (shift + 8)) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1u);
    }
    knn_bar<NT, BAR>();
    if (tid < 32) {
      uint32_t c8[8], s = 0;
#pragma unroll
      for (int i = 0; i < 8; ++i) { c8[i] = hist[lane * 8 + i]; s += c8[i]; }
      uint32_t incl = s;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
      }
      const uint32_t before = incl - s;
      if (before < static_cast<uint32_t>(rem) && static_cast<uint32_t>(rem) <= incl) {     // exactly one lane
        uint32_t run = before;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          if (run < static_cast<uint32_t>(rem) && static_cast<uint32_t>(rem) <= run + c8[i]) {
            sel[0] = lane * 8 + i;
            sel[1] = rem - static_cast<int>(run);
          }
          run += c8[i];
        }
      }
    }
    knn_bar<NT, BAR>();
    prefix = (prefix << 8) | static_cast<uint32_t>(sel[0]);
    rem = sel[1];
    knn_bar<NT, BAR>();
  }
  const uint32_t limit = limit_of(prefix);          // prefix is now the k-th smallest key
  if (tid == 0) sel[2] = 0;
  knn_bar<NT, BAR>();
  for (int i0 = 0; i0 < n; i0 += NT) {
    const int i = i0 + tid;
    const unsigned long long e = i < n ? bq[i] : ~0ull;
    const bool keep = i < n && static_cast<uint32_t>(e >> 32) <= limit;
    const uint32_t m = __ballot_sync(0xffffffffu, keep);
    int pos0 = 0;
    if (lane == 0 && m) pos0 = atomicAdd(&sel[2], __popc(m));
    pos0 = __shfl_sync(0xffffffffu, pos0, 0);
    if (keep) tmp[pos0 + __popc(m & ((1u << lane) - 1u))] = e;
  }
  knn_bar<NT, BAR>();
  const int kept = sel[2];
  for (int i = tid; i < kept; i += NT) bq[i] = tmp[i];
  *limit_out = limit;
  knn_bar<NT, BAR>();
  return kept;
}

template <typename T>
__device__ __forceinline__ double exact_dist(const T* __restrict__ cb, int d, int i, int j) {
  const T* a = cb + static_cast<long long>(i) * d;
  const T* b = cb + static_cast<long long>(j) * d;
  double s = 0.0;
  for (int t = 0; t < d; ++t) {
    double diff = static_cast<double>(widen<T>(a[t])) - static_cast<double>(widen<T>(b[t]));
    s = fma(diff, diff, s);
  }
  return s;
}

// The same sum, in the same order, for a bfloat16 query row held in shared memory and a candidate
// row read from global memory with 16-byte loads (d a multiple of 8, both rows 16-byte aligned).
__device__ __forceinline__ double exact_dist_bf16x8(const __nv_bfloat16* a, const __nv_bfloat16* __restrict__ b, int d) {
  double s = 0.0;
  for (int t = 0; t < d; t += 8) {
    const uint4 av = *reinterpret_cast<const uint4*>(a + t);
    const uint4 bv = __ldg(reinterpret_cast<const uint4*>(b + t));
    const uint32_t aw[4] = {av.x, av.y, av.z, av.w}, bw[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const double d0 = static_cast<double>(__uint_as_float(aw[i] << 16)) - static_cast<double>(__uint_as_float(bw[i] << 16));
      s = fma(d0, d0, s);
      const double d1 = static_cast<double>(__uint_as_float(aw[i] & 0xffff0000u)) -
                        static_cast<double>(__uint_as_float(bw[i] & 0xffff0000u));
      s = fma(d1, d1, s);
    }
  }
  return s;
}

// Exact ranking of one query's surviving candidates (keys carry the candidate index in their
// low 32 bits): distances re-evaluated in double, sorted by (distance, index), first k written.
// With `overflow` the buffer is ignored and k rounds of an exact arg-min over all rows are run.
// `q_row`, if given, is the query's bfloat16 row in shared memory (d a multiple of 8): the distances
// then come from exact_dist_bf16x8.
template <typename T>
__device__ __forceinline__ void rank_query(const T* __restrict__ cb, int L, int d, int k, int qi,
                                           const unsigned long long* bq, int n_in, bool overflow, int CAP,
                                           double* sortd, int* sorti, double* redd, int* redi,
                                           int32_t* out_i, float* out_d, const __nv_bfloat16* q_row = nullptr) {
  const int tid = threadIdx.x;
    if (!overflow) {
    const int n = min(n_in, CAP);
          for (int i = tid; i < CAP; i += kKnnThreads) {
      if (i < n) {
        int j = static_cast<int>(bq[i] & 0xffffffffu);
        sorti[i] = j;
        if (sizeof(T) == 2 && q_row)
          sortd[i] = exact_dist_bf16x8(q_row, reinterpret_cast<const __nv_bfloat16*>(cb) + static_cast<long long>(j) * d, d);
        else
          sortd[i] = exact_dist<T>(cb, d, qi, j);
      } else {
        sorti[i] = 0x7fffffff;
        sortd[i] = INFINITY;
      }
    }
    __syncthreads();
    bitonic_pair(sortd, sorti, CAP);
    for (int r = tid; r < k; r += kKnnThreads) {
      out_i[r] = sorti[r];
      if (out_d) out_d[r] = static_cast<float>(sortd[r]);
    }
    __syncthreads();
  } else {
    // exact fallback: k rounds of arg-min over (distance, index) greater than the last pick
    double pd = -1.0;
    int pj = -1;
    for (int r = 0; r < k; ++r) {
      double bd = INFINITY;
      int bj = 0x7fffffff;
      for (int j = tid; j < L; j += kKnnThreads) {
        if (j == qi) continue;
        double dj = exact_dist<T>(cb, d, qi, j);
        bool after = dj > pd || (dj == pd && j > pj);
        if (after && (dj < bd || (dj == bd && j < bj))) { bd = dj; bj = j; }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        double od = __shfl_xor_sync(0xffffffffu, bd, o);
        int oj = __shfl_xor_sync(0xffffffffu, bj, o);
        if (od < bd || (od == bd && oj < bj)) { bd = od; bj = oj; }
      }
      if ((tid & 31) == 0) { redd[tid >> 5] = bd; redi[tid >> 5] = bj; }
      __syncthreads();
      bd = redd[0]; bj = redi[0];
      for (int w = 1; w < kKnnThreads / 32; ++w)
        if (redd[w] < bd || (redd[w] == bd && redi[w] < bj)) { bd = redd[w]; bj = redi[w]; }
      __syncthreads();
      pd = bd; pj = bj;
      if (tid == 0) {
        out_i[r] = bj;
        if (out_d) out_d[r] = static_cast<float>(bd);
      }
    }
  }
}

template <typename T>
__global__ void __launch_bounds__(kKnnThreads) knn_kernel(const KnnArgs a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int QT = a.QT, CAP = a.CAP, d = a.d, L = a.L, k = a.k;
  const T* cb = static_cast<const T*>(a.cb);
  // layout: buf[QT][CAP] u64 | sortd[CAP] f64 | sorti[CAP] i32 | cand[256][kDC+1] f32 | tau[QT] f32 |
  //         cnt[QT] i32 | ovf[QT] i32 | redd[8] f64 | redi[8] i32 | queries
  unsigned long long* buf = reinterpret_cast<unsigned long long*>(smem_raw);
  double* sortd = reinterpret_cast<double*>(buf + static_cast<size_t>(QT) * CAP);
  double* redd = sortd + CAP;
  int* sorti = reinterpret_cast<int*>(redd + 8);
  float* cand = reinterpret_cast<float*>(sorti + CAP);
  float* tau = cand + kKnnThreads * (kDC + 1);
  int* cnt = reinterpret_cast<int*>(tau + QT);
  int* ovf = cnt + QT;
  int* redi = ovf + QT;
  uint32_t* hist = reinterpret_cast<uint32_t*>(redi + 8);       // [256] radix-select histogram
  int* sel = reinterpret_cast<int*>(hist + 256);               // [4]
  unsigned char* qraw = reinterpret_cast<unsigned char*>(sel + 4);
  qraw += (16 - (reinterpret_cast<uintptr_t>(qraw) & 15)) & 15;
  double* qd = reinterpret_cast<double*>(qraw);
  float* qf = reinterpret_cast<float*>(qraw);

  const int tid = threadIdx.x;
  const int q0 = blockIdx.x * QT;
  const int nq = min(QT, L - q0);

  const int dpad = (d + 7) & ~7;
  if (a.f32acc) {
    for (int i = tid; i < QT * dpad; i += kKnnThreads) {
      int q = i / dpad, t = i - q * dpad;
      qf[i] = (q < nq && t < d) ? widen<T>(cb[static_cast<long long>(q0 + q) * d + t]) : 0.f;
    }
  } else {
    for (int i = tid; i < QT * d; i += kKnnThreads) {
      int q = i / d, t = i - q * d;
      float v = (q < nq) ? widen<T>(cb[static_cast<long long>(q0 + q) * d + t]) : 0.f;
      if (a.q_double) qd[i] = static_cast<double>(v); else qf[i] = v;
    }
  }
  if (tid < QT) { tau[tid] = INFINITY; cnt[tid] = 0; ovf[tid] = 0; }
  __syncthreads();

  constexpr int MAXQT = 8;
  // d <= 8 (one chunk of dimensions): the candidate row of the next tile is fetched while this
  // tile is being processed
  float cnext[8];
  const bool prefetch = a.f32acc && d <= 8;
  auto fetch_row = [&](int row, float (&out)[8]) {
#pragma unroll
    for (int t = 0; t < 8; ++t) out[t] = (row < L && t < d) ? widen<T>(cb[static_cast<long long>(row) * d + t]) : 0.f;
  };
  if (prefetch) fetch_row(tid, cnext);
  for (int base = 0; base < L; base += kKnnThreads) {
    double acc[MAXQT];
#pragma unroll
    for (int q = 0; q < MAXQT; ++q) acc[q] = 0.0;
    const int ncand = min(kKnnThreads, L - base);
    if (a.f32acc) {
      // Filter distances in float32: every thread reads its candidate's row straight from global
      // memory, eight dimensions at a time, against the query rows in shared memory.  The relative
      // error of such a sum is below (d + 2) 2^-24, so with the margin applied to tau nothing
      // that can belong to the exact top k is dropped; exact duplicates still give 0.
      float accf[MAXQT];
#pragma unroll
      for (int q = 0; q < MAXQT; ++q) accf[q] = 0.f;
      for (int db = 0; db < d; db += 8) {
        float cv[8];
        if (prefetch) {
#pragma unroll
          for (int t = 0; t < 8; ++t) cv[t] = cnext[t];
          fetch_row(base + kKnnThreads + tid, cnext);
        } else {
#pragma unroll
          for (int t = 0; t < 8; ++t)
            cv[t] = (tid < ncand && db + t < d) ? widen<T>(cb[static_cast<long long>(base + tid) * d + db + t]) : 0.f;
        }
#pragma unroll
        for (int q = 0; q < MAXQT; ++q) {
          if (q < QT) {
            const float4 qa = *reinterpret_cast<const float4*>(qf + q * dpad + db);
            const float4 qb = *reinterpret_cast<const float4*>(qf + q * dpad + db + 4);
            const float qv[8] = {qa.x, qa.y, qa.z, qa.w, qb.x, qb.y, qb.z, qb.w};
#pragma unroll
            for (int t = 0; t < 8; ++t) {
              const float diff = qv[t] - cv[t];
              accf[q] = fmaf(diff, diff, accf[q]);
            }
          }
        }
      }
#pragma unroll
      for (int q = 0; q < MAXQT; ++q) acc[q] = static_cast<double>(accf[q]);
    } else
    for (int db = 0; db < d; db += kDC) {
      const int dc = min(kDC, d - db);
      __syncthreads();
      for (int i = tid; i < ncand * dc; i += kKnnThreads) {
        int r = i / dc, t = i - r * dc;
        cand[r * (kDC + 1) + t] = widen<T>(cb[static_cast<long long>(base + r) * d + db + t]);
      }
      __syncthreads();
      if (tid < ncand) {
        for (int t = 0; t < dc; ++t) {
          const double cv = static_cast<double>(cand[tid * (kDC + 1) + t]);
#pragma unroll
          for (int q = 0; q < MAXQT; ++q) {
            if (q < QT) {
              double qv = a.q_double ? qd[q * d + db + t] : static_cast<double>(qf[q * d + db + t]);
              double diff = qv - cv;
              acc[q] = fma(diff, diff, acc[q]);
            }
          }
        }
      }
    }
    // filter into the per-query buffers
    if (tid < ncand) {
      const int j = base + tid;
#pragma unroll
      for (int q = 0; q < MAXQT; ++q) {
        if (q < nq && j != q0 + q) {
          float f = static_cast<float>(acc[q]);
          if (f <= tau[q]) {
            int pos = atomicAdd(&cnt[q], 1);
            if (pos < CAP) buf[static_cast<size_t>(q) * CAP + pos] =
                (static_cast<unsigned long long>(__float_as_uint(f)) << 32) | static_cast<unsigned>(j);
          }
        }
      }
    }
    __syncthreads();
    // cut back buffers that might overflow during the next tile
    for (int q = 0; q < nq; ++q) {
      int n = cnt[q];
      if (n <= CAP - kKnnThreads || ovf[q]) continue;     // uniform: cnt/ovf are shared
      unsigned long long* bq = buf + static_cast<size_t>(q) * CAP;
      // keep everything up to the k-th smallest filter distance (times the margin in float32 mode)
      uint32_t limit;
      const float margin = a.f32acc ? a.margin : 1.0f;
      const int m = radix_cut(bq, min(n, CAP), k, reinterpret_cast<unsigned long long*>(sortd), hist, sel,
                              [&](uint32_t kth) { return __float_as_uint(__fmul_ru(__uint_as_float(kth), margin)); }, &limit);
      if (tid == 0) {
        tau[q] = __uint_as_float(limit);      // (non-negative floats order as their bits)
        cnt[q] = m;
        if (m > CAP - kKnnThreads) ovf[q] = 1;      // ties at tau fill the buffer
      }
      __syncthreads();
    }
  }

  // final ranking per query
  for (int q = 0; q < nq; ++q) {
    const int qi = q0 + q;
    rank_query<T>(cb, L, d, k, qi, buf + static_cast<size_t>(q) * CAP, cnt[q], ovf[q] != 0, CAP, sortd, sorti, redd, redi,
                  a.nbr_idx + static_cast<long long>(qi) * k,
                  a.nbr_dist ? a.nbr_dist + static_cast<long long>(qi) * k : nullptr);
  }
}

}  // namespace lantern

#include "knn_tc.cuh"
#include "knn_t5.cuh"

using namespace lantern;

// The tensor-core path is taken for bfloat16 codebooks with d a multiple of 16 in [32, 256] and
// k small enough for its per-query buffers.
static bool use_tensor_path(lantern_dtype dt, int L, int d, int k) {
  return dt == LANTERN_BF16 && d % 16 == 0 && d >= 32 && d <= kTcMaxD && k <= 320 && L >= 64;
}

// bfloat16 codebooks of at least this many rows, d a multiple of 8 up to 256, take the tcgen05 kernel
// (tiles of 128 queries per CTA); smaller ones would leave most SMs without a tile and stay on the
// mma.sync kernel (or, for d it does not serve, on the brute-force kernel).
#ifndef LANTERN_T5_MIN_L
#define LANTERN_T5_MIN_L 8192
#endif
constexpr int kT5GridCap = 160;          // CTAs the workspace is sized for (one per SM)
static bool use_t5_path(lantern_dtype dt, int L, int d, int k) {
  return dt == LANTERN_BF16 && d % 8 == 0 && d >= 8 && d <= 256 && k <= kT5MaxK && L >= LANTERN_T5_MIN_L;
}
static size_t norms_bytes(int L) { return ((static_cast<size_t>(L) + 64) * sizeof(float) + 255) / 256 * 256; }
static size_t t5_cta_bytes(int k) { return static_cast<size_t>(kT5Q) * knn_t5_cap(k) * 8; }

extern "C" size_t lantern_build_neighbors_workspace(lantern_dtype dt, int32_t L, int32_t d, int32_t k) {
  if (L < 2 || d < 1 || k < 1) return 0;
  // squared norms of all rows and their maximum (tensor-core paths), plus the per-CTA candidate
  // lists of the tcgen05 kernel; the brute-force kernel keeps all of its state on chip
  if (!use_t5_path(dt, L, d, k)) return use_tensor_path(dt, L, d, k) ? norms_bytes(L) : 0;
  const int nqt = (L + 63) / 64;                   // the kernel may run tiles of 64 queries (see the launch)
  return norms_bytes(L) + static_cast<size_t>(nqt < kT5GridCap ? nqt : kT5GridCap) * t5_cta_bytes(k);
}

extern "C" lantern_status lantern_build_neighbors(const void* codebook, lantern_dtype dt, int32_t L, int32_t d,
                                                  int32_t k, int32_t* nbr_idx, float* nbr_dist, void* workspace,
                                                  size_t workspace_bytes, void* stream) {
  if (!codebook || !nbr_idx) return LANTERN_ERR_INVALID_ARG;
  if (dt != LANTERN_F32 && dt != LANTERN_BF16) return LANTERN_ERR_INVALID_ARG;
  if (L < 2 || d < 1 || k < 1 || k > L - 1) return LANTERN_ERR_INVALID_ARG;
  if (k > 1024 || d > 4096) return LANTERN_ERR_UNSUPPORTED;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (use_t5_path(dt, L, d, k) || use_tensor_path(dt, L, d, k)) {
    const size_t need = lantern_build_neighbors_workspace(dt, L, d, k);
    if (!workspace || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) % 256)) return LANTERN_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(codebook) % 16) return LANTERN_ERR_INVALID_ARG;
    float* nrm = static_cast<float*>(workspace);
    if (cudaMemsetAsync(nrm + L, 0, sizeof(float), st) != cudaSuccess) return LANTERN_ERR_CUDA;
    knn_norms_kernel<<<(L * 32 + 255) / 256, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(codebook), L, d, nrm);
    if (cudaGetLastError() != cudaSuccess) return LANTERN_ERR_CUDA;
    if (use_t5_path(dt, L, d, k)) {
      KnnT5Args fa;
      fa.cb = static_cast<const __nv_bfloat16*>(codebook); fa.nrm = nrm; fa.L = L; fa.d = d; fa.k = k;
      fa.CAP = knn_t5_cap(k);
      fa.lists = reinterpret_cast<unsigned long long*>(static_cast<unsigned char*>(workspace) + norms_bytes(L));
      fa.nbr_idx = nbr_idx; fa.nbr_dist = nbr_dist;
      int dev = 0, sms = 0;
      if (cudaGetDevice(&dev) != cudaSuccess ||
          cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
        return LANTERN_ERR_CUDA;
      const long long afford = static_cast<long long>((workspace_bytes - norms_bytes(L)) / t5_cta_bytes(k));
      // tiles of 128 queries, or of 64 (half of the tensor-memory lanes idle: the contraction is a small part
      // of the kernel) when that is what it takes to give every SM a tile
      fa.qtile = (L + kT5Q - 1) / kT5Q * 2 <= sms ? kT5Q / 2 : kT5Q;
      int grid = (L + fa.qtile - 1) / fa.qtile;
      if (grid > sms) grid = sms;
      if (grid > afford) grid = static_cast<int>(afford);
      if (grid < 1) return LANTERN_ERR_WORKSPACE;
      const size_t fsm = knn_t5_smem(d, fa.CAP);
      if (cudaFuncSetAttribute(knn_t5_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(fsm)) != cudaSuccess)
        return LANTERN_ERR_CUDA;
      knn_t5_kernel<<<grid, kT5Threads, fsm, st>>>(fa);
      return cudaGetLastError() == cudaSuccess ? LANTERN_OK : LANTERN_ERR_CUDA;
    }
    KnnTcArgs ta;
    ta.cb = static_cast<const __nv_bfloat16*>(codebook); ta.nrm = nrm; ta.L = L; ta.d = d; ta.k = k;
    ta.CAP = 256;
    while (ta.CAP < k + 192) ta.CAP *= 2;
    ta.nbr_idx = nbr_idx; ta.nbr_dist = nbr_dist;
    const int ld = d + kTcPad;
    const size_t tsm = static_cast<size_t>(kTcQT) * ta.CAP * 8 + static_cast<size_t>(kTcQT) * ld * 2 +
                       static_cast<size_t>(2) * kTcCT * ld * 2 + 2 * kTcCT * 4 + 5 * kTcQT * 4 + 64 +
                       260 * 4 + static_cast<size_t>(ta.CAP) * 8;
    if (cudaFuncSetAttribute(knn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(tsm)) != cudaSuccess)
      return LANTERN_ERR_CUDA;
    knn_tc_kernel<<<(L + kTcQT - 1) / kTcQT, kKnnThreads, tsm, st>>>(ta);
    return cudaGetLastError() == cudaSuccess ? LANTERN_OK : LANTERN_ERR_CUDA;
  }
  KnnArgs a;
  a.cb = codebook; a.L = L; a.d = d; a.k = k; a.nbr_idx = nbr_idx; a.nbr_dist = nbr_dist;
  int cap = 512;
  while (cap < k + 2 * kKnnThreads) cap *= 2;
  a.CAP = cap;
  a.QT = cap <= 1024 ? 8 : 4;
  auto smem_for = [&](int qt, int qdouble) {
    return static_cast<size_t>(qt) * cap * 8 + static_cast<size_t>(cap) * 12 + 8 * 12 +
           static_cast<size_t>(kKnnThreads) * (kDC + 1) * 4 + static_cast<size_t>(qt) * 12 + 16 + 260 * 4 +
           static_cast<size_t>(qt) * ((d + 7) & ~7) * (qdouble ? 8 : 4);
  };
  a.f32acc = d <= 64 ? 1 : 0;
  a.margin = 1.0f + 3.0f * static_cast<float>(d + 2) * 5.9604644775390625e-8f;
  a.q_double = (!a.f32acc && smem_for(a.QT, 1) <= 160 * 1024) ? 1 : 0;
  while (a.QT > 1 && smem_for(a.QT, a.q_double) > 220 * 1024) a.QT /= 2;
  size_t smem = smem_for(a.QT, a.q_double);
  if (smem > 227 * 1024) return LANTERN_ERR_UNSUPPORTED;
  const int grid = (L + a.QT - 1) / a.QT;
  cudaError_t e;
  if (dt == LANTERN_F32) {
    e = cudaFuncSetAttribute(knn_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e == cudaSuccess) { knn_kernel<float><<<grid, kKnnThreads, smem, st>>>(a); e = cudaGetLastError(); }
  } else {
    e = cudaFuncSetAttribute(knn_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e == cudaSuccess) { knn_kernel<__nv_bfloat16><<<grid, kKnnThreads, smem, st>>>(a); e = cudaGetLastError(); }
  }
  return e == cudaSuccess ? LANTERN_OK : LANTERN_ERR_CUDA;
}
