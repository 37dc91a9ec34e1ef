// Blackwell tensor path of the latent-neighbour table (Sec. 2.2 / Sec. 4: B_k; App. A.1: the
// codebook) for bfloat16 codebooks with d a multiple of 8 in [8, 256]: the distance contraction on
// the fifth-generation tensor cores (tcgen05.mma, bf16 x bf16 -> float32 accumulators in tensor
// memory), the selection fused behind it.  Rows are zero-padded in shared memory to a multiple of
// 16 elements (the K extent of one MMA), which changes no inner product.
//
//   approximate distance  f(i,j) = |c_i|^2 + |c_j|^2 - 2 <c_i, c_j>   (float32),  |f - D| <= eps_i
// as in knn_tc.cuh; a query keeps every candidate with f <= tau + 2 eps (tau: an upper bound of the
// k-th smallest f at its last cut-back), so no true neighbour is ever dropped, and ranks the
// survivors exactly (double precision, ties by index) at the end.  f is formed as
// fl(g + |c_i|^2), g = fl(|c_j|^2 - 2 <c_i, c_j>): the same two roundings as in knn_tc.cuh.
//
// One persistent CTA of 256 threads per SM; a CTA takes tiles of 128 queries (tensor-memory lane =
// query) and streams all rows past them in tiles of 128 candidates (tensor-memory column =
// candidate):
//   warps 5-7  load operand tiles with 16-byte cp.async into the K-major core-matrix layout the
//              tensor core reads without swizzling (a core matrix = 8 rows x 16 bytes, contiguous),
//              two candidate stages in flight;
//   warp 4     one thread issues d/16 tcgen05.mma per tile into one of two 128-column accumulators
//              and commits to the mbarriers that free the stage and publish the accumulator;
//   warps 0-3  thread t owns query t: it reads its lane of the accumulator with tcgen05.ld, forms f,
//              and appends the few candidates under its threshold to its own list in global memory
//              (no atomics); a list that fills up is cut back by its warp (radix select on a copy in
//              shared memory), so the four warps never wait for one another.
// After the last candidate tile the eight warps rank the 128 queries exactly, one query per warp at
// a time.  Every wait on an mbarrier is bounded; a wait that runs out raises an abort flag that all
// roles poll, the CTA frees its tensor memory and returns, and the rows it had not finished are
// written as -1.
#pragma once

#include "knn_tc.cuh"

namespace lantern {

constexpr int kT5Q = 128;           // queries per CTA tile (tensor-memory lanes)
constexpr int kT5C = 128;           // candidates per tile (tensor-memory columns per accumulator)
constexpr int kT5Stages = 2;        // candidate tiles in flight in shared memory
constexpr int kT5Threads = 256;
constexpr int kT5Loaders = 96;      // warps 5-7
constexpr int kT5Sort = 512;        // exact ranking: candidates per query (power of two)
constexpr int kT5MaxK = 320;

struct KnnT5Args {
  const __nv_bfloat16* cb;
  const float* nrm;                 // [L] squared norms, nrm[L] = their maximum
  unsigned long long* lists;        // [gridDim.x][kT5Q][CAP] candidate lists (key << 32 | index)
  int L, d, k, CAP;
  int qtile;                        // queries a CTA tile really holds: 128, or 64 (the other lanes idle) when 128 would leave SMs without a tile
  int32_t* nbr_idx;
  float* nbr_dist;
};

// list capacity: room for one tile of appends above the cut-back level, which itself leaves the
// larger of k and 192 entries of slack above k
__host__ __device__ constexpr int knn_t5_dpad(int d) { return (d + 15) / 16 * 16; }     // K extent in shared memory
__host__ __device__ constexpr int knn_t5_cap(int k) { return (k + kT5C + (k > 192 ? k : 192) + 63) / 64 * 64; }

// bytes of one warp's slot in the final ranking: staged list, histogram, (distance, index) pairs,
// the query row in double precision
__host__ __device__ constexpr size_t knn_t5_slot(int cap, int d) {
  return static_cast<size_t>(cap) * 8 + 256 * 4 + static_cast<size_t>(kT5Sort) * 12 + static_cast<size_t>(d) * 8;
}
// the candidate stages and the final ranking share one region
__host__ __device__ constexpr size_t knn_t5_region(int d, int cap) {
  const size_t stages = static_cast<size_t>(kT5Stages) * kT5C * knn_t5_dpad(d) * 2, rank = 8 * knn_t5_slot(cap, d);
  return stages > rank ? stages : rank;
}
__host__ __device__ constexpr size_t knn_t5_smem(int d, int cap) {
  return static_cast<size_t>(kT5Q) * knn_t5_dpad(d) * 2 + knn_t5_region(d, cap)   // query tile; stages / ranking
         + 4 * kT5C * 4                                               // candidate norms, 4 tiles deep
         + kT5Q * 4 * 2                                               // 2 eps, list counts
         + 4 * static_cast<size_t>(cap) * 8 + 4 * 256 * 4             // per-warp staging and histogram of a cut
         + 16 * 8 + 8 * 8 + 24 * 4;                                   // mbarriers, arg-min scratch, misc
}

__device__ __forceinline__ uint64_t t5_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  // shared-memory matrix descriptor, no swizzle: start address, leading (K) and stride (M/N) byte
  // offsets between core matrices, all in units of 16 bytes; descriptor version 1
  return static_cast<uint64_t>((saddr & 0x3FFFFu) >> 4) | (static_cast<uint64_t>((lbo_bytes >> 4) & 0x3FFFu) << 16) |
         (static_cast<uint64_t>((sbo_bytes >> 4) & 0x3FFFu) << 32) | (static_cast<uint64_t>(1) << 46);
}

// bounded wait of one thread on an mbarrier phase that also gives up when another role has raised
// `abort`: non-blocking polls (test_wait) with a short sleep between them, so the bound is about a
// second and a waiting thread leaves the shared-memory pipe to the working warps
__device__ __forceinline__ bool t5_wait(uint32_t mbar, uint32_t parity, volatile int* abort) {
  for (int it = 0; it < (1 << 24); ++it) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(mbar), "r"(parity) : "memory");
    if (ok) return true;
    if (it >= 4) __nanosleep(40);
    if ((it & 1023) == 1023 && *abort) return false;
  }
  *abort = 1;
  return false;
}
// the same for a whole warp: lane 0 polls, the result is shared (__shfl_sync orders memory among the lanes)
__device__ __forceinline__ bool t5_wait_warp(uint32_t mbar, uint32_t parity, volatile int* abort) {
  int ok = 1;
  if ((threadIdx.x & 31) == 0) ok = t5_wait(mbar, parity, abort) ? 1 : 0;
  return __shfl_sync(0xffffffffu, ok, 0) != 0;
}
__device__ __forceinline__ void t5_arrive(uint32_t mbar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(mbar) : "memory");
}

// One operand tile (rows [row0, row0 + 128) of the codebook, zero beyond L and beyond d) into the
// core-matrix layout [dpad/8 chunks][16 row groups][8 rows][16 bytes].  A warp step covers 8 rows x 4 chunks: the
// 8 rows of a chunk are one contiguous core matrix (conflict-free), each row reads 64 contiguous
// bytes.  A warp walks along the rows of its row groups, so addresses advance by additions only.
__device__ __forceinline__ void t5_load_tile(const __nv_bfloat16* __restrict__ cb, int L, int d, int row0,
                                             unsigned char* dst, int ltid) {      // L: rows at or beyond it read as zero
  const int lane = ltid & 31, lw = ltid >> 5;
  const int r = lane & 7, c = lane >> 3;                          // row in the group, chunk in the quad
  const int nch = d >> 3, pch = knn_t5_dpad(d) >> 3;               // 16-byte chunks per row: real, padded
  for (int rg = lw; rg < 16; rg += kT5Loaders / 32) {
    const int grow = row0 + rg * 8 + r;
    const bool in = grow < L;
    const __nv_bfloat16* src = cb + static_cast<long long>(in ? grow : 0) * d + c * 8;
    uint32_t sdst = smem_u32(dst) + static_cast<uint32_t>((c * 16 + rg) * 128 + r * 16);
    for (int kc = c; kc < pch; kc += 4) {
      const bool real = in && kc < nch;
      cp_async16(sdst, real ? src : cb, real ? 16u : 0u);
      src += 32;
      sdst += 4u * 16u * 128u;
    }
  }
}

// Cut-back of one list by one warp (the radix select of knn.cu on warp scale).  Lists in global
// memory hold (float bits of f) << 32 | index.  The n entries of `src` are copied to `st` (shared
// memory) with f turned into its monotone 32-bit key.  An upper bound of the k-th smallest key is
// then found by histogram passes of up to 8 bits over key - min, starting at the highest bit in
// which the keys differ (distances of one list share their leading bits: passes over those would
// put every entry into one bin).  The passes stop when the bin that holds the k-th key has at most
// SLACK entries (or bit 0 is reached); the bound is the upper edge of that bin, so at most SLACK
// entries more than with the exact k-th key get through, which keeps the superset property.  The
// entries whose key is at most limit_of(bound) are written to `dst` in their old order: back to
// `src` as float bits (TO_RAW), or to `st` as keys.  Returns the number kept.  n >= k >= 1.
template <bool TO_RAW, int SLACK, typename F>
__device__ __forceinline__ int t5_warp_cut(const unsigned long long* src, int n, int k, unsigned long long* st,
                                           uint32_t* hist, unsigned long long* dst, F&& limit_of, uint32_t* limit_out) {
  const int lane = threadIdx.x & 31;
  __syncwarp();                                               // the owner's appends are visible to the warp
  uint32_t kmin = 0xffffffffu, kmax = 0u;
#pragma unroll 8
  for (int i = lane; i < n; i += 32) {
    const unsigned long long e = src[i];
    const uint32_t key = float_key(__uint_as_float(static_cast<uint32_t>(e >> 32)));
    st[i] = (static_cast<unsigned long long>(key) << 32) | (e & 0xffffffffull);
    kmin = min(kmin, key);
    kmax = max(kmax, key);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    kmin = min(kmin, __shfl_xor_sync(0xffffffffu, kmin, o));
    kmax = max(kmax, __shfl_xor_sync(0xffffffffu, kmax, o));
  }
  int hi = 32 - __clz(kmax - kmin);                           // key - kmin < 2^hi
  uint32_t prefix = 0;                                        // (k-th key - kmin) >> hi, known so far
  int rem = k;
  while (hi > 0) {
    const int lo = hi > 8 ? hi - 8 : 0;
    const uint32_t mask = (1u << (hi - lo)) - 1u;
#pragma unroll
    for (int i = 0; i < 8; ++i) hist[lane + 32 * i] = 0;
    __syncwarp();
#pragma unroll 4
    for (int i = lane; i < n; i += 32) {
      const uint32_t rel = static_cast<uint32_t>(st[i] >> 32) - kmin;
      if (hi == 32 || (rel >> hi) == prefix) atomicAdd(&hist[(rel >> lo) & mask], 1u);
    }
    __syncwarp();
    uint32_t c8[8], sum = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) { c8[i] = hist[lane * 8 + i]; sum += c8[i]; }
    uint32_t incl = sum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += t;
    }
    const uint32_t before = incl - sum, want = static_cast<uint32_t>(rem);
    const bool mine = before < want && want <= incl;          // exactly one lane
    int bin = 0, nrem = 0, pop = 0;
    if (mine) {
      uint32_t run = before;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        if (run < want && want <= run + c8[i]) { bin = lane * 8 + i; nrem = static_cast<int>(want - run); pop = static_cast<int>(c8[i]); }
        run += c8[i];
      }
    }
    const int owner = (__ffs(__ballot_sync(0xffffffffu, mine)) - 1) & 31;
    bin = __shfl_sync(0xffffffffu, bin, owner);
    rem = __shfl_sync(0xffffffffu, nrem, owner);
    pop = __shfl_sync(0xffffffffu, pop, owner);
    prefix = (prefix << (hi - lo)) | static_cast<uint32_t>(bin);
    hi = lo;
    __syncwarp();
    if (pop <= SLACK) break;
  }
  // keys whose (key - kmin) >> hi equals prefix: the k-th smallest is among them
  const unsigned long long edge = static_cast<unsigned long long>(kmin) + ((static_cast<unsigned long long>(prefix) + 1ull) << hi) - 1ull;
  const uint32_t limit = limit_of(edge < kmax ? static_cast<uint32_t>(edge) : kmax);
  int pos = 0;
  for (int i0 = 0; i0 < n; i0 += 32) {
    const int i = i0 + lane;
    const unsigned long long e = i < n ? st[i] : ~0ull;
    const bool keep = i < n && static_cast<uint32_t>(e >> 32) <= limit;
    const uint32_t m = __ballot_sync(0xffffffffu, keep);      // every lane has read its entry before slots <= i are rewritten
    if (keep)
      dst[pos + __popc(m & ((1u << lane) - 1u))] =
          TO_RAW ? (static_cast<unsigned long long>(__float_as_uint(key_float(static_cast<uint32_t>(e >> 32)))) << 32) | (e & 0xffffffffull)
                 : e;
    pos += __popc(m);
    __syncwarp();
  }
  *limit_out = limit;
  return pos;
}

// bfloat16 (low 16 bits of b16) to double without the conversion unit: for normal numbers the double's
// high word is the sign, the exponent rebiased by 1023 - 127 and the 7 mantissa bits, all by integer
// operations; zeros, subnormals, infinities and NaNs take the converting instruction.  Exact either way.
__device__ __forceinline__ double t5_bf16_to_double(uint32_t b16) {
  if (((b16 >> 7) & 0xffu) - 1u < 254u)
    return __hiloint2double(static_cast<int>(((b16 & 0x8000u) << 16) | (((b16 & 0x7fffu) << 13) + (896u << 20))), 0);
  return static_cast<double>(__uint_as_float(b16 << 16));
}

// Exact squared distances between the query row `qd` (doubles in shared memory) and the candidates
// st[base + 32 u + lane], u < kT5Chains, each the sum of exact_dist_bf16x8 term by term in the same
// order.  A double-precision FMA has a long latency and each sum is one dependent chain, so a lane
// runs the chains of its candidates side by side.  Entries in [n, p2) are padded with +inf.
constexpr int kT5Chains = 7;
__device__ __forceinline__ void t5_exact_block(const double* qd, const __nv_bfloat16* __restrict__ cb, int d,
                                               const unsigned long long* st, int n, int p2, int base, int nch,
                                               unsigned long long* sortd, int* sorti) {
  const int lane = threadIdx.x & 31;
  // this call covers entries [base, base + 32 nch); nu of its chains hold at least one candidate
  const int nu = min(nch, (min(n, p2) - base + 31) / 32);
  const __nv_bfloat16* row[kT5Chains];
  int idx[kT5Chains];
  double acc[kT5Chains];
#pragma unroll
  for (int u = 0; u < kT5Chains; ++u) {
    const int i = base + 32 * u + lane;
    idx[u] = (u < nch && i < n) ? static_cast<int>(st[i] & 0xffffffffu) : -1;
    row[u] = cb + static_cast<long long>(idx[u] < 0 ? 0 : idx[u]) * d;
    acc[u] = 0.0;
  }
  for (int t = 0; t < d; t += 8) {
    uint4 bv[kT5Chains];
#pragma unroll
    for (int u = 0; u < kT5Chains; ++u)
      if (u < nu) bv[u] = __ldg(reinterpret_cast<const uint4*>(row[u] + t));
    double q[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) q[i] = qd[t + i];
#pragma unroll
    for (int u = 0; u < kT5Chains; ++u) {
      if (u < nu) {
        const uint32_t bw[4] = {bv[u].x, bv[u].y, bv[u].z, bv[u].w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const double d0 = q[2 * i] - t5_bf16_to_double(bw[i] & 0xffffu);
          acc[u] = fma(d0, d0, acc[u]);
          const double d1 = q[2 * i + 1] - t5_bf16_to_double(bw[i] >> 16);
          acc[u] = fma(d1, d1, acc[u]);
        }
      }
    }
  }
#pragma unroll
  for (int u = 0; u < kT5Chains; ++u) {
    const int i = base + 32 * u + lane;
    if (u < nch && i < p2) {
      sorti[i] = idx[u] < 0 ? 0x7fffffff : idx[u];
      sortd[i] = idx[u] < 0 ? 0x7ff0000000000000ull : static_cast<unsigned long long>(__double_as_longlong(acc[u]));
    }
  }
}

// ascending bitonic sort of n (power of two) (distance, index) pairs by one warp.  Distances are
// non-negative doubles (or +inf padding), whose bit patterns order like their values: the compares
// run on the integer pipe.
__device__ __forceinline__ void t5_warp_sort(unsigned long long* dv, int* iv, int n) {
  const int lane = threadIdx.x & 31;
  for (int size = 2; size <= n; size <<= 1) {
    for (int stride = size >> 1; stride > 0; stride >>= 1) {
#pragma unroll 4
      for (int i = lane; i < (n >> 1); i += 32) {
        const int lo = 2 * i - (i & (stride - 1)), hi = lo + stride;
        const bool up = (lo & size) == 0;
        const unsigned long long dx = dv[lo], dy = dv[hi];
        const int ix = iv[lo], iy = iv[hi];
        const bool gt = dx > dy || (dx == dy && ix > iy);
        if (gt == up) { dv[lo] = dy; dv[hi] = dx; iv[lo] = iy; iv[hi] = ix; }
      }
      __syncwarp();
    }
  }
}

__global__ void __launch_bounds__(kT5Threads, 1) knn_t5_kernel(const KnnT5Args a) {
  extern __shared__ __align__(128) unsigned char t5_smem[];
  const int d = a.d, L = a.L, k = a.k, CAP = a.CAP, dp = knn_t5_dpad(a.d);
  const __nv_bfloat16* cb = a.cb;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  unsigned char* As = t5_smem;                                        // [d/8][16][8][16 B]
  unsigned char* Bs = As + static_cast<size_t>(kT5Q) * dp * 2;         // [stages][d/8][16][8][16 B] | ranking slots
  const size_t tile_bytes = static_cast<size_t>(kT5C) * dp * 2;
  float* ncs = reinterpret_cast<float*>(Bs + knn_t5_region(d, CAP));  // [4][kT5C] candidate norms
  float* eps2s = ncs + 4 * kT5C;                                      // [kT5Q]
  int* cnts = reinterpret_cast<int*>(eps2s + kT5Q);                   // [kT5Q] list lengths (-1: overflow, -2: exact fallback)
  unsigned long long* cut_st = reinterpret_cast<unsigned long long*>(cnts + kT5Q);     // [4][CAP]
  uint32_t* cut_hist = reinterpret_cast<uint32_t*>(cut_st + 4 * static_cast<size_t>(CAP));   // [4][256]
  uint64_t* bars = reinterpret_cast<uint64_t*>(cut_hist + 4 * 256);   // full[2] empty[2] tfull[2] tempty[2] afull aempty | redd[8]
  int* misc = reinterpret_cast<int*>(bars + 24);                      // [0] tensor-memory base, [1] abort, [16..23] redi

  const uint32_t bar0 = smem_u32(bars);
  auto full = [&](uint32_t s2) { return bar0 + 8u * s2; };
  auto empty = [&](uint32_t s2) { return bar0 + 8u * (2 + s2); };
  auto tfull = [&](uint32_t b) { return bar0 + 8u * (4 + b); };
  auto tempty = [&](uint32_t b) { return bar0 + 8u * (6 + b); };
  const uint32_t afull = bar0 + 8u * 8, aempty = bar0 + 8u * 9;
  volatile int* abort = misc + 1;

  if (tid == 0) {
    auto init = [&](uint32_t b, int count) { asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(b), "r"(count) : "memory"); };
    for (uint32_t s2 = 0; s2 < 2; ++s2) { init(full(s2), kT5Loaders); init(empty(s2), 1); init(tfull(s2), 1); init(tempty(s2), kT5Q); }
    init(afull, kT5Loaders);
    init(aempty, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    misc[1] = 0;
  }
  if (warp == 4) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(misc)), "r"(2 * kT5C) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tbase = static_cast<uint32_t>(misc[0]);

  const int QT = a.qtile;
  const int nqt = (L + QT - 1) / QT;                // query tiles
  const int nct = (L + kT5C - 1) / kT5C;            // candidate tiles per query tile
  const float nmax = a.nrm[L];
  unsigned long long* my_lists = a.lists + static_cast<size_t>(blockIdx.x) * kT5Q * CAP;
  bool dead = false;                                // a wait ran out (here or in another role): work is skipped, barriers are kept
  uint32_t tiles_done = 0, qtiles_done = 0;         // per role: candidate tiles / query tiles handled so far

  for (int qt = blockIdx.x; qt < nqt; qt += gridDim.x) {
    const int q0 = qt * QT;
    if (warp >= 5) {
      // ---------------------------------------------------------------- loaders (warps 5-7)
      const int ltid = tid - 160;
      uint32_t pending;                              // barrier of the copy group committed last
      if (!dead) dead = !t5_wait_warp(aempty, (qtiles_done & 1u) ^ 1u, abort);
      if (!dead) t5_load_tile(cb, min(L, q0 + QT), d, q0, As, ltid);
      cp_async_commit();
      pending = afull;
      for (int t = 0; t < nct; ++t) {
        const uint32_t s2 = tiles_done & 1u;
        if (!dead) dead = !t5_wait_warp(empty(s2), ((tiles_done >> 1) & 1u) ^ 1u, abort);
        if (!dead) {
          t5_load_tile(cb, L, d, t * kT5C, Bs + s2 * tile_bytes, ltid);
          for (int i = ltid; i < kT5C; i += kT5Loaders) {
            const int j = t * kT5C + i;
            const bool in = j < L;
            asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(smem_u32(ncs + (tiles_done & 3u) * kT5C + i)),
                         "l"(a.nrm + (in ? j : 0)), "r"(in ? 4u : 0u) : "memory");
          }
        }
        cp_async_commit();
        cp_async_wait<1>();                          // the group committed before this one has landed: publish it
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        t5_arrive(pending);
        pending = full(s2);
        ++tiles_done;
      }
      cp_async_wait<0>();
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      t5_arrive(pending);
      ++qtiles_done;
    } else if (warp == 4) {
      // ---------------------------------------------------------------- tensor-core issue (one thread)
      if (lane == 0) {
        const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(kT5C >> 3) << 17) |
                               (static_cast<uint32_t>(kT5Q >> 4) << 24);     // f32 += bf16 x bf16, K-major, N, M
        const uint32_t lbo = 16u * 128u, sbo = 128u;
        if (!dead) dead = !t5_wait(afull, qtiles_done & 1u, abort);
        for (int t = 0; t < nct; ++t) {
          const uint32_t s2 = tiles_done & 1u, par = (tiles_done >> 1) & 1u;
          if (!dead) dead = !t5_wait(full(s2), par, abort);
          if (!dead) dead = !t5_wait(tempty(s2), par ^ 1u, abort);
          if (!dead) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t a0 = smem_u32(As), b0 = smem_u32(Bs + s2 * tile_bytes);
            for (int kk = 0; kk < dp / 16; ++kk) {
              const uint64_t da = t5_desc(a0 + kk * 2u * lbo, lbo, sbo);
              const uint64_t db = t5_desc(b0 + kk * 2u * lbo, lbo, sbo);
              const uint32_t acc = kk > 0 ? 1u : 0u;
              asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %4, 0;\n\t"
                           "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                           ::"r"(tbase + s2 * kT5C), "l"(da), "l"(db), "r"(idesc), "r"(acc) : "memory");
            }
            asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(empty(s2)) : "memory");
            asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(tfull(s2)) : "memory");
          }
          ++tiles_done;
        }
        if (!dead)
          asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(aempty) : "memory");
        ++qtiles_done;
      }
    } else {
      // ---------------------------------------------------------------- selection (warps 0-3): thread = query
      const int qi = q0 + tid;
      const bool active = qi < L && tid < QT;
      const float nq = active ? a.nrm[qi] : 0.f;
      const float e2 = 2.f * static_cast<float>(d + 8) * 4.76837158203125e-7f * (nq + nmax);     // 2 eps, 2^-21
      eps2s[tid] = e2;
      unsigned long long* lst = my_lists + static_cast<size_t>(tid) * CAP;
      unsigned long long* st_w = cut_st + static_cast<size_t>(warp) * CAP;
      uint32_t* hist_w = cut_hist + warp * 256;
      // the filter compares g with thr_g >= thr - |q|^2, the slack covering the roundings of f = fl(g + |q|^2)
      // and of the subtraction, so it passes a superset of {f <= thr}
      float thr_g = INFINITY;
      uint32_t woff = 0;                             // byte offset of the next free entry of the own list
      int cnt = 0;
      bool ovf = false;
      for (int t = 0; t < nct; ++t) {
        const uint32_t b = tiles_done & 1u;
        const bool special = t == nct - 1 || t == q0 / kT5C;
        if (!dead) dead = !t5_wait_warp(tfull(b), (tiles_done >> 1) & 1u, abort);   // warp-uniform
        if (!dead) {
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const float* nc = ncs + (tiles_done & 3u) * kT5C;
#pragma unroll 1
          for (int c0 = 0; c0 < kT5C; c0 += 32) {
            uint32_t r[32];
            const uint32_t taddr = tbase + (static_cast<uint32_t>(warp * 32) << 16) + b * kT5C + c0;
            asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                         "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
                         : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                           "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                           "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                           "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                         : "r"(taddr) : "memory");
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            if (active && !ovf) {
              const int cbase = t * kT5C + c0;
              if (!special) {
                // per candidate: one FMA, one compare, and a store and pointer step that are predicated
                // in the instruction stream (a branch here would diverge on nearly every candidate
                // while the thresholds are still loose)
#pragma unroll
                for (int j4 = 0; j4 < 32; j4 += 4) {
                  const float4 n4 = *reinterpret_cast<const float4*>(nc + c0 + j4);
                  const float nn[4] = {n4.x, n4.y, n4.z, n4.w};
#pragma unroll
                  for (int jj = 0; jj < 4; ++jj) {
                    const float g = fmaf(-2.f, __uint_as_float(r[j4 + jj]), nn[jj]);
                    asm volatile("{\n\t.reg .pred p;\n\t.reg .u64 a;\n\t.reg .f32 f;\n\tsetp.le.f32 p, %1, %2;\n\t"
                                 "cvt.u64.u32 a, %0;\n\tadd.u64 a, a, %5;\n\t"
                                 "@p add.rn.f32 f, %1, %4;\n\t"
                                 "@p st.global.v2.b32 [a], {%3, f};\n\t"
                                 "@p add.u32 %0, %0, 8;\n\t}"
                                 : "+r"(woff) : "f"(g), "f"(thr_g), "r"(cbase + j4 + jj), "f"(nq), "l"(lst) : "memory");
                  }
                }
              } else {
                // the ragged last candidate tile and the tile that holds the queries themselves
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                  const float g = fmaf(-2.f, __uint_as_float(r[j]), nc[c0 + j]);
                  const int cand = cbase + j;
                  if (g <= thr_g && cand < L && cand != qi) {
                    lst[woff >> 3] = (static_cast<unsigned long long>(__float_as_uint(g + nq)) << 32) | static_cast<unsigned>(cand);
                    woff += 8;
                  }
                }
              }
            }
          }
          asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
          t5_arrive(tempty(b));
        }
        ++tiles_done;
        cnt = static_cast<int>(woff >> 3);
        // a list that could overflow during the next tile is cut back by its warp
        uint32_t m = __ballot_sync(0xffffffffu, active && !ovf && !dead && cnt > CAP - kT5C);
        while (m) {
          const int src = __ffs(m) - 1;
          m &= m - 1;
          const int nq_l = __shfl_sync(0xffffffffu, cnt, src);
          const float eq = __shfl_sync(0xffffffffu, e2, src);
          unsigned long long* lq = my_lists + static_cast<size_t>(warp * 32 + src) * CAP;
          uint32_t limit;
          const int kept = t5_warp_cut<true, 32>(lq, nq_l, k, st_w, hist_w, lq,
                                       [&](uint32_t kth) { return float_key(key_float(kth) + eq); }, &limit);
          if (lane == src) {
            cnt = kept;
            woff = static_cast<uint32_t>(kept) * 8u;
            const float thr = key_float(limit);
            thr_g = (thr - nq) + 4.76837158203125e-7f * (fabsf(thr) + nq);
            if (kept > CAP - kT5C) ovf = true;                  // too many rows within the error margin
          }
        }
      }
      cnts[tid] = ovf ? -1 : cnt;
    }
    __syncthreads();                                 // every role is through this query tile; the stages are free
    dead = dead || *abort != 0;
    // ---------------------------------------------------------------- exact ranking: one query per warp at a time
    {
      unsigned char* slot = Bs + static_cast<size_t>(warp) * knn_t5_slot(CAP, d);
      unsigned long long* st = reinterpret_cast<unsigned long long*>(slot);
      uint32_t* hist = reinterpret_cast<uint32_t*>(st + CAP);
      unsigned long long* sortd = reinterpret_cast<unsigned long long*>(hist + 256);   // bit patterns of doubles >= 0
      int* sorti = reinterpret_cast<int*>(sortd + kT5Sort);
      double* qd = reinterpret_cast<double*>(sorti + kT5Sort);
      for (int q = warp; q < QT; q += kT5Threads / 32) {
        const int qi = q0 + q;
        if (qi >= L) break;
        int32_t* out_i = a.nbr_idx + static_cast<long long>(qi) * k;
        float* out_d = a.nbr_dist ? a.nbr_dist + static_cast<long long>(qi) * k : nullptr;
        if (dead) {
          for (int r = lane; r < k; r += 32) { out_i[r] = -1; if (out_d) out_d[r] = 0.f; }
          continue;
        }
        const unsigned long long* lq = my_lists + static_cast<size_t>(q) * CAP;
        int n = cnts[q];
        bool fallback = n < 0;
        if (!fallback) {
          if (n > k) {
            const float eq = eps2s[q];
            uint32_t limit;
            n = t5_warp_cut<false, 2>(lq, n, k, st, hist, st, [&](uint32_t kth) { return float_key(key_float(kth) + eq); }, &limit);
          } else {
            for (int i = lane; i < n; i += 32) st[i] = lq[i];
            __syncwarp();
          }
          fallback = n > kT5Sort;
        }
        if (fallback) {
          if (lane == 0) cnts[q] = -2;
          continue;
        }
        int p2 = 32;
        while (p2 < n) p2 *= 2;
        const __nv_bfloat16* q_row = cb + static_cast<long long>(qi) * d;
        for (int t = lane; t < d; t += 32) qd[t] = t5_bf16_to_double(__bfloat16_as_ushort(q_row[t]));
        __syncwarp();
        {
          // groups of 32 candidates, spread evenly over as few calls as the chains per lane allow
          const int groups = max((n + 31) / 32, 1), calls = (groups + kT5Chains - 1) / kT5Chains;
          const int nch = (groups + calls - 1) / calls;
          for (int c2 = 0; c2 < calls; ++c2) t5_exact_block(qd, cb, d, st, n, p2, c2 * 32 * nch, nch, sortd, sorti);
          for (int i = calls * 32 * nch + lane; i < p2; i += 32) {       // padding of the sort beyond the calls' range
            sorti[i] = 0x7fffffff;
            sortd[i] = 0x7ff0000000000000ull;
          }
        }
        __syncwarp();
        t5_warp_sort(sortd, sorti, p2);
        for (int r = lane; r < k; r += 32) {
          out_i[r] = sorti[r];
          if (out_d) out_d[r] = static_cast<float>(__longlong_as_double(static_cast<long long>(sortd[r])));
        }
        __syncwarp();
      }
    }
    __syncthreads();
    // queries with too many rows inside the error margin (duplicated rows): exact arg-min rounds by the whole CTA
    if (!dead) {
      double* redd = reinterpret_cast<double*>(bars + 16);
      int* redi = misc + 16;
      for (int q = 0; q < QT && q0 + q < L; ++q) {
        if (cnts[q] != -2) continue;                 // shared value: the same decision in every thread
        const int qi = q0 + q;
        rank_query<__nv_bfloat16>(cb, L, d, k, qi, nullptr, 0, true, 0, nullptr, nullptr, redd, redi,
                                  a.nbr_idx + static_cast<long long>(qi) * k,
                                  a.nbr_dist ? a.nbr_dist + static_cast<long long>(qi) * k : nullptr);
      }
    }
    __syncthreads();                                 // the stages go back to the loaders
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 4) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tbase), "r"(2 * kT5C) : "memory");
}

}  // namespace lantern
