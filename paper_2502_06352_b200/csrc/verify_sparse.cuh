// Relaxed tree verification for rows that are truncated to their top-k entries before the
// softmax (App. B "Models": top-k sampling), for vocabularies of up to 16384 tokens.
//
// After the truncation a row has only k (plus ties) non-zero probabilities, so the dense row is
// needed just long enough to find them.  A CTA of 512 threads handles one tree node:
//   1. target row: stream cond (asynchronous copies into shared memory) and uncond (registers),
//      form the pre-softmax values z, locate the exact k-th largest (histogram of max - z, exact
//      ranking inside the located bin) and compact the survivors into a (token, value) list;
//   2. the same for the drafter row, in the same 64 KB row buffer;
//   3. merge both lists into arrays over the union of their supports, ordered by token
//      (bitmap + popcount ranks); the sibling loop (Sec. 4; App. A.2 Eq. 1-2), the residual
//      updates and the inverse-CDF draw then sweep a few thousand entries instead of 2 x V.
// The footprint of ~100 KB lets two CTAs share an SM, so one node's streaming overlaps the other
// node's on-chip phases.  A node whose located bin or survivor list would not fit the fixed
// buffers (massive ties) sets its flag in `redo`; the dense kernel then processes exactly those.
#pragma once

#include "rowops.cuh"

namespace lantern {
namespace sparse {

constexpr int ST = 512;            // threads per CTA
constexpr int SW = ST / 32;
constexpr int kMaxV = 16384;       // widest row
constexpr int kCap = 1536;         // list entries per side
constexpr int kMaxTopK = 1280;     // largest top-k routed here (slack for the located bin)
constexpr int kCand = 512;         // entries of the located bin that are ranked exactly
constexpr int kUCap = 2 * kCap;    // union of both supports
constexpr int kWords = kMaxV / 32; // bitmap words
constexpr int kMisc = 96;     // [12..19] accept uniforms, [20..27] child tokens, [28..35] their union
                              // positions, [64..95] per-warp results of the draw

__host__ __device__ constexpr int z_floats(int e) { return ST * e > 3 * kUCap ? ST * e : 3 * kUCap; }
__host__ __device__ constexpr size_t smem_bytes(int e, int max_children, int kpad) {
  return static_cast<size_t>(z_floats(e)) * 4 + 4 * kCap * 4 + kBins * 4 + 3 * kWords * 4 + kCand * 4 +
         2 * SW * 2 * 4 + SW * 4 + kMisc * 4 + 16 + static_cast<size_t>(max_children) * kpad * 4;
}

struct Ctx {
  float* red;      // [2][SW*2]
  float* last_red; // buffer of the last reduction: per-warp partials at [w*2 + i]
  int parity;
};

// Block-wide sum or max of two values per thread; every thread gets the result.
template <bool IS_MAX, int NW = SW>
__device__ __forceinline__ void block_reduce2(Ctx& c, float (&v)[2]) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  float* red = c.red + c.parity * (NW * 2);
#pragma unroll
  for (int i = 0; i < 2; ++i) v[i] = IS_MAX ? warp_max(v[i]) : warp_sum(v[i]);
  if (lane == 0) { red[warp * 2] = v[0]; red[warp * 2 + 1] = v[1]; }
  __syncthreads();
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    const float t = lane < NW ? red[lane * 2 + i] : (IS_MAX ? -INFINITY : 0.f);
    v[i] = IS_MAX ? warp_max(t) : warp_sum(t);
  }
  c.last_red = red;
  c.parity ^= 1;
}

// Pre-softmax values of one row into Z (entries beyond the row end and outside the allowed
// token range become -inf); returns this thread's maximum.  cond arrives through asynchronous
// 16-byte copies into the place its values will occupy, uncond through registers in two batches.
template <typename T, bool CFG, int E>
__device__ __forceinline__ float load_row(const T* __restrict__ cond, const T* __restrict__ uncond, float g,
                                          float inv_tau, int len, int allow_lo, int allow_hi, bool masked,
                                          float* __restrict__ Z) {
  using VTT = Vec<T>;
  constexpr int VN = VTT::N, NV = E / VN, OFF = (VN == 8 ? 4 : 0);
  constexpr int NH = NV >= 2 ? NV / 2 : 1;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int wb = warp * 32 * E + lane * VN;
#pragma unroll
  for (int v = 0; v < NV; ++v) {
    const int j = wb + v * 32 * VN;
    if (j + VN <= len) cp_async16(smem_u32(Z + j + OFF), cond + j);
  }
  cp_async_commit();
  float mx = -INFINITY;
#pragma unroll
  for (int h = 0; h < NV; h += NH) {
    uint4 ur[NH];
    if (CFG) {
#pragma unroll
      for (int v = 0; v < NH; ++v) {
        const int j = wb + (h + v) * 32 * VN;
        ur[v] = make_uint4(0u, 0u, 0u, 0u);
        if (j + VN <= len) ur[v] = ldg_stream_u128(uncond + j);
      }
    }
    if (h == 0) cp_async_wait<0>();
#pragma unroll
    for (int v = 0; v < NH; ++v) {
      const int j = wb + (h + v) * 32 * VN;
      float zf[VN];
      if (j + VN <= len) {
        float cf[VN], uf[VN];
        const uint4 cr = lds_u128(Z + j + OFF);
        VTT::unpack_raw(cr, cf);
        if (CFG) VTT::unpack_raw(ur[v], uf);
#pragma unroll
        for (int e = 0; e < VN; ++e) zf[e] = combine<CFG>(cf[e], CFG ? uf[e] : 0.f, g, inv_tau);
      } else {
#pragma unroll
        for (int e = 0; e < VN; ++e) {
          float val = -INFINITY;
          if (j + e < len) {
            const float cc = VTT::widen(cond[j + e]);
            const float uu = CFG ? VTT::widen(uncond[j + e]) : 0.f;
            val = combine<CFG>(cc, uu, g, inv_tau);
          }
          zf[e] = val;
        }
      }
      if (masked) {
#pragma unroll
        for (int e = 0; e < VN; ++e)
          if (j + e < allow_lo || j + e >= allow_hi) zf[e] = -INFINITY;
      }
#pragma unroll
      for (int e = 0; e < VN; ++e) mx = fmaxf(mx, zf[e]);
      float4* d4 = reinterpret_cast<float4*>(Z + j);
#pragma unroll
      for (int e = 0; e < VN; e += 4) d4[e / 4] = make_float4(zf[e], zf[e + 1], zf[e + 2], zf[e + 3]);
    }
  }
  return mx;
}

struct Smem {
  float* Z;          // [z_floats]   dense row; later the union arrays
  int* ltok[2];      // [kCap]       survivors of the target / drafter row: token, pre-softmax value
  float* lval[2];
  uint32_t* bins;    // [kBins]
  uint32_t* bm[2];   // [kWords]     support bitmaps of the two lists
  uint32_t* rk;      // [kWords]     union entries before bitmap word w
  float* cand;       // [kCand]
  uint32_t* wtot;    // [SW]
  int* misc;         // [kMisc]
};

// Survivors of one row: every entry of Z in a histogram bin up to the one that holds the k-th
// largest becomes a list entry (token, z) and a bit of the side's bitmap; theta = the exact k-th
// largest value (ranking inside the located bin).  List entries below theta are dropped later
// (value 0).  Returns false when the fixed buffers cannot hold the row.  The order of the list
// depends on the order in which the warps reserve their ranges; nothing that is summed may
// depend on it.
// With DET the warps' ranges follow warp order (one more barrier instead of the atomic), so the
// list order is the same from run to run.
template <int E, bool DET = false, bool BITMAP = true>
__device__ __forceinline__ bool compact_topk(const Smem& s, int side, float mx, int kth, int& n_list,
                                             float& theta) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  constexpr int NV4 = E / 4;
  const float* Z = s.Z;
  int* ltok = s.ltok[side];
  float* lval = s.lval[side];
  uint32_t* bm = s.bm[side];
  // bins were cleared before the row was loaded (a barrier lies in between)
#pragma unroll
  for (int v = 0; v < NV4; ++v) {
    const float4 q = *reinterpret_cast<const float4*>(Z + warp * 32 * E + v * 128 + lane * 4);
    atomicAdd(&s.bins[dist_bin(mx, q.x)], 1u);
    atomicAdd(&s.bins[dist_bin(mx, q.y)], 1u);
    atomicAdd(&s.bins[dist_bin(mx, q.z)], 1u);
    atomicAdd(&s.bins[dist_bin(mx, q.w)], 1u);
  }
  if (tid == 0) { s.misc[8] = 0; s.misc[9] = 0; }        // list and candidate counters
  __syncthreads();
  {
    // smallest bin whose cumulative count reaches k: thread t scans bins 4t .. 4t+3
    const uint4 b4 = *reinterpret_cast<const uint4*>(s.bins + 4 * tid);
    const uint32_t c0 = b4.x, c1 = c0 + b4.y, c2 = c1 + b4.z, c3 = c2 + b4.w;
    uint32_t incl = c3;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += t;
    }
    if (lane == 31) s.wtot[warp] = incl;
    __syncthreads();
    uint32_t wt = lane < SW ? s.wtot[lane] : 0u, wincl = wt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t t = __shfl_up_sync(0xffffffffu, wincl, o);
      if (lane >= o) wincl += t;
    }
    const uint32_t before = __shfl_sync(0xffffffffu, wincl - wt, warp) + incl - c3;
    const uint32_t need = static_cast<uint32_t>(kth);
    const uint32_t lo4[4] = {before, before + c0, before + c1, before + c2};
    const uint32_t cn4[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      if (lo4[i] < need && need <= lo4[i] + cn4[i]) {
        s.misc[0] = 4 * tid + i;
        s.misc[1] = static_cast<int>(need - lo4[i]);
        s.misc[2] = static_cast<int>(cn4[i]);
      }
    }
  }
  __syncthreads();
  const int bstar = s.misc[0], krem = s.misc[1], nb = s.misc[2];
  if (nb > kCand || kth - krem + nb > kCap) return false;          // same decision in every thread
  // Entries of the bins up to the located one -> list; those of the located bin also -> the
  // candidate array.  Each thread marks its entries in a bit mask, a warp reserves its range of the
  // list with one atomic (or, with DET, by a scan over the warps' counts).
  const uint32_t hi_bits = bin_hi_bits(bstar), lo_bits = bin_lo_bits(bstar);
  uint32_t mask = 0;
#pragma unroll
  for (int v = 0; v < NV4; ++v) {
    const float4 q = *reinterpret_cast<const float4*>(Z + warp * 32 * E + v * 128 + lane * 4);
    if (__float_as_uint(mx - q.x) <= hi_bits) mask |= 1u << (4 * v);
    if (__float_as_uint(mx - q.y) <= hi_bits) mask |= 1u << (4 * v + 1);
    if (__float_as_uint(mx - q.z) <= hi_bits) mask |= 1u << (4 * v + 2);
    if (__float_as_uint(mx - q.w) <= hi_bits) mask |= 1u << (4 * v + 3);
  }
  {
    const int cnt = __popc(mask);
    int incl = cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += t;
    }
    int base = 0;
    if (DET) {
      if (lane == 31) s.wtot[warp] = static_cast<uint32_t>(incl);
      __syncthreads();
      int wt = lane < SW ? static_cast<int>(s.wtot[lane]) : 0, wincl = wt;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, wincl, o);
        if (lane >= o) wincl += t;
      }
      base = __shfl_sync(0xffffffffu, wincl - wt, warp) + incl - cnt;
      const int total = __shfl_sync(0xffffffffu, wincl, SW - 1);
      if (tid == 0) s.misc[8] = total;
    } else {
      if (lane == 31) base = atomicAdd(&s.misc[8], incl);
      base = __shfl_sync(0xffffffffu, base, 31) + incl - cnt;
    }
    int pos = base;
    while (mask) {
      const int i = __ffs(mask) - 1;
      mask &= mask - 1;
      const int j = warp * 32 * E + (i >> 2) * 128 + lane * 4 + (i & 3);
      const float z = Z[j];
      if (pos < kCap) { ltok[pos] = j; lval[pos] = z; }
      ++pos;
      if (BITMAP) atomicOr(&bm[j >> 5], 1u << (j & 31));
      if (__float_as_uint(mx - z) >= lo_bits) {
        const int cp = atomicAdd(&s.misc[9], 1);
        if (cp < kCand) s.cand[cp] = z;
      }
    }
  }
  __syncthreads();
  n_list = min(s.misc[8], kCap);
  const int ncand = min(s.misc[9], kCand);
  // exact rank by counting inside the located bin: theta = v with #(> v) < krem <= #(>= v);
  // eight lanes share the comparisons of one candidate
  {
    const int nc8 = (ncand + (ST / 8) - 1) / (ST / 8) * (ST / 8);
    for (int i = tid >> 3; i < nc8; i += ST / 8) {
      const float v = i < ncand ? s.cand[i] : 0.f;
      int gt = 0, ge = 0;
      for (int t = tid & 7; t < ncand; t += 8) {
        const float w = s.cand[t];
        gt += (w > v);
        ge += (w >= v);
      }
#pragma unroll
      for (int o = 1; o < 8; o <<= 1) {
        gt += __shfl_xor_sync(0xffffffffu, gt, o);
        ge += __shfl_xor_sync(0xffffffffu, ge, o);
      }
      if (i < ncand && (tid & 7) == 0 && gt < krem && krem <= ge) reinterpret_cast<float*>(s.misc)[3] = v;
    }
  }
  __syncthreads();
  theta = reinterpret_cast<const float*>(s.misc)[3];
  return true;
}

// Shared memory and identity of the per-node part (union build, sibling loop, draw), which the
// kernel runs after compacting its two rows.
struct NodeSmem {
  int* ut;           // [kUCap]  union arrays: token, target mass, drafter mass
  float* uq;
  float* up;
  uint32_t* bm[2];   // [kWords] support bitmaps of the two lists
  uint32_t* rk;      // [kWords] union entries before bitmap word w
  uint32_t* wtot;    // [NT/32]
  int* misc;         // [kMisc]
  uint64_t* mbar;
  int* nbr_s;        // [max_children][kpad]
};
struct NodeId {
  int b, n, fc, nc;
  long long out_b;
  const int32_t* tok_b;
};

// Starts the copy of the children's neighbour rows and fetches the node's uniforms and draft
// tokens.  Returns whether a bulk copy is in flight (to be awaited by node_tail).
template <int NT>
__device__ __forceinline__ bool node_prologue(const VerifyArgs& a, const NodeSmem& ns, const NodeId& id) {
  const int tid = threadIdx.x;
  const int n = id.n, fc = id.fc, nc = id.nc;
  const long long out_b = id.out_b;
  const int32_t* tok_b = id.tok_b;
  int* misc = ns.misc;
  float* miscf = reinterpret_cast<float*>(ns.misc);
  int* nbr_s = ns.nbr_s;
  uint64_t* mbar = ns.mbar;
  // ---- stage the children's neighbour rows (bulk async copy when rows are 16-byte aligned)
  const bool want_nbr = nc > 0 && a.k > 0;
  const uint32_t mbar_a = smem_u32(mbar);
  bool bulk_issued = false;
  if (want_nbr && a.use_bulk) {
    if (tid == 0) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(mbar_a) : "memory");
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
      uint32_t bytes = 0;
      const uint32_t row_bytes = static_cast<uint32_t>(((a.k + 3) & ~3) * 4);
      for (int ci = 0; ci < nc; ++ci) {
        int code = tok_b[fc + ci] - a.code_offset;
        if (code >= 0 && code < a.n_codes) bytes += row_bytes;
      }
      asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(mbar_a), "r"(bytes) : "memory");
      for (int ci = 0; ci < nc; ++ci) {
        int code = tok_b[fc + ci] - a.code_offset;
        if (code >= 0 && code < a.n_codes) {
          const int32_t* src = a.nbr + static_cast<long long>(code) * a.k_table;
          uint32_t dst = smem_u32(nbr_s + ci * a.kpad);
          asm volatile(
              "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
              ::"r"(dst), "l"(src), "r"(row_bytes), "r"(mbar_a) : "memory");
        }
      }
    }
    bulk_issued = true;
  } else if (want_nbr) {
    for (int ci = 0; ci < nc; ++ci) {
      int code = tok_b[fc + ci] - a.code_offset;
      if (code >= 0 && code < a.n_codes)
        for (int r = tid; r < a.k; r += NT)
          nbr_s[ci * a.kpad + r] = a.nbr[static_cast<long long>(code) * a.k_table + r];
    }
  }

  // ---- uniforms of this node
  if (tid == 32) {
    float u;
    if (a.u_res) {
      u = a.u_res[out_b + n];
    } else {
      u = uniform_halfopen(philox_stream(a.seed, a.step, static_cast<uint32_t>(out_b + n), kStreamResample, 0).x);
    }
    miscf[7] = u;
  }
  if (tid < nc) {
    float u;
    if (a.u_acc) {
      u = a.u_acc[out_b + fc + tid];
    } else {
      u = uniform_halfopen(philox_stream(a.seed, a.step, static_cast<uint32_t>(out_b + fc + tid), kStreamAccept, 0).x);
    }
    miscf[12 + tid] = u;
    misc[20 + tid] = tok_b[fc + tid];
  }
  return bulk_issued;
}

// The per-node part: merges the two lists (token, unnormalised probability; the bitmaps hold their
// supports) into the union arrays, runs the sibling loop (Sec. 4; App. A.2 Eq. 1-2) and the
// inverse-CDF draw, and writes the node's results.  NT threads; a barrier must separate the last
// write of the bitmaps and lists from the call.
template <int NT>
__device__ __forceinline__ void node_tail(const VerifyArgs& a, Ctx& c, const NodeSmem& ns, const NodeId& id,
                                          const bool bulk_issued, const int* ltok0, const float* lval0, const int n0,
                                          const int* ltok1, const float* lval1, const int n1) {
  constexpr int NW = NT / 32;
  static_assert(kWords % NT == 0, "whole bitmap words per thread");
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n = id.n, fc = id.fc, nc = id.nc;
  const long long out_b = id.out_b;
  const int32_t* tok_b = id.tok_b;
  int* misc = ns.misc;
  float* miscf = reinterpret_cast<float*>(ns.misc);
  int* nbr_s = ns.nbr_s;
  const uint32_t mbar_a = smem_u32(ns.mbar);
  const bool want_nbr = nc > 0 && a.k > 0;
  // ---- union of the two supports, ordered by token: popcount ranks of the OR-ed bitmaps, then
  // every list entry is scattered to its rank
  int* ut = ns.ut;
  float* uq = ns.uq;
  float* up = ns.up;
  int n_u;
  {
    constexpr int WPT = kWords / NT;            // bitmap words per thread
    int before[WPT], cnt = 0;
#pragma unroll
    for (int j = 0; j < WPT; ++j) {
      before[j] = cnt;
      cnt += __popc(ns.bm[0][tid * WPT + j] | ns.bm[1][tid * WPT + j]);
    }
    int incl = cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += t;
    }
    if (lane == 31) ns.wtot[warp] = incl;
    __syncthreads();
    int wt = lane < NW ? static_cast<int>(ns.wtot[lane]) : 0, wincl = wt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(0xffffffffu, wincl, o);
      if (lane >= o) wincl += t;
    }
    const int base = __shfl_sync(0xffffffffu, wincl - wt, warp) + incl - cnt;
#pragma unroll
    for (int j = 0; j < WPT; ++j) ns.rk[tid * WPT + j] = static_cast<uint32_t>(base + before[j]);
    n_u = __shfl_sync(0xffffffffu, wincl, NW - 1);
  }
  // ---- neighbour rows must have landed
  if (bulk_issued) {
    bool landed = mbar_wait_bounded(mbar_a, 0);
    if (!__syncthreads_and(landed)) {
      if (tid == 0) vflag(a.status, LANTERN_DEV_TIMEOUT);
      for (int ci = 0; ci < nc; ++ci) {
        int code = tok_b[fc + ci] - a.code_offset;
        if (code >= 0 && code < a.n_codes)
          for (int r = tid; r < a.k; r += NT)
            nbr_s[ci * a.kpad + r] = a.nbr[static_cast<long long>(code) * a.k_table + r];
      }
    }
  }
  __syncthreads();
  // position of token t in the union arrays, or -1
  auto uidx = [&](int t) -> int {
    const uint32_t w = ns.bm[0][t >> 5] | ns.bm[1][t >> 5], bit = 1u << (t & 31);
    return (w & bit) ? static_cast<int>(ns.rk[t >> 5]) + __popc(w & (bit - 1u)) : -1;
  };
#pragma unroll
  for (int side = 0; side < 2; ++side) {
    float* mine = side ? up : uq;
    float* other = side ? uq : up;
    const uint32_t* obm = ns.bm[side ^ 1];
    const int* lt = side ? ltok1 : ltok0;
    const float* lv = side ? lval1 : lval0;
    const int nl = side ? n1 : n0;
    for (int i = tid; i < nl; i += NT) {
      const int t = lt[i], u = uidx(t);
      ut[u] = t;
      mine[u] = lv[i];
      if (!((obm[t >> 5] >> (t & 31)) & 1u)) other[u] = 0.f;
    }
  }
  // the staged neighbour codes become positions in the union arrays (-1: not in either support,
  // -2: outside the vocabulary), so that the serial sibling loop below only follows one index
  if (tid < nc) {
    const int x = misc[20 + tid];
    misc[28 + tid] = (x >= 0 && x < a.V) ? uidx(x) : -1;
  }
  if (want_nbr) {
    for (int i = tid; i < nc * a.k; i += NT) {
      const int ci = i / a.k, r = i - ci * a.k;
      const int t = a.code_offset + nbr_s[ci * a.kpad + r];
      nbr_s[ci * a.kpad + r] = (t >= 0 && t < a.V) ? uidx(t) : -2;
    }
  }
  __syncthreads();
  // From here on thread t owns the union entries [t*per, t*per + per) in every sweep, so that a
  // thread re-reads only what it wrote itself and the per-warp partial sums of a reduction are
  // sums over consecutive tokens.  per is odd: consecutive threads hit different banks.
  const int per = ((n_u + NT - 1) / NT) | 1;
  const int i0 = min(tid * per, n_u), i1 = min(i0 + per, n_u);
  float tot[2] = {0.f, 0.f};
  for (int i = i0; i < i1; ++i) { tot[0] += uq[i]; tot[1] += up[i]; }
  block_reduce2<false, NW>(c, tot);
  float qtot = tot[0];
  float qs = qtot > 0.f ? 1.f / qtot : 0.f;
  float psum = tot[1];

  if (n == 0 && tid == 0) {
    if (a.node_mass) a.node_mass[out_b] = -1.f;
    if (a.node_thresh) a.node_thresh[out_b] = -1.f;
  }

  // ---- sibling loop (Sec. 4; Eq. 1-2) on the union arrays.  Warp 0 evaluates a child: relaxed
  // mass, decision and, on rejection, q~ (the mass of A moved onto x); one barrier publishes all
  // of it, the residual sweep and its reduction follow.
  int accepted = -1;
  for (int ci = 0; ci < nc && accepted < 0; ++ci) {
    const int child = fc + ci;
    const int x = misc[20 + ci];
    if (x < 0 || x >= a.V) {
      if (tid == 0) {
        if (x >= a.V) vflag(a.status, LANTERN_DEV_BAD_INDEX);
        if (a.node_mass) a.node_mass[out_b + child] = -1.f;
        if (a.node_thresh) a.node_thresh[out_b + child] = -1.f;
      }
      continue;
    }
    const int code = x - a.code_offset;
    const bool has_code = a.k > 0 && code >= 0 && code < a.n_codes;
    const int* nrow = nbr_s + ci * a.kpad;
    const float ps = psum > 0.f ? 1.f / psum : 0.f;
    if (warp == 0) {
      const int ix = misc[28 + ci];
      const float qx = ix >= 0 ? uq[ix] * qs : 0.f;
      const float pxraw = ix >= 0 ? up[ix] : 0.f;
      const float px = pxraw * ps;
      const float bound = a.delta > 0.f ? qx + a.delta : a.lambda * qx;      // Sec. 2.2 / Sec. 4
      float cum = qx;
      int nA = 0;
      bool bad = false, open = has_code;
      for (int base8 = 0; base8 < a.k && open; base8 += 256) {
        float qa[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int r = base8 + i * 32 + lane;
          qa[i] = 0.f;
          if (r < a.k) {
            const int it = nrow[r];
            if (it >= 0) qa[i] = uq[it] * qs;
            bad |= it == -2;
          }
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          if (!open) break;
          const int r = base8 + i * 32 + lane;
          if (base8 + i * 32 >= a.k) { open = false; break; }
          const float incl = warp_incl_scan(qa[i], lane);
          const bool okr = r < a.k && (cum + incl < bound);
          const uint32_t ballot = __ballot_sync(0xffffffffu, okr);
          const int ntake = __ffs(~ballot) - 1;
          const int take = ntake < 0 ? 32 : ntake;
          if (take > 0) cum += __shfl_sync(0xffffffffu, incl, take - 1);
          nA += take;
          if (take < 32) open = false;
        }
      }
      if (__any_sync(0xffffffffu, bad) && lane == 0) vflag(a.status, LANTERN_DEV_BAD_INDEX);
      const float m = cum;
      const float thr = px > 0.f ? fminf(1.f, m / px) : (m > 0.f ? 1.f : 0.f);
      const bool acc = miscf[12 + ci] < thr;
      if (!acc) {
        // q~: the first nA neighbours give their mass to x
        __syncwarp();
        for (int r = lane; r < nA; r += 32) {
          const int it = nrow[r];
          if (it >= 0) uq[it] = 0.f;
        }
        __syncwarp();
        if (lane == 0 && ix >= 0) uq[ix] = qs > 0.f ? m / qs : 0.f;
      }
      if (lane == 0) {
        misc[0] = acc ? 1 : 0;
        miscf[3] = pxraw;
        misc[4] = ix;
        if (a.node_mass) a.node_mass[out_b + child] = m;
        if (a.node_thresh) a.node_thresh[out_b + child] = thr;
      }
    }
    __syncthreads();
    if (misc[0]) {
      accepted = child;       // leaves the loop: misc is not rewritten
      break;
    }
    const float pxraw = miscf[3];
    const int ix = misc[4];
    // Q <- [Q * rho - P]_+ with rho = qs * psum: the residual of Eq. 2 in the (unnormalised)
    // units of P.  The drafter mass left without x is psum - P[x] unless that cancels badly.
    const bool resum = pxraw > 0.5f * psum;
    const float rho = psum > 0.f ? qs * psum : qs;
    float zs[2] = {0.f, 0.f};
    for (int i = i0; i < i1; ++i) {
      float p = up[i];
      const float q = fmaxf(fmaf(uq[i], rho, -p), 0.f);
      uq[i] = q;
      zs[0] += q;
      if (i == ix) { up[i] = 0.f; p = 0.f; }
      if (resum) zs[1] += p;
    }
    block_reduce2<false, NW>(c, zs);
    const float ps_old = ps;
    psum = resum ? zs[1] : psum - pxraw;
    if (zs[0] > 0.f) {
      qtot = zs[0];
      qs = 1.f / zs[0];
    } else {
      // q~ <= p_cur everywhere: both sum to one, so q~ equals p_cur (before x was dropped)
      float s2[2] = {0.f, 0.f};
      for (int i = i0; i < i1; ++i) {
        const float p = i == ix ? pxraw : up[i];
        uq[i] = p;
        s2[0] += p;
      }
      block_reduce2<false, NW>(c, s2);
      qtot = s2[0];
      qs = ps_old;
    }
  }
  // children that were not tested because an earlier sibling was accepted
  if (accepted >= 0 && tid > accepted - fc && tid < nc) {
    if (a.node_mass) a.node_mass[out_b + fc + tid] = -1.f;
    if (a.node_thresh) a.node_thresh[out_b + fc + tid] = -1.f;
  }

  // ---- no child accepted (or leaf): draw node_token from q_cur by inverse CDF in token order.
  // The last reduction left the sums of uq over each warp's (consecutive) entries in
  // c.last_red[w*2]; a thread re-reads only the entries it wrote itself.
  if (accepted < 0) {
    const float target = miscf[7] * qtot;
    float sc = 0.f;
    for (int i = i0; i < i1; ++i) sc += uq[i];
    const float incl = warp_incl_scan(sc, lane);
    const float wt = lane < NW ? c.last_red[lane * 2] : 0.f;
    const float wincl = warp_incl_scan(wt, lane);
    float run = __shfl_sync(0xffffffffu, wincl - wt, warp) + (incl - sc);
    int cand = 0x7fffffff, lastp = -1;
    for (int i = i0; i < i1; ++i) {
      const float v = uq[i];
      run += v;
      if (v > 0.f) {
        lastp = i;
        if (cand == 0x7fffffff && run > target) cand = i;
      }
    }
    cand = __reduce_min_sync(0xffffffffu, cand);      // first crossing / last positive entry of the warp
    lastp = __reduce_max_sync(0xffffffffu, lastp);
    if (lane == 0) { misc[64 + warp] = cand; misc[80 + warp] = lastp; }
    __syncthreads();
    if (warp == 0) {
      cand = __reduce_min_sync(0xffffffffu, lane < NW ? misc[64 + lane] : 0x7fffffff);
      lastp = __reduce_max_sync(0xffffffffu, lane < NW ? misc[80 + lane] : -1);
      if (lane == 0) {
        const int found = cand != 0x7fffffff ? cand : lastp;
        a.node_token[out_b + n] = found >= 0 ? ut[found] : -1;
        if (found < 0) vflag(a.status, LANTERN_DEV_EMPTY_ROW);
      }
    }
  } else if (tid == 0) {
    a.node_token[out_b + n] = -1;
  }
  if (tid == 0) a.node_next[out_b + n] = accepted;
}

// ------------------------------------------------------------------------------------------------
// One CTA of 512 threads per node does everything (both rows, then the per-node part).
// E = row entries per thread (V <= 512 * E).
// `redo[b*N + n]` is set to 1 when node (b, n) has to be processed by the dense kernel instead, else to 0.
template <typename T, bool CFG, int E>
__global__ void __launch_bounds__(ST, 2) verify_sparse_kernel(const VerifyArgs a, int32_t* __restrict__ redo, const int chunk) {
  grid_dependency_sync();
  extern __shared__ __align__(16) unsigned char smem_raw[];
  Smem s;
  s.Z = reinterpret_cast<float*>(smem_raw);
  s.ltok[0] = reinterpret_cast<int*>(s.Z + z_floats(E));
  s.lval[0] = reinterpret_cast<float*>(s.ltok[0] + kCap);
  s.ltok[1] = reinterpret_cast<int*>(s.lval[0] + kCap);
  s.lval[1] = reinterpret_cast<float*>(s.ltok[1] + kCap);
  s.bins = reinterpret_cast<uint32_t*>(s.lval[1] + kCap);
  s.bm[0] = s.bins + kBins;
  s.bm[1] = s.bm[0] + kWords;
  s.rk = s.bm[1] + kWords;
  s.cand = reinterpret_cast<float*>(s.rk + kWords);
  Ctx c;
  c.red = s.cand + kCand;
  c.last_red = c.red;
  c.parity = 0;
  s.wtot = reinterpret_cast<uint32_t*>(c.red + 2 * SW * 2);
  s.misc = reinterpret_cast<int*>(s.wtot + SW);
  NodeSmem ns;
  ns.ut = reinterpret_cast<int*>(s.Z);          // the union arrays take over the row buffer
  ns.uq = s.Z + kUCap;
  ns.up = ns.uq + kUCap;
  ns.bm[0] = s.bm[0];
  ns.bm[1] = s.bm[1];
  ns.rk = s.rk;
  ns.wtot = s.wtot;
  ns.misc = s.misc;
  ns.mbar = reinterpret_cast<uint64_t*>(s.misc + kMisc);
  ns.nbr_s = reinterpret_cast<int*>(ns.mbar + 2);

  const int tid = threadIdx.x;
  if (blockIdx.x == 0 && tid == 0 && a.done) *a.done = 0;      // counter of the repair launch that follows
  // Launch order: blocks of `chunk` CTAs (one per SM) alternate between internal nodes (two rows,
  // sibling loop) and leaves (one row), so that the two CTAs sharing an SM start in different
  // phases and one's streaming overlaps the other's on-chip work.  The grid is padded to whole
  // blocks; CTAs beyond the last node of their kind leave at once.
  int idx;
  {
    const int nI = a.B * a.n_internal, nL = a.B * (a.N - a.n_internal);
    const int mI = (nI + chunk - 1) / chunk, mL = (nL + chunk - 1) / chunk;
    const int cb = blockIdx.x / chunk, off = blockIdx.x - cb * chunk;
    const int both = 2 * min(mI, mL);
    int kind, k;
    if (cb < both) {
      kind = cb & 1;
      k = (cb >> 1) * chunk + off;
    } else {
      kind = mI > mL ? 0 : 1;
      k = (min(mI, mL) + (cb - both)) * chunk + off;
    }
    if (k >= (kind ? nL : nI)) return;
    idx = kind ? nI + k : k;            // position in the internal-first node order
  }
  NodeId id;
  id.b = idx % a.B;
  id.n = a.order[idx / a.B];
  id.fc = a.first_child[id.n];
  id.nc = a.n_child[id.n];
  id.out_b = static_cast<long long>(id.b) * a.N;
  id.tok_b = a.tokens + id.out_b;
  const int len = min(a.V, ST * E);
  const long long row_off = static_cast<long long>(id.b) * a.seq_stride + static_cast<long long>(id.n) * a.row_stride;

  const bool bulk_issued = node_prologue<ST>(a, ns, id);
  static_assert(kWords == ST, "one bitmap word per thread");
  s.bm[0][tid] = 0;
  s.bm[1][tid] = 0;

  // ---- both rows, one after the other through the same row buffer
  const bool masked = a.allow_lo > 0 || a.allow_hi < a.V;
  const int nside = id.nc > 0 ? 2 : 1;
  int n_list[2] = {0, 0};
  bool ok = true;
  for (int side = 0; side < nside && ok; ++side) {
    const T* cond = static_cast<const T*>(side ? a.dc : a.tc) + row_off;
    const T* uncond = CFG ? static_cast<const T*>(side ? a.du : a.tu) + row_off : nullptr;
    for (int i = tid; i < kBins; i += ST) s.bins[i] = 0;
    float mx[2];
    mx[0] = load_row<T, CFG, E>(cond, uncond, a.g, a.inv_tau, len, a.allow_lo, a.allow_hi, masked, s.Z);
    mx[1] = -INFINITY;
    block_reduce2<true>(c, mx);
    if (mx[0] == -INFINITY) { ok = false; break; }           // no finite logit: the dense kernel reports it
    float theta;
    ok = compact_topk<E>(s, side, mx[0], side ? a.topk_d : a.topk_t, n_list[side], theta);
    if (ok) {
      // list values become 2^((z - max) log2 e), or 0 below the threshold; the same thread reads
      // them back when the lists are merged
      const float c0 = -mx[0] * kLog2e;
      float* lv = s.lval[side];
      for (int i = tid; i < n_list[side]; i += ST) {
        const float z = lv[i];
        lv[i] = z >= theta ? ex2_approx(fmaf(z, kLog2e, c0)) : 0.f;
      }
    }
  }
  if (!ok) {
    // finish the outstanding bulk copy before leaving (bounded), then hand the node over
    if (bulk_issued) mbar_wait_bounded(smem_u32(ns.mbar), 0);
    if (tid == 0) redo[id.out_b + id.n] = 1;
    return;
  }
  node_tail<ST>(a, c, ns, id, bulk_issued, s.ltok[0], s.lval[0], n_list[0], s.ltok[1], s.lval[1], n_list[1]);
  if (tid == 0) redo[id.out_b + id.n] = 0;
}

}  // namespace sparse
}  // namespace lantern
