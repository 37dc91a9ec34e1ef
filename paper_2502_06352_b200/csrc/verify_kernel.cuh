// Device code of the relaxed tree-verification kernel (Sec. 4; App. A.2 Eq. 1-2; Sec. 2.1).
//
// One CTA of 1024 threads owns a slice of SL = 1024*E row entries; a row wider than one slice
// is split over the CTAs of a thread-block cluster (CTA `rank` owns [rank*SL, rank*SL+SL)).
// With V <= 16384 a node is one CTA and every reduction is a block reduction; only wider
// rows pay for cluster barriers and distributed-shared-memory reads.
//
// The node's target row (and, if it has children, its drafter row) is read from HBM once with
// 128-bit streaming loads and post-processed (guidance, temperature, top-k, softmax); the
// unnormalised distributions stay in shared memory: q_cur[j] = Q[j]*qs, p_cur[j] = P[j]/psum.
// The sibling loop, the residual updates and the inverse-CDF draw run on chip.
#include "rowops.cuh"

#ifndef LANTERN_VT
#define LANTERN_VT 1024
#endif
#ifndef LANTERN_VNS
#define LANTERN_VNS v1024
#endif

// This header is compiled once per thread count, each time into its own namespace.
namespace lantern {
namespace LANTERN_VNS {

constexpr int VT = LANTERN_VT;    // threads per CTA (1024 or 512)
constexpr int VW = VT / 32;       // warps per CTA
static_assert(VT == 1024 || VT == 512, "thread count");
constexpr int kCandLocal = 512;   // top-k candidates one CTA may contribute per row
constexpr int kCandTotal = 1024;  // and the whole cluster


constexpr int kMiscInts = 16;
constexpr int kCntInts = 2 + 2 * kMaxCluster + 2;
// Dynamic shared memory: [Q][P]([U] with guidance) [scratch] [small] [neighbour rows].
// scratch = buffers that only the top-k routine needs while the rows still hold pre-softmax
// values (row-wide bins, compacted and gathered candidates); with guidance it aliases U, which is
// dead once the rows are loaded, when U is large enough.
constexpr int kScratchBytes = 2 * kBins * 4 + 2 * kCandLocal * 4 + 2 * kCandTotal * 4;
constexpr int kSmallSmem = 2 * kBins * 4 + 2 * kCandLocal * 4 + 2 * VW * 4 + 2 * (kBins / 32) * 4   // bins, lists, counts, block totals
                           + 2 * VW * 4 * 4      // red (two buffers)
                           + 2 * 4 * 4           // xch
                           + kMaxCluster * 4 * 4 // gath
                           + 8 * 4 + kCntInts * 4 + kMiscInts * 4 + 16;
__host__ __device__ constexpr bool scratch_aliases_u(bool cfg, int e) { return cfg && VT * e * 4 >= kScratchBytes; }
__host__ __device__ constexpr size_t row_smem_bytes(bool cfg, int e) {
  return static_cast<size_t>(cfg ? 3 : 2) * VT * e * 4 + (scratch_aliases_u(cfg, e) ? 0 : kScratchBytes) + kSmallSmem;
}

struct VCtx {
  uint32_t rank, nrank;
  int parity;
  float* red;      // [2][VW*4]
  float* xch;      // [2][4]
  float* gath;     // [kMaxCluster*4] per-rank values of the last reduction
  float* last_red; // red buffer of the last reduction (per-warp values)
};

__device__ __forceinline__ void csync(const VCtx& c) {       // whole row: block or cluster
  if (c.nrank > 1) cluster_sync(); else __syncthreads();
}

// Row-wide sum or max of NV values per thread.  Every thread of the row's CTAs gets the same
// result (fixed combination order).  The per-warp partials stay in c.last_red[w*NV+i] and the
// per-rank partials in c.gath[r*NV+i] until the next call.
template <int NV, bool IS_MAX>
__device__ __forceinline__ void row_reduce(VCtx& c, float (&v)[NV]) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  float* red = c.red + c.parity * (VW * 4);
#pragma unroll
  for (int i = 0; i < NV; ++i) v[i] = IS_MAX ? warp_max(v[i]) : warp_sum(v[i]);
  if (lane == 0) {
#pragma unroll
    for (int i = 0; i < NV; ++i) red[warp * NV + i] = v[i];
  }
  __syncthreads();
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    float t = lane < VW ? red[lane * NV + i] : (IS_MAX ? -INFINITY : 0.f);   // one partial per lane
    v[i] = IS_MAX ? warp_max(t) : warp_sum(t);
  }
  if (c.nrank > 1) {
    if (threadIdx.x < NV) c.xch[c.parity * 4 + threadIdx.x] = v[threadIdx.x];
    cluster_sync();
#pragma unroll
    for (int i = 0; i < NV; ++i) {
      float t = IS_MAX ? -INFINITY : 0.f;
      if (lane < static_cast<int>(c.nrank)) t = dsmem_ld_f32(dsmem_addr(smem_u32(&c.xch[c.parity * 4 + i]), lane));
      if (warp == 0 && lane < static_cast<int>(c.nrank)) c.gath[lane * NV + i] = t;
      v[i] = IS_MAX ? warp_max(t) : warp_sum(t);
    }
  } else if (threadIdx.x < NV) {
    c.gath[threadIdx.x] = v[threadIdx.x];
  }
  c.last_red = red;
  c.parity ^= 1;
}

// Loading a row slice is split in two so that several operands can be in flight at once:
// issue_row starts asynchronous 16-byte copies of this thread's chunks of one operand straight
// into shared memory (no registers are held), finish_row turns the landed chunks into
// pre-softmax values in place.  A thread only ever touches the chunks it issued itself, so the
// two need no block-wide barrier between them, only the thread's own cp.async wait.
// float32 chunks land where their 4 values will live; bfloat16 chunks (8 values, 16 bytes) land
// in the upper half of the 32 bytes their 8 float32 values will occupy.
template <typename T, int E>
__device__ __forceinline__ void issue_row(const T* __restrict__ src, int lo, int len, float* __restrict__ dst) {
  constexpr int VN = Vec<T>::N, NV = E / VN;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int wb = warp * 32 * E + lane * VN;
#pragma unroll
  for (int v = 0; v < NV; ++v) {
    const int j = wb + v * 32 * VN;
    if (j + VN <= len) cp_async16(smem_u32(dst + j + (VN == 8 ? 4 : 0)), src + lo + j);
  }
}

// Pre-softmax values of one row slice, in place (entries beyond the row end and outside the
// allowed token range become -inf).  `dst` holds the landed cond chunks, `ubuf` the uncond
// chunks; the ragged last vector of a row is read with scalar loads.  Returns this thread's max.
template <typename T, bool CFG, int E>
__device__ __forceinline__ float finish_row(const T* __restrict__ cond, const T* __restrict__ uncond, float g,
                                            float inv_tau, int lo, int len, int allow_lo, int allow_hi,
                                            bool masked, float* __restrict__ dst, const float* __restrict__ ubuf) {
  using VTT = Vec<T>;
  constexpr int VN = VTT::N, NV = E / VN, OFF = (VN == 8 ? 4 : 0);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int wb = warp * 32 * E + lane * VN;
  float mx = -INFINITY;
#pragma unroll
  for (int v = 0; v < NV; ++v) {
    const int j = wb + v * 32 * VN;
    float zf[VN];
    if (j + VN <= len) {
      float cf[VN], uf[VN];
      const uint4 cr = lds_u128(dst + j + OFF);
      VTT::unpack_raw(cr, cf);
      if (CFG) {
        const uint4 ur = lds_u128(ubuf + j + OFF);
        VTT::unpack_raw(ur, uf);
      }
#pragma unroll
      for (int e = 0; e < VN; ++e) zf[e] = combine<CFG>(cf[e], CFG ? uf[e] : 0.f, g, inv_tau);
    } else {
#pragma unroll
      for (int e = 0; e < VN; ++e) {
        float val = -INFINITY;
        if (j + e < len) {
          const float cc = VTT::widen(cond[lo + j + e]);
          const float uu = CFG ? VTT::widen(uncond[lo + j + e]) : 0.f;
          val = combine<CFG>(cc, uu, g, inv_tau);
        }
        zf[e] = val;
      }
    }
    if (masked) {
#pragma unroll
      for (int e = 0; e < VN; ++e)
        if (lo + j + e < allow_lo || lo + j + e >= allow_hi) zf[e] = -INFINITY;
    }
#pragma unroll
    for (int e = 0; e < VN; ++e) mx = fmaxf(mx, zf[e]);
    float4* d4 = reinterpret_cast<float4*>(dst + j);
#pragma unroll
    for (int e = 0; e < VN; e += 4) d4[e / 4] = make_float4(zf[e], zf[e + 1], zf[e + 2], zf[e + 3]);
  }
  return mx;
}

struct TopkSmem {
  uint32_t* bins;   // [2][kBins]
  uint32_t* gbins;  // [2][kBins]  bins of the whole row (clusters only)
  float* wl;        // [2][VW][kCandLocal/VW] per-warp candidate lists
  float* comp;      // [2][kCandLocal]   compacted candidates
  uint32_t* wtot;   // [2][kBins/32] inclusive totals of 32-bin blocks
  float* all;       // [2][kCandTotal]
  int* wcnt;        // [2][VW]
  int* sel;         // [8]
  int* cnts;        // [2] local counts, then [2][kMaxCluster] counts of every rank
};

// Exact top-k thresholds of up to two rows whose pre-softmax values sit in shared memory
// (row r active iff kth[r] > 0): theta[r] = the kth[r]-th largest entry of the whole row.
// A histogram over dist_bin locates the bin of the k-th entry; the entries of that bin are
// gathered from all CTAs of the row and ranked exactly.  If they do not fit, the bin is
// refined by a radix select on the raw keys restricted to it.
template <int E>
__device__ __forceinline__ void topk_thresholds(VCtx& c, const TopkSmem& s, const float* __restrict__ z0,
                                                const float* __restrict__ z1, const float (&mx)[2],
                                                const int (&kth)[2], float (&theta)[2]) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  constexpr int NV4 = E / 4;
  for (int i = tid; i < 2 * kBins; i += VT) s.bins[i] = 0;
  __syncthreads();
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    if (kth[r] <= 0) continue;
    const float* z = r ? z1 : z0;
#pragma unroll
    for (int v = 0; v < NV4; ++v) {
      const float4 q = *reinterpret_cast<const float4*>(z + warp * 32 * E + v * 128 + lane * 4);
      atomicAdd(&s.bins[r * kBins + dist_bin(mx[r], q.x)], 1u);
      atomicAdd(&s.bins[r * kBins + dist_bin(mx[r], q.y)], 1u);
      atomicAdd(&s.bins[r * kBins + dist_bin(mx[r], q.z)], 1u);
      atomicAdd(&s.bins[r * kBins + dist_bin(mx[r], q.w)], 1u);
    }
  }
  csync(c);
  uint32_t* gb = s.gbins;                                  // [2][kBins] bins of the whole row
  if (c.nrank > 1) {
    for (int i = tid; i < 2 * kBins; i += VT) {
      uint32_t g = 0;
      if (kth[i / kBins] > 0) {
        const uint32_t addr = smem_u32(&s.bins[i]);
        for (uint32_t q = 0; q < c.nrank; ++q) g += dsmem_ld_u32(dsmem_addr(addr, q));
      }
      gb[i] = g;
    }
    __syncthreads();
  } else {
    gb = s.bins;
  }
  {
    // smallest bin whose cumulative count reaches k.  Two-level scan over the 2 x kBins bins:
    // in round `it` thread t holds entry it*VT + t of the [row][bin] array.
    constexpr int RPT = 2 * kBins / VT;
    constexpr int WPR = kBins / 32;                            // warps' worth of bins per row
    uint32_t cnt[RPT], incl[RPT];
    uint32_t* wtot = s.wtot;                                   // [2 * WPR] inclusive totals
#pragma unroll
    for (int it = 0; it < RPT; ++it) {
      const int g = it * VT + tid, r = g / kBins;
      cnt[it] = kth[r] > 0 ? gb[g] : 0u;
      incl[it] = cnt[it];
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_up_sync(0xffffffffu, incl[it], o);
        if (lane >= o) incl[it] += t;
      }
      if (lane == 31) wtot[it * VW + warp] = incl[it];
    }
    __syncthreads();
    // offsets of the warps' blocks within each row: every warp scans its row's WPR block totals
    // (WPR / 32 per lane), so no further barrier is needed
    constexpr int PL = WPR / 32;
#pragma unroll
    for (int it = 0; it < RPT; ++it) {
      const int g = it * VT + tid, r = g / kBins, bin = g % kBins, gw = it * VW + warp;
      uint32_t part[PL], lsum = 0;
#pragma unroll
      for (int i = 0; i < PL; ++i) { part[i] = wtot[r * WPR + lane * PL + i]; lsum += part[i]; }
      uint32_t linc = lsum;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_up_sync(0xffffffffu, linc, o);
        if (lane >= o) linc += t;
      }
      // blocks before block (gw - r*WPR): whole lanes before its lane, then the lane's own prefix
      const int blk = gw - r * WPR, bl = blk / PL, bo = blk % PL;
      uint32_t before = __shfl_sync(0xffffffffu, linc - lsum, bl);
#pragma unroll
      for (int i = 0; i < PL; ++i) {
        const uint32_t pv = __shfl_sync(0xffffffffu, part[i], bl);
        if (i < bo) before += pv;
      }
      const uint32_t need = static_cast<uint32_t>(kth[r] > 0 ? kth[r] : 0);
      const uint32_t hi = before + incl[it], lo_ = hi - cnt[it];
      if (kth[r] > 0 && lo_ < need && need <= hi) {
        s.sel[r * 2 + 0] = bin;
        s.sel[r * 2 + 1] = static_cast<int>(need - lo_);
      }
    }
  }
  __syncthreads();           // also: the staged bins have been consumed, candl may be overwritten
  int bstar[2], krem[2];
#pragma unroll
  for (int r = 0; r < 2; ++r) { bstar[r] = kth[r] > 0 ? s.sel[r * 2] : -1; krem[r] = kth[r] > 0 ? s.sel[r * 2 + 1] : 0; }
  // Entries of the located bin -> per-warp lists (ballot-compacted, no atomics): warp w keeps
  // up to kWarpCand entries of row r in wl[(r*VW + w)*kWarpCand ..] and their count in wcnt.
  constexpr int kWarpCand = kCandLocal / VW;
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    if (kth[r] <= 0) continue;
    const float* z = r ? z1 : z0;
    float* wl = s.wl + (r * VW + warp) * kWarpCand;
    // dist_bin(z) == bstar  <=>  bits(max - z) - lo_bits < span  (unsigned); the clamped end
    // bins take everything below / above
    const uint32_t lo_bits = bstar[r] == 0 ? 0u : static_cast<uint32_t>(bstar[r] + kBinBase) << kBinShift;
    const uint32_t hi_bits = bstar[r] == kBins - 1 ? 0xffffffffu : (static_cast<uint32_t>(bstar[r] + kBinBase + 1) << kBinShift) - 1u;
    const uint32_t span = hi_bits - lo_bits;
    const float mxr = mx[r];
    int run = 0;
#pragma unroll
    for (int v = 0; v < NV4; ++v) {
      const float4 q = *reinterpret_cast<const float4*>(z + warp * 32 * E + v * 128 + lane * 4);
      const float ev[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const bool match = (__float_as_uint(mxr - ev[e]) - lo_bits) <= span;
        const uint32_t m = __ballot_sync(0xffffffffu, match);
        if (m) {                                   // rare: a few entries per warp
          if (match) {
            const int pos = run + __popc(m & ((1u << lane) - 1u));
            if (pos < kWarpCand) wl[pos] = ev[e];
          }
          run += __popc(m);
        }
      }
    }
    if (lane == 0) s.wcnt[r * VW + warp] = run;
  }
  __syncthreads();
  int total[2] = {0, 0};
  bool fits[2] = {true, true};
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    if (kth[r] <= 0) continue;
    const int n = lane < VW ? s.wcnt[r * VW + lane] : 0;
    total[r] = __reduce_add_sync(0xffffffffu, n);
    if (__any_sync(0xffffffffu, n > kWarpCand)) fits[r] = false;
  }
  // compact the per-warp lists: every warp places its own entries behind those of the
  // warps before it
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    if (kth[r] <= 0) continue;
    const int n = lane < VW ? min(s.wcnt[r * VW + lane], kWarpCand) : 0;
    int incl = n;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += t;
    }
    const int my_off = __shfl_sync(0xffffffffu, incl - n, warp);
    const int my_n = __shfl_sync(0xffffffffu, n, warp);
    if (lane < my_n) s.comp[r * kCandLocal + my_off + lane] = s.wl[(r * VW + warp) * kWarpCand + lane];
    if (warp == 0 && lane == 31) s.cnts[r] = fits[r] ? incl : kCandLocal + 1;
  }
  csync(c);
  const float* cand_base = s.comp;             // [2][cand_stride] candidates of the whole row
  int cand_stride = kCandLocal;
  if (c.nrank > 1) {
    int* rc = s.cnts + 2;
    if (tid < 2 * static_cast<int>(c.nrank)) {
      const int r = tid / c.nrank, q = tid % c.nrank;
      rc[r * kMaxCluster + q] = static_cast<int>(dsmem_ld_u32(dsmem_addr(smem_u32(&s.cnts[r]), q)));
    }
    __syncthreads();
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      total[r] = 0;
      fits[r] = true;
      if (kth[r] <= 0) continue;
      for (uint32_t q = 0; q < c.nrank; ++q) {
        const int n = rc[r * kMaxCluster + q];
        if (n > kCandLocal) fits[r] = false;
        total[r] += n;
      }
      if (total[r] > kCandTotal) fits[r] = false;
    }
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      if (kth[r] <= 0 || !fits[r]) continue;
      int off = 0;
      for (uint32_t q = 0; q < c.nrank; ++q) {
        const int n = rc[r * kMaxCluster + q];
        const uint32_t base = dsmem_addr(smem_u32(&s.comp[r * kCandLocal]), q);
        for (int i = tid; i < n; i += VT) s.all[r * kCandTotal + off + i] = dsmem_ld_f32(base + 4u * i);
        off += n;
      }
    }
    __syncthreads();
    cand_base = s.all;
    cand_stride = kCandTotal;
  }
  // exact rank by counting: theta = v with #(> v) < k' <= #(>= v); eight lanes share the
  // comparisons of one candidate
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    if (kth[r] <= 0 || !fits[r]) continue;
    const float* al = cand_base + r * cand_stride;
    const int nc8 = (total[r] + (VT / 8) - 1) / (VT / 8) * (VT / 8);
    for (int i = tid >> 3; i < nc8; i += VT / 8) {
      const float v = i < total[r] ? al[i] : 0.f;
      int gt = 0, ge = 0;
      for (int t = tid & 7; t < total[r]; t += 8) {
        const float w = al[t];
        gt += (w > v);
        ge += (w >= v);
      }
#pragma unroll
      for (int o = 1; o < 8; o <<= 1) {
        gt += __shfl_xor_sync(0xffffffffu, gt, o);
        ge += __shfl_xor_sync(0xffffffffu, ge, o);
      }
      if (i < total[r] && (tid & 7) == 0 && gt < krem[r] && krem[r] <= ge) reinterpret_cast<float*>(s.sel)[4 + r] = v;
    }
  }
  __syncthreads();
#pragma unroll
  for (int r = 0; r < 2; ++r) theta[r] = (kth[r] > 0 && fits[r]) ? reinterpret_cast<float*>(s.sel)[4 + r] : -INFINITY;
  // ---- refinement when a bin holds too many entries: radix select (4 x 8 bits) on the
  // monotone key, restricted to that bin, rank krem within it
  for (int r = 0; r < 2; ++r) {
    if (kth[r] <= 0 || fits[r]) continue;        // same decision in every CTA of the row
    const float* z = r ? z1 : z0;
    uint32_t prefix = 0;
    int remaining = krem[r];
    for (int pass = 0; pass < 4; ++pass) {
      const int shift = 24 - 8 * pass;
      __syncthreads();
      if (tid < 256) s.bins[tid] = 0;
      __syncthreads();
      for (int v = 0; v < NV4; ++v) {
        const float4 q = *reinterpret_cast<const float4*>(z + warp * 32 * E + v * 128 + lane * 4);
        const float ev[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          if (dist_bin(mx[r], ev[e]) != bstar[r]) continue;
          const uint32_t key = float_key(ev[e]);
          if (pass == 0 || (key >> (shift + 8)) == prefix) atomicAdd(&s.bins[(key >> shift) & 255u], 1u);
        }
      }
      csync(c);
      uint32_t g = 0;
      if (tid < 256) {
        const uint32_t addr = smem_u32(&s.bins[tid]);
        for (uint32_t q = 0; q < c.nrank; ++q) g += dsmem_ld_u32(dsmem_addr(addr, q));
      }
      csync(c);               // every CTA has read the bins before anyone clears them again
      if (tid < 256) s.bins[256 + tid] = g;
      __syncthreads();
      if (tid == 0) {
        uint32_t run = 0;
        for (int dgt = 255; dgt >= 0; --dgt) {
          const uint32_t cnt = s.bins[256 + dgt];
          if (run < static_cast<uint32_t>(remaining) && static_cast<uint32_t>(remaining) <= run + cnt) {
            s.sel[6] = dgt;
            s.sel[7] = remaining - static_cast<int>(run);
            break;
          }
          run += cnt;
        }
      }
      __syncthreads();
      prefix = (prefix << 8) | static_cast<uint32_t>(s.sel[6]);
      remaining = s.sel[7];
    }
    theta[r] = key_float(prefix);
  }
  __syncthreads();
}


// One tree node (sequence b, node n): rows into shared memory, post-processing, sibling loop,
// resampling.  Returns the accepted child or -1 (the same value in every thread of the row's CTAs).
template <typename T, bool CFG, int E>
__device__ __forceinline__ int verify_node(const VerifyArgs& a, const int b, const int n, VCtx& c, const TopkSmem& tk,
                                            float* __restrict__ Q, float* __restrict__ P, float* __restrict__ U,
                                            int* misc, const uint32_t mbar_a, uint32_t& mphase, bool& bulk_ok, int* nbr_s) {
  constexpr int SL = VT * E;
  constexpr int NV4 = E / 4;                 // float4 per thread in a shared-memory sweep
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int fc = a.first_child[n], nc = a.n_child[n];
  const int lo = c.rank * SL;
  const int len = max(0, min(a.V - lo, SL));
  const long long row_off = static_cast<long long>(b) * a.seq_stride + static_cast<long long>(n) * a.row_stride;
  const int32_t* tok_b = a.tokens + static_cast<long long>(b) * a.N;
  const long long out_b = static_cast<long long>(b) * a.N;
  const uint32_t q_base = smem_u32(Q), p_base = smem_u32(P);
  const bool single = c.nrank == 1;

  // ---- stage the children's neighbour rows (bulk async copy when rows are 16-byte aligned)
  const bool want_nbr = nc > 0 && a.k > 0;
  bool bulk_issued = false;
  if (want_nbr && a.use_bulk && bulk_ok) {
    if (tid == 0) {
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
        for (int r = tid; r < a.k; r += VT)
          nbr_s[ci * a.kpad + r] = a.nbr[static_cast<long long>(code) * a.k_table + r];
    }
  }

  // ---- uniforms of this node (fetched early: off the critical path later)
  if (tid == 32) {
    float u;
    if (a.u_res) {
      u = a.u_res[out_b + n];
    } else {
      u = uniform_halfopen(philox_stream(a.seed, a.step, static_cast<uint32_t>(out_b + n), kStreamResample, 0).x);
    }
    reinterpret_cast<float*>(misc)[7] = u;
  }
  if (tid < nc) {
    float u;
    if (a.u_acc) {
      u = a.u_acc[out_b + fc + tid];
    } else {
      u = uniform_halfopen(philox_stream(a.seed, a.step, static_cast<uint32_t>(out_b + fc + tid), kStreamAccept, 0).x);
    }
    reinterpret_cast<float*>(misc)[8 + tid] = u;
  }

  // ---- read the rows once: every operand is copied asynchronously straight into shared
  // memory, target cond / uncond and drafter cond all in flight together; the drafter's uncond
  // row follows as soon as this thread has consumed its target chunks of U
  const bool masked = a.allow_lo > 0 || a.allow_hi < a.V;
  const T* tc = static_cast<const T*>(a.tc) + row_off;
  const T* tu = CFG ? static_cast<const T*>(a.tu) + row_off : nullptr;
  const T* dc = nc > 0 ? static_cast<const T*>(a.dc) + row_off : nullptr;
  const T* du = (CFG && nc > 0) ? static_cast<const T*>(a.du) + row_off : nullptr;
  issue_row<T, E>(tc, lo, len, Q);
  if (CFG) issue_row<T, E>(tu, lo, len, U);
  cp_async_commit();
  if (nc > 0) issue_row<T, E>(dc, lo, len, P);
  cp_async_commit();
  cp_async_wait<1>();
  float mx[2];
  mx[0] = finish_row<T, CFG, E>(tc, tu, a.g, a.inv_tau, lo, len, a.allow_lo, a.allow_hi, masked, Q, U);
  mx[1] = -INFINITY;
  if (nc > 0) {
    if (CFG) {
      issue_row<T, E>(du, lo, len, U);
      cp_async_commit();
    }
    cp_async_wait<0>();
    mx[1] = finish_row<T, CFG, E>(dc, du, a.g, a.inv_tau, lo, len, a.allow_lo, a.allow_hi, masked, P, U);
  }
  row_reduce<2, true>(c, mx);
  if (mx[0] == -INFINITY || (nc > 0 && mx[1] == -INFINITY)) {
    if (tid == 0 && c.rank == 0) vflag(a.status, LANTERN_DEV_EMPTY_ROW);
    if (mx[0] == -INFINITY) mx[0] = 0.f;
  }
  if (mx[1] == -INFINITY) mx[1] = 0.f;

  // ---- top-k truncation thresholds (exact)
  float theta[2] = {-INFINITY, -INFINITY};
  const int kth[2] = {(a.topk_t > 0 && a.topk_t < a.V) ? a.topk_t : 0,
                      (nc > 0 && a.topk_d > 0 && a.topk_d < a.V) ? a.topk_d : 0};
  const bool has_topk = kth[0] > 0 || kth[1] > 0;
  if (has_topk) topk_thresholds<E>(c, tk, Q, P, mx, kth, theta);

  // ---- softmax numerators 2^((z - max) log2 e) in place, row sums
  float sm[2] = {0.f, 0.f};
  {
    const float c0 = -mx[0] * kLog2e, c1 = -mx[1] * kLog2e;
#pragma unroll
    for (int v = 0; v < NV4; ++v) {
      const int j = warp * 32 * E + v * 128 + lane * 4;
      float4 q4 = *reinterpret_cast<const float4*>(Q + j);
      float ev[4] = {q4.x, q4.y, q4.z, q4.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        float x = ex2_approx(fmaf(ev[e], kLog2e, c0));
        if (has_topk) x = (ev[e] >= theta[0]) ? x : 0.f;
        ev[e] = x;
      }
      *reinterpret_cast<float4*>(Q + j) = make_float4(ev[0], ev[1], ev[2], ev[3]);
      sm[0] += (ev[0] + ev[1]) + (ev[2] + ev[3]);
    }
    if (nc > 0) {
#pragma unroll
      for (int v = 0; v < NV4; ++v) {
        const int j = warp * 32 * E + v * 128 + lane * 4;
        float4 p4 = *reinterpret_cast<const float4*>(P + j);
        float ev[4] = {p4.x, p4.y, p4.z, p4.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          float x = ex2_approx(fmaf(ev[e], kLog2e, c1));
          if (has_topk) x = (ev[e] >= theta[1]) ? x : 0.f;
          ev[e] = x;
        }
        *reinterpret_cast<float4*>(P + j) = make_float4(ev[0], ev[1], ev[2], ev[3]);
        sm[1] += (ev[0] + ev[1]) + (ev[2] + ev[3]);
      }
    }
  }
  row_reduce<2, false>(c, sm);     // its barrier also publishes Q and P
  float qs = sm[0] > 0.f ? 1.f / sm[0] : 0.f;
  float psum = sm[1];

  // ---- neighbour rows must have landed
  if (bulk_issued) {
    const bool ok = mbar_wait_bounded(mbar_a, mphase);
    if (__syncthreads_and(ok)) {
      mphase ^= 1u;
    } else {
      // The copy did not complete in time: the barrier's phase is still pending, so the barrier
      // is not touched again and this CTA stages every later table row with plain loads.  For
      // this node a late arrival writes the values that are re-read below anyway; if the CTA
      // goes on to other nodes (repair launch, path walk) a copy arriving that late could still
      // overwrite their rows, which is why the status bit is raised.
      bulk_ok = false;
      if (tid == 0) vflag(a.status, LANTERN_DEV_TIMEOUT);
      for (int ci = 0; ci < nc; ++ci) {
        int code = tok_b[fc + ci] - a.code_offset;
        if (code >= 0 && code < a.n_codes)
          for (int r = tid; r < a.k; r += VT)
            nbr_s[ci * a.kpad + r] = a.nbr[static_cast<long long>(code) * a.k_table + r];
      }
    }
  }
  __syncthreads();

  if (n == 0 && c.rank == 0 && tid == 0) {
    if (a.node_mass) a.node_mass[out_b] = -1.f;
    if (a.node_thresh) a.node_thresh[out_b] = -1.f;
  }

  // value of Q / P at a token of the row, wherever its slice lives
  auto row_at = [&](const float* loc, uint32_t base, int t) -> float {
    if (single) return loc[t];
    const uint32_t tr = static_cast<uint32_t>(t) / SL, to = static_cast<uint32_t>(t) - tr * SL;
    return dsmem_ld_f32(dsmem_addr(base + to * 4, tr));
  };

  // ---- sibling loop (Sec. 4; Eq. 1-2)
  int accepted = -1;
  for (int ci = 0; ci < nc; ++ci) {
    const int child = fc + ci;
    const int x = tok_b[child];
    bool skip = accepted >= 0 || x < 0 || x >= a.V;
    if (skip) {
      if (accepted < 0 && x >= a.V && tid == 0 && c.rank == 0) vflag(a.status, LANTERN_DEV_BAD_INDEX);
      if (c.rank == 0 && tid == 0) {
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
      // every CTA evaluates the relaxed mass redundantly (same values, same order, same result)
      const float qx = row_at(Q, q_base, x) * qs;
      const float pxraw = row_at(P, p_base, x);
      const float px = pxraw * ps;
      const float bound = a.delta > 0.f ? qx + a.delta : a.lambda * qx;      // Sec. 2.2 / Sec. 4
      float cum = qx;
      int nA = 0;
      bool bad = false, open = has_code;
      for (int base8 = 0; base8 < a.k && open; base8 += 256) {
        float qa[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {           // all loads of this lane first, then the scans
          const int r = base8 + i * 32 + lane;
          qa[i] = 0.f;
          if (r < a.k) {
            const int t = a.code_offset + nrow[r];
            if (t >= 0 && t < a.V) qa[i] = row_at(Q, q_base, t) * qs; else bad = true;
          }
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          if (!open) break;
          const int r = base8 + i * 32 + lane;
          if (base8 + i * 32 >= a.k) { open = false; break; }
          const float incl = warp_incl_scan(qa[i], lane);
          const bool ok = r < a.k && (cum + incl < bound);
          const uint32_t ballot = __ballot_sync(0xffffffffu, ok);
          const int ntake = __ffs(~ballot) - 1;          // leading accepted entries; -1 when all 32
          const int take = ntake < 0 ? 32 : ntake;
          if (take > 0) cum += __shfl_sync(0xffffffffu, incl, take - 1);
          nA += take;
          if (take < 32) open = false;
        }
      }
      if (__any_sync(0xffffffffu, bad) && lane == 0 && c.rank == 0) vflag(a.status, LANTERN_DEV_BAD_INDEX);
      const float m = cum;
      const float thr = px > 0.f ? fminf(1.f, m / px) : (m > 0.f ? 1.f : 0.f);
      const float u = reinterpret_cast<const float*>(misc)[8 + ci];
      if (lane == 0) {
        misc[0] = (u < thr) ? 1 : 0;
        misc[1] = nA;
        reinterpret_cast<float*>(misc)[2] = m;
        reinterpret_cast<float*>(misc)[3] = pxraw;
        if (c.rank == 0) {
          if (a.node_mass) a.node_mass[out_b + child] = m;
          if (a.node_thresh) a.node_thresh[out_b + child] = thr;
        }
      }
    }
    __syncthreads();
    const int acc = misc[0];
    const int nA = misc[1];
    const float m = reinterpret_cast<float*>(misc)[2];
    const float pxraw = reinterpret_cast<float*>(misc)[3];
    if (acc) {
      accepted = child;
      __syncthreads();       // misc is rewritten by the next tested child
      continue;
    }
    // ---- rejection: q~ (mass of A moved onto x), residual, drafter without x
    if (!single) cluster_sync();     // every CTA has finished reading q_cur / p_cur of this round
    const int xl = x - lo;                                   // position of x in this slice, if any
    for (int r = tid; r < nA; r += VT) {
      const int t = a.code_offset + nrow[r] - lo;
      if (t >= 0 && t < len && t != xl) Q[t] = 0.f;          // (a row that lists x itself: x is written below)
    }
    if (tid == 0 && xl >= 0 && xl < len) Q[xl] = qs > 0.f ? m / qs : 0.f;
    __syncthreads();
    // One sweep: Q <- [Q * rho - P]_+ with rho = qs * psum, i.e. the residual of Eq. 2 in the
    // (unnormalised) units of P; its sum gives the new scale.  The drafter mass left without
    // x is psum - P[x] unless that cancels badly, in which case it is summed in the sweep.
    const bool resum = pxraw > 0.5f * psum;
    const float rho = psum > 0.f ? qs * psum : qs;
    const int xj4 = (xl >= 0 && xl < len) ? (xl & ~3) : -1;
    float zs[2] = {0.f, 0.f};
#pragma unroll
    for (int v = 0; v < NV4; ++v) {
      const int j = warp * 32 * E + v * 128 + lane * 4;
      float4 q4 = *reinterpret_cast<const float4*>(Q + j);
      float4 p4 = *reinterpret_cast<const float4*>(P + j);
      q4.x = fmaxf(fmaf(q4.x, rho, -p4.x), 0.f);
      q4.y = fmaxf(fmaf(q4.y, rho, -p4.y), 0.f);
      q4.z = fmaxf(fmaf(q4.z, rho, -p4.z), 0.f);
      q4.w = fmaxf(fmaf(q4.w, rho, -p4.w), 0.f);
      *reinterpret_cast<float4*>(Q + j) = q4;
      zs[0] += (q4.x + q4.y) + (q4.z + q4.w);
      if (j == xj4) {                                        // drop x from the drafter
        P[xl] = 0.f;
        const int e = xl & 3;
        if (e == 0) p4.x = 0.f; else if (e == 1) p4.y = 0.f; else if (e == 2) p4.z = 0.f; else p4.w = 0.f;
      }
      if (resum) zs[1] += (p4.x + p4.y) + (p4.z + p4.w);
    }
    row_reduce<2, false>(c, zs);
    const float ps_old = ps;
    psum = resum ? zs[1] : psum - pxraw;
    if (zs[0] > 0.f) {
      qs = 1.f / zs[0];
    } else {
      // q~ <= p_cur everywhere: both sum to one, so q~ equals p_cur (before x was dropped);
      // keep it as the target
      float s2[2] = {0.f, 0.f};
#pragma unroll
      for (int v = 0; v < NV4; ++v) {
        const int j = warp * 32 * E + v * 128 + lane * 4;
        float4 p4 = *reinterpret_cast<const float4*>(P + j);
        if (j == xj4) {
          const int e = xl & 3;
          if (e == 0) p4.x = pxraw; else if (e == 1) p4.y = pxraw; else if (e == 2) p4.z = pxraw; else p4.w = pxraw;
        }
        *reinterpret_cast<float4*>(Q + j) = p4;
        s2[0] += (p4.x + p4.y) + (p4.z + p4.w);
      }
      row_reduce<2, false>(c, s2);       // leaves the per-warp and per-rank sums of Q in place
      qs = ps_old;
    }
  }

  // ---- no child accepted (or leaf): draw node_token from q_cur by inverse CDF in token order.
  // The last reduction left the per-warp sums of Q in c.last_red[w*2] and the per-rank sums in
  // c.gath[r*2]; the slice and the warp segment that hold the draw follow from those.
  if (accepted < 0) {
    __syncthreads();                      // c.gath was written by warp 0
    const float u = reinterpret_cast<const float*>(misc)[7];
    float total = 0.f;
    for (uint32_t r = 0; r < c.nrank; ++r) total += c.gath[r * 2];
    const float target = u * total;
    int owner = -1, last_pos = -1;
    float Erun = 0.f, E_owner = 0.f;
    for (uint32_t r = 0; r < c.nrank; ++r) {
      const float t = c.gath[r * 2];
      if (t > 0.f) last_pos = r;
      if (owner < 0 && Erun + t > target) { owner = r; E_owner = Erun; }
      Erun += t;
    }
    bool fallback = false;
    if (owner < 0) { owner = last_pos; fallback = true; }     // rounding pushed the target past the end
    if (owner == static_cast<int>(c.rank)) {
      // every warp finds the owner warp: lane w holds the sum of warp w's segment
      const float wt = lane < VW ? c.last_red[lane * 2] : 0.f;
      const float wincl = warp_incl_scan(wt, lane);
      const uint32_t hit = fallback ? 0u : __ballot_sync(0xffffffffu, E_owner + wincl > target);
      const uint32_t pos = __ballot_sync(0xffffffffu, wt > 0.f);
      int ow = hit ? __ffs(hit) - 1 : -1;
      bool wfallback = fallback;
      if (ow < 0) { ow = pos ? 31 - __clz(pos) : 0; wfallback = true; }
      const float Ew_owner = E_owner + __shfl_sync(0xffffffffu, wincl - wt, ow);
      if (warp == ow) {
        int found = -1;
        const int wlo = warp * 32 * E;
        if (!wfallback) {
          float runw = Ew_owner;
          for (int v = 0; v < NV4 && found < 0; ++v) {
            const int j = wlo + v * 128 + lane * 4;
            const float4 q4 = *reinterpret_cast<const float4*>(Q + j);
            const float s4 = (q4.x + q4.y) + (q4.z + q4.w);
            const float incl = warp_incl_scan(s4, lane);
            const uint32_t ballot = __ballot_sync(0xffffffffu, runw + incl > target);
            if (ballot) {
              const int src = __ffs(ballot) - 1;
              int cand = -1;
              if (lane == src) {
                float cc = runw + (incl - s4);
                const float ev[4] = {q4.x, q4.y, q4.z, q4.w};
                int lastp = -1;
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                  cc += ev[t];
                  if (ev[t] > 0.f) lastp = t;
                  if (cand < 0 && ev[t] > 0.f && cc > target) cand = t;
                }
                if (cand < 0) cand = lastp;
                cand = (cand >= 0) ? j + cand : -1;
              }
              found = __shfl_sync(0xffffffffu, cand, src);
              if (found < 0) found = -2;       // numerically empty quad: use the fallback below
            }
            runw += __shfl_sync(0xffffffffu, incl, 31);
          }
        }
        if (found < 0) {
          // last positive entry of this warp's segment
          int best = -1;
          for (int j = wlo + lane; j < wlo + 32 * E; j += 32)
            if (Q[j] > 0.f) best = j;
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) best = max(best, __shfl_xor_sync(0xffffffffu, best, o));
          found = best;
        }
        if (lane == 0) a.node_token[out_b + n] = found >= 0 ? lo + found : -1;
      }
    } else if (owner < 0 && c.rank == 0 && tid == 0) {
      a.node_token[out_b + n] = -1;      // empty distribution
      vflag(a.status, LANTERN_DEV_EMPTY_ROW);
    }
  } else if (c.rank == 0 && tid == 0) {
    a.node_token[out_b + n] = -1;
  }
  if (c.rank == 0 && tid == 0) a.node_next[out_b + n] = accepted;
  return accepted;
}

// E = row entries per thread; the CTA's slice holds SL = 1024 * E entries.
#ifndef LANTERN_MINB
#define LANTERN_MINB 1
#endif
template <typename T, bool CFG, int E>
__global__ void __launch_bounds__(VT, LANTERN_MINB) verify_nodes_kernel(const VerifyArgs a) {
  grid_dependency_sync();
  constexpr int SL = VT * E;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  float* Q = reinterpret_cast<float*>(smem_raw);
  float* P = Q + SL;
  float* U = P + SL;                                   // uncond staging (guidance only)
  unsigned char* nxt = reinterpret_cast<unsigned char*>(P + (CFG ? 2 : 1) * SL);
  unsigned char* scratch = reinterpret_cast<unsigned char*>(U);
  if (!scratch_aliases_u(CFG, E)) { scratch = nxt; nxt += kScratchBytes; }
  TopkSmem tk;
  tk.gbins = reinterpret_cast<uint32_t*>(scratch);
  tk.comp = reinterpret_cast<float*>(tk.gbins + 2 * kBins);
  tk.all = tk.comp + 2 * kCandLocal;
  tk.bins = reinterpret_cast<uint32_t*>(nxt);
  tk.wl = reinterpret_cast<float*>(tk.bins + 2 * kBins);
  tk.wcnt = reinterpret_cast<int*>(tk.wl + 2 * kCandLocal);
  tk.wtot = reinterpret_cast<uint32_t*>(tk.wcnt + 2 * VW);
  VCtx c;
  c.red = reinterpret_cast<float*>(tk.wtot + 2 * (kBins / 32));
  c.xch = c.red + 2 * VW * 4;
  c.gath = c.xch + 8;
  tk.sel = reinterpret_cast<int*>(c.gath + kMaxCluster * 4);
  tk.cnts = tk.sel + 8;
  int* misc = tk.cnts + kCntInts;
  uint64_t* mbar = reinterpret_cast<uint64_t*>(misc + kMiscInts);
  int* nbr_s = reinterpret_cast<int*>(mbar + 2);
  c.rank = cluster_ctarank();
  c.nrank = cluster_nctarank();
  c.parity = 0;
  c.last_red = c.red;

  const int tid = threadIdx.x;
  const uint32_t mbar_a = smem_u32(mbar);
  if (tid == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(mbar_a) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  uint32_t mphase = 0;
  bool bulk_ok = true;        // false after a bounded wait on the table-row copy has expired
  // A regular launch has one CTA (cluster) per node.  A repair launch (a.only given) has fewer:
  // cluster g of G takes the flagged nodes idx = g (mod G) one after another, and leaves at once
  // when none of them is flagged.
  const int rows = a.B * a.N, G = gridDim.x / c.nrank, g0 = blockIdx.x / c.nrank;
  if (a.lazy) {
    // Path walk (Sec. 2.1) instead of verifying every node: one cluster per sequence verifies the
    // root, moves to the accepted child and so on, so only the rows on the accepted path are
    // read.  The per-node results of the other nodes are not written.
    const int b = g0;
    const bool writer = c.rank == 0 && tid == 0;
    int32_t* ot = a.out_tokens + static_cast<long long>(b) * a.D1;
    int32_t* on = a.out_nodes + static_cast<long long>(b) * a.D1;
    int cur = 0, len = 0;
    for (;;) {
      const int acc = verify_node<T, CFG, E>(a, b, cur, c, tk, Q, P, U, misc, mbar_a, mphase, bulk_ok, nbr_s);
      csync(c);     // also orders the owner CTA's store of node_token before the read below
      if (acc <= cur || acc >= a.N || len >= a.D1 - 1) break;      // -1, or anything that is not a forward edge
      cur = acc;
      if (writer) { ot[len] = a.tokens[static_cast<long long>(b) * a.N + cur]; on[len] = cur; }
      ++len;
    }
    if (writer) {
      ot[len] = __ldcg(a.node_token + static_cast<long long>(b) * a.N + cur);
      on[len] = cur;
      a.accept_len[b] = len;
      for (int i = len + 1; i < a.D1; ++i) { ot[i] = -1; on[i] = -1; }
    }
    return;
  }
  bool work = true;
  if (a.only) {
    bool any = false;
    for (long long i = g0 + static_cast<long long>(tid) * G; i < rows; i += static_cast<long long>(VT) * G)
      any |= a.only[i] != 0;
    work = __syncthreads_or(any) != 0;       // the same flags, hence the same decision, in every CTA of a cluster
  }
  if (work) {
    for (int idx = g0; idx < rows; idx += G) {
      if (a.only && a.only[idx] == 0) continue;
      verify_node<T, CFG, E>(a, idx % a.B, a.order[idx / a.B], c, tk, Q, P, U, misc, mbar_a, mphase, bulk_ok, nbr_s);
      csync(c);     // peers may still be reading this CTA's shared memory; the next node overwrites it
    }
  }
  if (a.done) {
    // The CTA that finishes last (the counter wraps back to zero with it) walks every tree.
    __syncthreads();
    if (tid == 0) {
      __threadfence();
      const unsigned old = atomicInc(reinterpret_cast<unsigned*>(a.done), gridDim.x - 1);
      misc[0] = old == gridDim.x - 1 ? 1 : 0;
    }
    __syncthreads();
    if (misc[0]) {
      __threadfence();
      int32_t* stage = reinterpret_cast<int32_t*>(Q);          // Q and P: 2 * SL ints, free by now
      const int per_pass = max(1, SL / a.N);                    // sequences whose rows fit the stage
      for (int b0 = 0; b0 < a.B; b0 += per_pass)
        walk_staged(a.node_next, a.node_token, a.tokens, b0, min(per_pass, a.B - b0), a.N, a.D1, a.accept_len,
                    a.out_tokens, a.out_nodes, stage);
    }
  }
}

}  // namespace LANTERN_VNS
}  // namespace lantern
