// Relaxed verification of tree nodes whose rows are not truncated by top-k (Sec. 4; App. A.2
// Eq. 1-2; Sec. 2.1): streaming kernel, no row is ever held on chip or rewritten.
//
// The sibling loop of a node rejects children one after another; after r rejections the
// current target of every token j that was never a draft token nor a member of a set A is
//     q_r(j) = max(q_0(j) - alpha_r * p_0(j), 0) / beta_r,          p_r(j) = p_0(j) / W_r
// with three scalars per node (alpha_0 = 0, beta_0 = W_0 = 1): the nested positive parts of
// Eq. 2 collapse because every round subtracts a multiple of the same p_0,
//     alpha_{r+1} = alpha_r + beta_r / W_r,    beta_{r+1} = sum_j max(q_0(j) - alpha_{r+1} p_0(j), 0)
// (sum over the tokens outside the exception set below), W_{r+1} = W_r - p_0(x_r).  The tokens
// whose mass was moved (members of A) are zero from then on, and so is a rejected draft token
// x (rejection means m < p_cur(x), so its residual is empty): they form an exception set kept as
// a bitmap.  So the rows are streamed from HBM exactly once (one pass: sum of exponentials per
// row relative to a per-thread reference value), a rejection is one read-only reduction over
// both rows, served by L2, and the final draw re-reads one warp's range.  The values the
// sibling loop needs (q_0, p_0 at the draft tokens and at their neighbours) are gathered with
// 4-byte asynchronous copies issued before the streaming pass.
//
// One CTA of 256 threads per node, or a thread-block cluster of C CTAs when few nodes must fill
// the machine; warp w of CTA `rank` owns a contiguous range of 16-byte vectors of the row, so
// per-warp partial sums are sums over consecutive tokens and locate the inverse-CDF draw.
#pragma once
#include "rowops.cuh"

namespace lantern {
namespace stream {

#ifndef LANTERN_STREAM_THREADS
#define LANTERN_STREAM_THREADS 256
#endif
#ifndef LANTERN_STREAM_MINB
#define LANTERN_STREAM_MINB 4
#endif
#ifndef LANTERN_STREAM_PAD
#define LANTERN_STREAM_PAD 0
#endif
constexpr int ST = LANTERN_STREAM_THREADS;            // threads per CTA
constexpr int SW = ST / 32;        // warps per CTA
constexpr int kMaxV = 1 << 20;     // bitmap: V / 8 bytes of shared memory
constexpr int kSmallBytes = 2048 + LANTERN_STREAM_PAD;  // reductions, per-warp sums, scalars

// shared-memory bytes of one CTA
__host__ __device__ constexpr size_t smem_bytes(int V, int max_children, int kp1, bool cfg) {
  return static_cast<size_t>((V + 127) / 128) * 16                             // exception bitmap
         + static_cast<size_t>(max_children) * kp1 * ((cfg ? 4 : 2) + 1) * 4   // gathered words, token ids
         + kSmallBytes;
}

struct SCtx {
  uint32_t rank, nrank;
  int parity;
  float* red;    // [2][SW*4]
  float* xch;    // [2][4]
  float* gath;   // [kMaxCluster*4] per-CTA values of the last reduction
};

__device__ __forceinline__ void csync(const SCtx& c) {
  if (c.nrank > 1) cluster_sync(); else __syncthreads();
}

// v[] holds this warp's values (the same in every lane).  On return v[] holds the totals over
// the node's CTAs, identical in every thread (fixed combination order), and c.gath[r*NV+i] the
// per-CTA totals (valid in warp 0's lanes at once, for the others after the next barrier).
template <int NV, bool IS_MAX>
__device__ __forceinline__ void combine(SCtx& c, float (&v)[NV]) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  float* red = c.red + c.parity * (SW * 4);
  if (lane == 0) {
#pragma unroll
    for (int i = 0; i < NV; ++i) red[warp * NV + i] = v[i];
  }
  __syncthreads();
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    const float t = lane < SW ? red[lane * NV + i] : (IS_MAX ? -INFINITY : 0.f);
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
  } else if (warp == 0 && lane == 0) {
#pragma unroll
    for (int i = 0; i < NV; ++i) c.gath[i] = v[i];
  }
  c.parity ^= 1;
}

__device__ __forceinline__ void cp_async4(uint32_t dst, const void* src) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(src) : "memory");
}

// One row (cond and, with guidance, uncond) as a sequence of 16-byte vectors starting at token j0.
template <typename T, bool CFG, bool TAU1>
struct RowIO {
  using VT = Vec<T>;
  static constexpr int VN = VT::N;
  const T* c;
  const T* u;
  float g, it;
  int j0;
  __device__ __forceinline__ void load(int vec, uint4& rc, uint4& ru) const {
    rc = ldg_stream_u128(c + j0 + vec * VN);
    if (CFG) ru = ldg_stream_u128(u + j0 + vec * VN);
  }
  __device__ __forceinline__ float z1(float cc, float uu) const {
    if (CFG) return __fmul_rn(__fmaf_rn(g, __fsub_rn(cc, uu), uu), it);
    return TAU1 ? cc : __fmul_rn(cc, it);
  }
  __device__ __forceinline__ void z(const uint4& rc, const uint4& ru, float (&out)[VN]) const {
    float cf[VN], uf[VN];
    VT::unpack_raw(rc, cf);
    if (CFG) VT::unpack_raw(ru, uf);
#pragma unroll
    for (int e = 0; e < VN; ++e) out[e] = z1(cf[e], CFG ? uf[e] : 0.f);
  }
  __device__ __forceinline__ float z_at(int tok) const {        // scalar read of one token
    return z1(VT::widen(c[tok]), CFG ? VT::widen(u[tok]) : 0.f);
  }
};

// Geometry of a row: the allowed tokens [alo, ahi) are covered by nvec vectors from token j0;
// vectors [vi0, vi1) lie wholly inside and are read with 16-byte loads, the at most two ragged
// ones with scalar loads.  Warp gw owns vectors [gw*vw, (gw+1)*vw).
struct Geo {
  int alo, ahi, j0, nvec, vi0, vi1, vw;
};
// the ragged vector on side 0 (front) / 1 (back) of the row, if there is one
__device__ __forceinline__ bool ragged_vec(const Geo& ge, int side, int& vv) {
  if (side == 0) { vv = 0; return ge.vi0 > 0; }
  vv = ge.nvec - 1;
  return ge.vi1 < ge.nvec;      // (a single vector ragged on both sides counts as the front one)
}

// Sum of exponentials of one vector relative to the thread's reference m (s is scaled by
// 2^(-m log2 e)); the reference is the first finite value seen and moves only when a vector's sum gets huge.
template <int VN>
__device__ __forceinline__ void acc_exp(const float (&z)[VN], float& m, float& s) {
  if (m == -INFINITY) {
    float bm = z[0];
#pragma unroll
    for (int e = 1; e < VN; ++e) bm = fmaxf(bm, z[e]);
    if (bm == -INFINITY) return;
    m = bm;
  }
  float c0 = -m * kLog2e;
  float s0 = 0.f, s1 = 0.f;
#pragma unroll
  for (int e = 0; e < VN; e += 2) {
    s0 += ex2_approx(fmaf(z[e], kLog2e, c0));
    s1 += ex2_approx(fmaf(z[e + 1], kLog2e, c0));
  }
  float sb = s0 + s1;
  if (!(sb < 1e30f)) {             // an entry far above the reference: move the reference
    float bm = z[0];
#pragma unroll
    for (int e = 1; e < VN; ++e) bm = fmaxf(bm, z[e]);
    s *= ex2_approx((m - bm) * kLog2e);
    m = bm;
    c0 = -m * kLog2e;
    sb = 0.f;
#pragma unroll
    for (int e = 0; e < VN; ++e) sb += ex2_approx(fmaf(z[e], kLog2e, c0));
  }
  s += sb;
}

// the ragged first / last vector of a row, read by lane 0 of the warp that owns it
template <typename IO>
__device__ __forceinline__ void edge_sum(const IO& io, const Geo& ge, int vbeg, int vend, float& m, float& s) {
  constexpr int VN = IO::VN;
#pragma unroll
  for (int side = 0; side < 2; ++side) {
    int vv;
    if (!ragged_vec(ge, side, vv) || vv < vbeg || vv >= vend) continue;
    float z[VN];
#pragma unroll
    for (int e = 0; e < VN; ++e) {
      const int t = ge.j0 + vv * VN + e;
      z[e] = (t >= ge.alo && t < ge.ahi) ? io.z_at(t) : -INFINITY;
    }
    acc_exp<VN>(z, m, s);
  }
}

// Parameters of the current target in units of the first pass:
//   term_j = max(2^(zq_j L + cq) * aq - 2^(zp_j L + cp) * ap, 0)     (0 for exception tokens)
struct Cur {
  float cq, cp, aq, ap;
  bool has_p;
};

struct StreamSmem {
  uint32_t* bits;   // [ceil(V/32)] exception bitmap (members of the sets A and rejected draft tokens)
  float* ent;       // [nc][kp1][NOPS] gathered raw words, then (q_0, p_0) in words 0, 1
  int* tok;         // [nc][kp1] token ids of the gathered entries (entry 0: the draft token), -1 = invalid
  float* wpart;     // [SW] per-warp sums of the current target (committed)
  float* wtmp;      // [SW] per-warp sums of the pass in flight
  float* rtot;      // [kMaxCluster] per-CTA sums of the current target (committed)
  float* scan;      // [SW]
  int* misc;        // [32]
  uint32_t* memb;   // [33] greedy-skip rule: bit r = entry r of the neighbour list joined A
};

// term of every token of vector vv under the current target (exception and masked tokens: 0)
template <typename IO>
__device__ __forceinline__ void vec_terms(const IO& ioq, const IO& iop, const Geo& ge, const Cur& k,
                                          const uint32_t* __restrict__ bits, int vv, float (&out)[IO::VN]) {
  constexpr int VN = IO::VN;
  const int j = ge.j0 + vv * VN;
  float zq[VN], zp[VN];
  if (vv >= ge.vi0 && vv < ge.vi1) {
    uint4 rc, ru;
    ioq.load(vv, rc, ru);
    ioq.z(rc, ru, zq);
    if (k.has_p) { iop.load(vv, rc, ru); iop.z(rc, ru, zp); }
  } else {
#pragma unroll
    for (int e = 0; e < VN; ++e) {
      const bool in = j + e >= ge.alo && j + e < ge.ahi;
      zq[e] = in ? ioq.z_at(j + e) : -INFINITY;
      zp[e] = (in && k.has_p) ? iop.z_at(j + e) : -INFINITY;
    }
  }
  const uint32_t ex = (bits[j >> 5] >> (j & 31)) & ((1u << VN) - 1u);
#pragma unroll
  for (int e = 0; e < VN; ++e) {
    const float x = ex2_approx(fmaf(zq[e], kLog2e, k.cq)) * k.aq;
    float t = x;
    if (k.has_p) t = fmaxf(fmaf(-ex2_approx(fmaf(zp[e], kLog2e, k.cp)), k.ap, x), 0.f);
    out[e] = ((ex >> e) & 1u) ? 0.f : t;
  }
}

// Rejection pass: sum of term_j over this thread's share of warp range [vbeg, vend), skipping
// the exception tokens; with RESUM also the sum of 2^(zp L + cp) over the tokens not dropped
// from the drafter.
template <typename IO, int U, bool RESUM, bool HASP = true>
__device__ __forceinline__ void pass_residual(const IO& ioq, const IO& iop, const Geo& ge, int vbeg, int vend, int lane,
                                              const Cur& k, const uint32_t* __restrict__ bits,
                                              const int* __restrict__ dropped, int n_dropped, float& acc, float& accp) {
  constexpr int VN = IO::VN;
  const int hb = max(vbeg, ge.vi0), he = min(vend, ge.vi1);
  float a0 = 0.f, a1 = 0.f, p0 = 0.f, p1 = 0.f;
  // Backwards: the end of the range was streamed last, so it is what L2 still holds.
  const int n_it = he > hb ? (he - hb + 32 * U - 1) / (32 * U) : 0;
  for (int it = n_it - 1; it >= 0; --it) {
    const int base = hb + it * 32 * U;
    uint4 qc[U], qu[U], pc[U], pu[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int vv = base + 32 * u + lane;
      if (vv < he) {
        ioq.load(vv, qc[u], qu[u]);
        if (HASP) iop.load(vv, pc[u], pu[u]);
      }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int vv = base + 32 * u + lane;
      if (vv < he) {
        float zq[VN], zp[VN];
        ioq.z(qc[u], qu[u], zq);
        if (HASP) iop.z(pc[u], pu[u], zp);
        const int j = ge.j0 + vv * VN;
        const uint32_t ex = (bits[j >> 5] >> (j & 31)) & ((1u << VN) - 1u);
        if (ex == 0u) {
#pragma unroll
          for (int e = 0; e < VN; e += 2) {
            const float x0 = ex2_approx(fmaf(zq[e], kLog2e, k.cq)) * k.aq;
            const float y0 = HASP ? ex2_approx(fmaf(zp[e], kLog2e, k.cp)) : 0.f;
            const float x1 = ex2_approx(fmaf(zq[e + 1], kLog2e, k.cq)) * k.aq;
            const float y1 = HASP ? ex2_approx(fmaf(zp[e + 1], kLog2e, k.cp)) : 0.f;
            a0 += fmaxf(fmaf(-y0, k.ap, x0), 0.f);
            a1 += fmaxf(fmaf(-y1, k.ap, x1), 0.f);
            if (RESUM) { p0 += y0; p1 += y1; }
          }
        } else {
#pragma unroll
          for (int e = 0; e < VN; ++e) {
            const float y = HASP ? ex2_approx(fmaf(zp[e], kLog2e, k.cp)) : 0.f;
            if (!((ex >> e) & 1u)) {
              const float x = ex2_approx(fmaf(zq[e], kLog2e, k.cq)) * k.aq;
              a0 += fmaxf(fmaf(-y, k.ap, x), 0.f);
              if (RESUM) p0 += y;
            } else if (RESUM) {
              bool gone = false;
              for (int d = 0; d < n_dropped; ++d) gone |= dropped[d] == j + e;
              if (!gone) p0 += y;
            }
          }
        }
      }
    }
  }
  if (lane == 0) {
#pragma unroll
    for (int side = 0; side < 2; ++side) {
      int vv;
      if (!ragged_vec(ge, side, vv) || vv < vbeg || vv >= vend) continue;
      for (int e = 0; e < VN; ++e) {
        const int t = ge.j0 + vv * VN + e;
        if (t < ge.alo || t >= ge.ahi) continue;
        const float y = HASP ? ex2_approx(fmaf(iop.z_at(t), kLog2e, k.cp)) : 0.f;
        const bool ex = (bits[t >> 5] >> (t & 31)) & 1u;
        if (!ex) {
          const float x = ex2_approx(fmaf(ioq.z_at(t), kLog2e, k.cq)) * k.aq;
          a0 += fmaxf(fmaf(-y, k.ap, x), 0.f);
          if (RESUM) p0 += y;
        } else if (RESUM) {
          bool gone = false;
          for (int d = 0; d < n_dropped; ++d) gone |= dropped[d] == t;
          if (!gone) p0 += y;
        }
      }
    }
  }
  acc = a0 + a1;
  accp = p0 + p1;
}

// One tree node (sequence b, node n).  Returns the accepted child or -1, the same value in
// every thread of the node's CTAs.
// VAR: the acceptance-rule variants (greedy-skip subset, deterministic drafts) are compiled in.
template <typename T, bool CFG, bool TAU1, bool VAR>
__device__ __forceinline__ int stream_node(const VerifyArgs& a, const int b, const int n, SCtx& c, const StreamSmem& sm) {
  using IO = RowIO<T, CFG, TAU1>;
  constexpr int VN = IO::VN;
  constexpr int NOPS = CFG ? 4 : 2;
  constexpr int U1 = CFG ? 2 : 4;       // vectors in flight per thread and operand, single row
  constexpr int U2 = CFG ? 1 : 2;       // ... when two rows are read together
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int toff = VAR ? b * a.tree_stride : 0;            // a forest keeps one set of tree arrays per sequence
  const int fc = a.first_child[toff + n], nc = a.n_child[toff + n];
  const long long row_off = static_cast<long long>(b) * a.seq_stride + static_cast<long long>(n) * a.row_stride;
  const int32_t* tok_b = a.tokens + static_cast<long long>(b) * a.N;
  const long long out_b = static_cast<long long>(b) * a.N;
  const int kp1 = a.k + 1;
  const bool writer = c.rank == 0 && tid == 0;
  const bool det = VAR && a.det != 0;       // deterministic drafts (Sec. 3): p(x) = 1, no drafter row
  const bool skip = VAR && a.skip != 0;     // greedy-skip subset rule
  const bool has_p = nc > 0 && !det;
  float* fm = reinterpret_cast<float*>(sm.misc);
  int* dropped = sm.misc + 16;          // [LANTERN_MAX_CHILDREN] rejected draft tokens

  Geo ge;
  ge.alo = a.allow_lo; ge.ahi = a.allow_hi;
  ge.j0 = ge.alo / VN * VN;
  ge.nvec = (ge.ahi - ge.j0 + VN - 1) / VN;
  ge.vi0 = ge.alo > ge.j0 ? 1 : 0;
  ge.vi1 = (ge.j0 + ge.nvec * VN > ge.ahi) ? ge.nvec - 1 : ge.nvec;
  if (ge.vi1 < ge.vi0) ge.vi1 = ge.vi0;
  const int nwarps = static_cast<int>(c.nrank) * SW;
  ge.vw = ((ge.nvec + nwarps - 1) / nwarps + 31) / 32 * 32;
  const int gw = static_cast<int>(c.rank) * SW + warp;
  const int vbeg = min(gw * ge.vw, ge.nvec), vend = min(vbeg + ge.vw, ge.nvec);

  IO ioq, iop;
  ioq.c = static_cast<const T*>(a.tc) + row_off;
  ioq.u = CFG ? static_cast<const T*>(a.tu) + row_off : nullptr;
  ioq.g = a.g; ioq.it = a.inv_tau; ioq.j0 = ge.j0;
  iop = ioq;
  iop.c = has_p ? static_cast<const T*>(a.dc) + row_off : nullptr;
  iop.u = (CFG && has_p) ? static_cast<const T*>(a.du) + row_off : nullptr;

  // ---- exception bitmap, uniforms
  {
    const int words = (a.V + 31) / 32;
    for (int i = tid; i < words; i += ST) sm.bits[i] = 0u;
  }
  if (tid == 32) {
    fm[7] = a.u_res ? a.u_res[out_b + n]
                    : uniform_halfopen(philox_stream(a.seed, a.step, static_cast<uint32_t>(out_b + n), kStreamResample, 0).x);
  }
  if (tid < nc) {
    fm[8 + tid] = a.u_acc ? a.u_acc[out_b + fc + tid]
                          : uniform_halfopen(philox_stream(a.seed, a.step, static_cast<uint32_t>(out_b + fc + tid), kStreamAccept, 0).x);
  }
  // ---- gather: raw logits at every draft token and at its neighbours, 4-byte asynchronous
  // copies into shared memory (in flight during the streaming pass).  The children's tokens are
  // staged first; the entries (child, list position) are then spread over all threads, four per
  // thread at a time with their table reads issued together, so the chain token -> neighbour ->
  // logit is walked once per node, not once per child.
  int* ctok = sm.misc + 24;               // [LANTERN_MAX_CHILDREN] the children's draft tokens
  if (tid < nc) ctok[tid] = tok_b[fc + tid];
  __syncthreads();
  bool bad = false;
  const int n_ent = nc * kp1;
  for (int e0 = tid; e0 < n_ent; e0 += 4 * ST) {
    int tt[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int e = e0 + i * ST;
      tt[i] = -2;                                             // no such entry
      if (e < n_ent) {
        const int ci = e / kp1, r = e - ci * kp1;
        const int x = ctok[ci];
        const int code = x - a.code_offset;
        if (x >= 0 && x < a.V) {
          if (r == 0) tt[i] = x;
          else if (a.k > 0 && code >= 0 && code < a.n_codes)
            tt[i] = a.code_offset + __ldg(a.nbr + static_cast<long long>(code) * a.k_table + (r - 1));
        }
      }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int e = e0 + i * ST;
      if (e >= n_ent) continue;
      const int t = tt[i];
      const bool ok = t >= 0 && t < a.V;
      bad |= !ok && t != -2;
      sm.tok[e] = ok ? t : -1;
      if (ok) {
        const int w = sizeof(T) == 4 ? t : (t & ~1);
        const uint32_t dst = smem_u32(sm.ent + e * NOPS);
        cp_async4(dst, ioq.c + w);
        if (has_p) cp_async4(dst + 4, iop.c + w);
        if (CFG) {
          cp_async4(dst + 8, ioq.u + w);
          if (has_p) cp_async4(dst + 12, iop.u + w);
        }
      }
    }
  }
  cp_async_commit();
  if (bad) vflag(a.status, LANTERN_DEV_BAD_INDEX);

  // ---- first pass: the rows are streamed once
  float mx[2] = {-INFINITY, -INFINITY}, sx[2] = {0.f, 0.f};
  {
    const int hb = max(vbeg, ge.vi0), he = min(vend, ge.vi1);
    if (has_p) {
      // the two rows alternate in the instruction stream so that both are in flight
      for (int base = hb; base < he; base += 32 * U2) {
        uint4 qc[U2], qu[U2], pc[U2], pu[U2];
#pragma unroll
        for (int u = 0; u < U2; ++u) {
          const int vv = base + 32 * u + lane;
          if (vv < he) { ioq.load(vv, qc[u], qu[u]); iop.load(vv, pc[u], pu[u]); }
        }
#pragma unroll
        for (int u = 0; u < U2; ++u) {
          const int vv = base + 32 * u + lane;
          if (vv < he) {
            float z[VN];
            ioq.z(qc[u], qu[u], z);
            acc_exp<VN>(z, mx[0], sx[0]);
            iop.z(pc[u], pu[u], z);
            acc_exp<VN>(z, mx[1], sx[1]);
          }
        }
      }
    } else {
      for (int base = hb; base < he; base += 32 * U1) {
        uint4 qc[U1], qu[U1];
#pragma unroll
        for (int u = 0; u < U1; ++u) {
          const int vv = base + 32 * u + lane;
          if (vv < he) ioq.load(vv, qc[u], qu[u]);
        }
#pragma unroll
        for (int u = 0; u < U1; ++u) {
          const int vv = base + 32 * u + lane;
          if (vv < he) {
            float z[VN];
            ioq.z(qc[u], qu[u], z);
            acc_exp<VN>(z, mx[0], sx[0]);
          }
        }
      }
    }
    if (lane == 0) {
      edge_sum(ioq, ge, vbeg, vend, mx[0], sx[0]);
      if (has_p) edge_sum(iop, ge, vbeg, vend, mx[1], sx[1]);
    }
  }
  // one combination for both rows: per-warp (reference, sum) pairs -> CTA -> cluster; the sums are
  // rescaled to the common reference in a fixed order, so every thread gets the same values
  float gm[2], ws[2];
  {
    float wm[2] = {warp_max(mx[0]), warp_max(mx[1])};
    float wsum[2];
#pragma unroll
    for (int i = 0; i < 2; ++i)
      wsum[i] = warp_sum(mx[i] == -INFINITY ? 0.f : sx[i] * ex2_approx((mx[i] - wm[i]) * kLog2e));
    float* red = c.red + c.parity * (SW * 4);
    if (lane == 0) { red[warp * 4] = wm[0]; red[warp * 4 + 1] = wsum[0]; red[warp * 4 + 2] = wm[1]; red[warp * 4 + 3] = wsum[1]; }
    __syncthreads();
    float cm[2] = {-INFINITY, -INFINITY}, cs2[2] = {0.f, 0.f};
    for (int w2 = 0; w2 < SW; ++w2) { cm[0] = fmaxf(cm[0], red[w2 * 4]); cm[1] = fmaxf(cm[1], red[w2 * 4 + 2]); }
    for (int w2 = 0; w2 < SW; ++w2) {
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        const float m2 = red[w2 * 4 + 2 * i];
        if (m2 != -INFINITY) cs2[i] += red[w2 * 4 + 2 * i + 1] * ex2_approx((m2 - cm[i]) * kLog2e);
      }
    }
    gm[0] = cm[0]; gm[1] = cm[1]; ws[0] = cs2[0]; ws[1] = cs2[1];
    if (c.nrank > 1) {
      if (tid == 0) { c.xch[c.parity * 4] = cm[0]; c.xch[c.parity * 4 + 1] = cs2[0]; c.xch[c.parity * 4 + 2] = cm[1]; c.xch[c.parity * 4 + 3] = cs2[1]; }
      cluster_sync();
      float rm[2] = {-INFINITY, -INFINITY}, rs[2] = {0.f, 0.f};
      for (uint32_t r = 0; r < c.nrank; ++r) {
        const uint32_t base = dsmem_addr(smem_u32(&c.xch[c.parity * 4]), r);
        const float v0 = dsmem_ld_f32(base), v1 = dsmem_ld_f32(base + 4), v2 = dsmem_ld_f32(base + 8), v3 = dsmem_ld_f32(base + 12);
        if (tid == 0) { c.gath[r * 4] = v0; c.gath[r * 4 + 1] = v1; c.gath[r * 4 + 2] = v2; c.gath[r * 4 + 3] = v3; }
        rm[0] = fmaxf(rm[0], v0); rm[1] = fmaxf(rm[1], v2);
      }
      for (uint32_t r = 0; r < c.nrank; ++r) {
        const uint32_t base = dsmem_addr(smem_u32(&c.xch[c.parity * 4]), r);
        const float v0 = dsmem_ld_f32(base), v1 = dsmem_ld_f32(base + 4), v2 = dsmem_ld_f32(base + 8), v3 = dsmem_ld_f32(base + 12);
        if (v0 != -INFINITY) rs[0] += v1 * ex2_approx((v0 - rm[0]) * kLog2e);
        if (v2 != -INFINITY) rs[1] += v3 * ex2_approx((v2 - rm[1]) * kLog2e);
      }
      gm[0] = rm[0]; gm[1] = rm[1]; ws[0] = rs[0]; ws[1] = rs[1];
    }
    // commit: the current target is q_0 (unnormalised, relative to gm[0])
    if (tid < SW) {
      const float m2 = red[tid * 4];
      sm.wpart[tid] = m2 == -INFINITY ? 0.f : red[tid * 4 + 1] * ex2_approx((m2 - gm[0]) * kLog2e);
    }
    if (tid < static_cast<int>(c.nrank)) {
      if (c.nrank > 1) {
        const uint32_t base = dsmem_addr(smem_u32(&c.xch[c.parity * 4]), tid);
        const float v0 = dsmem_ld_f32(base), v1 = dsmem_ld_f32(base + 4);
        sm.rtot[tid] = v0 == -INFINITY ? 0.f : v1 * ex2_approx((v0 - gm[0]) * kLog2e);
      } else {
        sm.rtot[0] = ws[0];
      }
    }
    c.parity ^= 1;
  }
  if (gm[0] == -INFINITY || (has_p && gm[1] == -INFINITY)) {
    if (writer) vflag(a.status, LANTERN_DEV_EMPTY_ROW);
  }
  if (gm[0] == -INFINITY) gm[0] = 0.f;
  if (gm[1] == -INFINITY) gm[1] = 0.f;
  const float rq = ws[0] > 0.f ? 1.f / ws[0] : 0.f;
  const float rp = ws[1] > 0.f ? 1.f / ws[1] : 0.f;
  Cur cur;
  cur.cq = -gm[0] * kLog2e; cur.cp = -gm[1] * kLog2e; cur.aq = 1.f; cur.ap = 0.f; cur.has_p = false;

  if (n == 0 && writer) {
    if (a.node_mass) a.node_mass[out_b] = -1.f;
    if (a.node_thresh) a.node_thresh[out_b] = -1.f;
  }

  // ---- gathered words -> (q_0, p_0) of every draft token and neighbour
  cp_async_wait<0>();
  __syncthreads();
  for (int e = tid; e < n_ent; e += ST) {
    const int t = sm.tok[e];
    float q0 = 0.f, p0 = 0.f;
    if (t >= ge.alo && t < ge.ahi) {
      const uint32_t* w = reinterpret_cast<const uint32_t*>(sm.ent + e * NOPS);
      float v[4];
#pragma unroll
      for (int o = 0; o < NOPS; ++o) {
        const uint32_t raw = w[o];
        v[o] = sizeof(T) == 4 ? __uint_as_float(raw) : __uint_as_float((t & 1) ? (raw & 0xffff0000u) : (raw << 16));
      }
      const float zq = ioq.z1(v[0], CFG ? v[2] : 0.f);
      q0 = ex2_approx(fmaf(zq, kLog2e, cur.cq)) * rq;
      if (has_p) p0 = ex2_approx(fmaf(ioq.z1(v[1], CFG ? v[3] : 0.f), kLog2e, cur.cp)) * rp;
    }
    sm.ent[e * NOPS] = q0;
    sm.ent[e * NOPS + 1] = p0;
  }
  __syncthreads();

  // ---- sibling loop (Sec. 4; Eq. 1-2) on the scalars alpha, beta, W
  float alpha = 0.f, beta = 1.f, ibeta = 1.f, W = 1.f, iW = 1.f;
  int n_dropped = 0;
  int accepted = -1;
  for (int ci = 0; ci < nc; ++ci) {
    const int child = fc + ci;
    const int x = ctok[ci];
    if (accepted >= 0 || x < 0 || x >= a.V) {
      if (accepted < 0 && x >= a.V && writer) vflag(a.status, LANTERN_DEV_BAD_INDEX);
      if (writer) {
        if (a.node_mass) a.node_mass[out_b + child] = -1.f;
        if (a.node_thresh) a.node_thresh[out_b + child] = -1.f;
      }
      continue;
    }
    const int code = x - a.code_offset;
    const bool has_code = a.k > 0 && code >= 0 && code < a.n_codes;
    const float* en = sm.ent + ci * kp1 * NOPS;
    const int* tk = sm.tok + ci * kp1;
    bool x_dropped = false;
    for (int d = 0; d < n_dropped; ++d) x_dropped |= dropped[d] == x;
    // current target at entry r: exception tokens are zero
    auto val = [&](int r) -> float {
      const int t = tk[r];
      if (t < 0) return 0.f;
      if ((sm.bits[t >> 5] >> (t & 31)) & 1u) return 0.f;
      return fmaxf(fmaf(-alpha, en[r * NOPS + 1], en[r * NOPS]), 0.f) * ibeta;
    };
    // Prefix rule over lists of up to 32 * SW entries, all warps at once: warp w scans entries
    // [32w, 32w + 32); with the sums of the warps before it (added in list order, as the one-warp
    // loop below does) it finds its first entry that would break the bound; the first warp that
    // has one ends the prefix.
    const bool par = has_code && !skip && a.k <= 32 * SW;
    float* pcum = reinterpret_cast<float*>(sm.memb + 8);          // (the member mask is unused without skip)
    if (par) {
      const int r = warp * 32 + lane;
      const float incl = warp_incl_scan(r < a.k ? val(1 + r) : 0.f, lane);
      if (lane == 31) sm.scan[warp] = incl;
      __syncthreads();
      const float qx = val(0);
      const float bound = a.delta > 0.f ? qx + a.delta : a.lambda * qx;
      float base = qx;
      for (int w2 = 0; w2 < warp; ++w2) base += sm.scan[w2];
      const uint32_t ballot = __ballot_sync(0xffffffffu, r < a.k && (base + incl < bound));
      const int ntake = __ffs(~ballot) - 1;
      const int take = ntake < 0 ? 32 : ntake;
      const float upto = take > 0 ? base + __shfl_sync(0xffffffffu, incl, take - 1) : base;
      if (lane == 0) { sm.memb[warp] = static_cast<uint32_t>(take); pcum[warp] = upto; }
      __syncthreads();
    }
    if (warp == 0) {
      const float qx = val(0);
      const float px = det ? 1.f : (x_dropped ? 0.f : en[1] * iW);
      const float bound = a.delta > 0.f ? qx + a.delta : a.lambda * qx;      // Sec. 2.2 / Sec. 4
      float cum = qx;
      int nA = 0;
      bool open = has_code;
      if (par) {
        for (int w2 = 0; w2 < SW && open; ++w2) {
          const int take = static_cast<int>(sm.memb[w2]);
          nA += take;
          cum = pcum[w2];
          if (take < 32) open = false;
        }
        open = false;
      }
      if (skip && open) {
        // greedy-skip rule: a neighbour that would break the bound is passed over and the list
        // is searched on; the running sum is sequential, 32 entries at a time through shuffles
        for (int base = 0; base < a.k; base += 32) {
          const int r = base + lane;
          const float v = r < a.k ? val(1 + r) : 0.f;
          uint32_t mask = 0u;
          const int lim = min(32, a.k - base);
          for (int i = 0; i < lim; ++i) {
            const float vi = __shfl_sync(0xffffffffu, v, i);
            if (cum + vi < bound) { cum += vi; mask |= 1u << i; }
          }
          if (lane == 0) sm.memb[base >> 5] = mask;
          nA += __popc(mask);
        }
        open = false;
      }
      for (int base8 = 0; base8 < a.k && open; base8 += 256) {
        float qa[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int r = base8 + i * 32 + lane;
          qa[i] = r < a.k ? val(1 + r) : 0.f;
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
      const float m = cum;
      const float thr = px > 0.f ? fminf(1.f, m / px) : (m > 0.f ? 1.f : 0.f);
      const float u = fm[8 + ci];
      if (lane == 0) {
        sm.misc[0] = (u < thr) ? 1 : 0;
        sm.misc[1] = nA;
        fm[2] = px;
        if (c.rank == 0) {
          if (a.node_mass) a.node_mass[out_b + child] = m;
          if (a.node_thresh) a.node_thresh[out_b + child] = thr;
        }
      }
    }
    __syncthreads();
    const int acc = sm.misc[0];
    const int nA = sm.misc[1];
    const float px = fm[2];
    if (acc) {
      accepted = child;
      __syncthreads();       // misc is rewritten by the next tested child
      continue;
    }
    // ---- rejection: the members of A and x join the exception set; x leaves the drafter
    if (skip) {
      if (has_code) {
        for (int r = tid; r < a.k; r += ST) {
          const int t = tk[1 + r];
          if (t >= 0 && ((sm.memb[r >> 5] >> (r & 31)) & 1u)) atomicOr(&sm.bits[t >> 5], 1u << (t & 31));
        }
      }
    } else {
      for (int r = tid; r < nA; r += ST) {
        const int t = tk[1 + r];
        if (t >= 0) atomicOr(&sm.bits[t >> 5], 1u << (t & 31));
      }
    }
    if (tid == 0) {
      atomicOr(&sm.bits[x >> 5], 1u << (x & 31));
      if (!x_dropped) dropped[n_dropped] = x;
    }
    if (!x_dropped) ++n_dropped;
    __syncthreads();
    const float alpha_n = fmaf(beta, iW, alpha);
    Cur nx;
    nx.cq = cur.cq; nx.cp = cur.cp; nx.aq = rq; nx.ap = det ? 0.f : alpha_n * rp; nx.has_p = !det;
    const bool resum = !det && px > 0.5f;
    float zs[2];
    {
      float accq, accp;
      if (det) pass_residual<IO, U1, false, false>(ioq, iop, ge, vbeg, vend, lane, nx, sm.bits, dropped, n_dropped, accq, accp);
      else if (resum) pass_residual<IO, U2, true>(ioq, iop, ge, vbeg, vend, lane, nx, sm.bits, dropped, n_dropped, accq, accp);
      else pass_residual<IO, U2, false>(ioq, iop, ge, vbeg, vend, lane, nx, sm.bits, dropped, n_dropped, accq, accp);
      zs[0] = warp_sum(accq);
      zs[1] = warp_sum(accp);
    }
    if (lane == 0) sm.wtmp[warp] = zs[0];
    combine<2, false>(c, zs);
    const float W_n = det ? W : (resum ? zs[1] * rp : W - en[1] * (x_dropped ? 0.f : 1.f));
    if (zs[0] > 0.f) {
      alpha = alpha_n;
      beta = zs[0];
      ibeta = 1.f / zs[0];
      cur = nx;
      if (warp == 0) {
        if (lane < SW) sm.wpart[lane] = sm.wtmp[lane];
        if (lane < static_cast<int>(c.nrank)) sm.rtot[lane] = c.gath[lane * 2];
      }
    }
    // (beta_{r+1} = 0 cannot follow a rejection in exact arithmetic unless m = 0 and the rows
    // coincide; the target then stays as it is)
    if (W_n > 0.f) { W = W_n; iW = 1.f / W_n; }
    __syncthreads();
  }

  // ---- no child accepted (or leaf): draw node_token from the current target by inverse CDF in
  // token order: CTA totals locate the CTA, per-warp sums the warp, whose range is then re-read.
  if (accepted < 0) {
    __syncthreads();
    const float u = fm[7];
    float total = 0.f;
    for (uint32_t r = 0; r < c.nrank; ++r) total += sm.rtot[r];
    const float target = u * total;
    int owner = -1, last_pos = -1;
    float Erun = 0.f, E_owner = 0.f;
    for (uint32_t r = 0; r < c.nrank; ++r) {
      const float t = sm.rtot[r];
      if (t > 0.f) last_pos = r;
      if (owner < 0 && Erun + t > target) { owner = r; E_owner = Erun; }
      Erun += t;
    }
    bool fallback = false;
    if (owner < 0) { owner = last_pos; fallback = true; }     // rounding pushed the target past the end
    if (owner == static_cast<int>(c.rank)) {
      const float wt = lane < SW ? sm.wpart[lane] : 0.f;
      const float wincl = warp_incl_scan(wt, lane);
      const uint32_t hit = fallback ? 0u : __ballot_sync(0xffffffffu, lane < SW && E_owner + wincl > target);
      const uint32_t pos = __ballot_sync(0xffffffffu, wt > 0.f);
      int ow = hit ? __ffs(hit) - 1 : -1;
      if (ow < 0) { ow = pos ? 31 - __clz(pos) : 0; fallback = true; }
      const float E0 = E_owner + __shfl_sync(0xffffffffu, wincl - wt, ow);
      // every thread of the CTA takes a contiguous piece of warp ow's range
      const int gwo = static_cast<int>(c.rank) * SW + ow;
      const int ob = min(gwo * ge.vw, ge.nvec), oe = min(ob + ge.vw, ge.nvec);
      const int pc = (oe - ob + ST - 1) / ST;
      const int mb = min(ob + tid * pc, oe), me = min(mb + pc, oe);
      float ts = 0.f;
      int lastpos = -1;
      for (int vv = mb; vv < me; ++vv) {
        float tv[VN];
        vec_terms(ioq, iop, ge, cur, sm.bits, vv, tv);
#pragma unroll
        for (int e = 0; e < VN; ++e) {
          ts += tv[e];
          if (tv[e] > 0.f) lastpos = ge.j0 + vv * VN + e;
        }
      }
      const float incl = warp_incl_scan(ts, lane);
      if (lane == 31) sm.scan[warp] = incl;
      if (tid == 0) sm.misc[3] = -1;
      __syncthreads();
      float before = 0.f;
      for (int w2 = 0; w2 < warp; ++w2) before += sm.scan[w2];
      const float prev = __shfl_up_sync(0xffffffffu, incl, 1);
      const float excl = before + (lane > 0 ? prev : 0.f);
      const float inc2 = before + incl;
      const bool mine = !fallback && !(E0 + excl > target) && (E0 + inc2 > target);
      if (mine) {                                  // at most one thread: its piece holds the draw
        sm.misc[4] = mb;
        sm.misc[5] = me;
        sm.misc[6] = lastpos;
        fm[1] = E0 + excl;
      }
      const int any = __syncthreads_or(mine ? 1 : 0);
      if (any && warp == 0) {
        // the 32 lanes walk that piece together, one token per lane and step
        const int t0 = ge.j0 + sm.misc[4] * VN, t1 = ge.j0 + sm.misc[5] * VN;
        float run = fm[1];
        int found = -1;
        for (int tb = t0; tb < t1 && found < 0; tb += 32) {
          const int t = tb + lane;
          float v = 0.f;
          if (t < t1 && t >= ge.alo && t < ge.ahi && !((sm.bits[t >> 5] >> (t & 31)) & 1u)) {
            v = ex2_approx(fmaf(ioq.z_at(t), kLog2e, cur.cq)) * cur.aq;
            if (cur.has_p) v = fmaxf(fmaf(-ex2_approx(fmaf(iop.z_at(t), kLog2e, cur.cp)), cur.ap, v), 0.f);
          }
          const float incl2 = warp_incl_scan(v, lane);
          const uint32_t hit = __ballot_sync(0xffffffffu, v > 0.f && run + incl2 > target);
          if (hit) found = tb + __ffs(hit) - 1;
          run += __shfl_sync(0xffffffffu, incl2, 31);
        }
        if (found < 0) found = sm.misc[6];
        if (lane == 0) a.node_token[out_b + n] = found;
      }
      if (!any) {
        // last positive entry of the range
        if (lastpos >= 0) atomicMax(&sm.misc[3], lastpos);
        __syncthreads();
        if (tid == 0) {
          a.node_token[out_b + n] = sm.misc[3];
          if (sm.misc[3] < 0) vflag(a.status, LANTERN_DEV_EMPTY_ROW);
        }
      }
    } else if (owner < 0 && writer) {
      a.node_token[out_b + n] = -1;      // empty distribution
      vflag(a.status, LANTERN_DEV_EMPTY_ROW);
    }
  } else if (writer) {
    a.node_token[out_b + n] = -1;
  }
  if (writer) a.node_next[out_b + n] = accepted;
  return accepted;
}

// GENERAL = false: one node per CTA (cluster), default acceptance rule (the benchmarked launch).
// GENERAL = true: the same plus what is decided at run time: the path walk and the rule variants.
template <typename T, bool CFG, bool TAU1, bool GENERAL>
__global__ void __launch_bounds__(ST, LANTERN_STREAM_MINB) verify_stream_kernel(const VerifyArgs a) {
  grid_dependency_sync();
  extern __shared__ __align__(16) unsigned char stream_smem[];
  constexpr int NOPS = CFG ? 4 : 2;
  const int kp1 = a.k + 1;
  StreamSmem sm;
  SCtx c;
  float* small = reinterpret_cast<float*>(stream_smem);
  c.red = small;                       // 2 * SW * 4
  c.xch = c.red + 2 * SW * 4;          // 8
  c.gath = c.xch + 8;                  // kMaxCluster * 4
  sm.wpart = c.gath + kMaxCluster * 4; // SW
  sm.wtmp = sm.wpart + SW;             // SW
  sm.rtot = sm.wtmp + SW;              // kMaxCluster
  sm.scan = sm.rtot + kMaxCluster;     // SW
  sm.misc = reinterpret_cast<int*>(sm.scan + SW);      // 32
  sm.memb = reinterpret_cast<uint32_t*>(sm.misc + 32); // 33
  static_assert((2 * SW * 4 + 8 + kMaxCluster * 4 + SW + SW + kMaxCluster + SW + 32 + 33) * 4 <= kSmallBytes, "small area");
  sm.bits = reinterpret_cast<uint32_t*>(stream_smem + kSmallBytes);
  sm.ent = reinterpret_cast<float*>(sm.bits + (a.V + 127) / 128 * 4);
  sm.tok = reinterpret_cast<int*>(sm.ent + static_cast<size_t>(a.max_children) * kp1 * NOPS);
  c.rank = cluster_ctarank();
  c.nrank = cluster_nctarank();
  c.parity = 0;
  const int idx = blockIdx.x / c.nrank;
  // A regular launch verifies one node per CTA (cluster).  With a.lazy the CTA (cluster) owns a
  // sequence and walks it (Sec. 2.1): it verifies the root, moves to the accepted child and so
  // on, so only the rows on the accepted path are read and the per-node results of the other
  // nodes are not written.
  const bool lazy = GENERAL && a.lazy != 0;
  const int b = lazy ? idx : idx % a.B;
  int cur = lazy ? 0 : a.order[(GENERAL ? b * a.tree_stride : 0) + idx / a.B];
  if (GENERAL && cur < 0) {            // padding of a forest's shorter tree: nothing to verify (the whole cluster leaves)
    if (c.rank == 0 && threadIdx.x == 0) {
      const long long o = static_cast<long long>(b) * a.N + idx / a.B;       // padding sits at the end of the order
      a.node_next[o] = -1;
      a.node_token[o] = -1;
      if (a.node_mass) a.node_mass[o] = -1.f;
      if (a.node_thresh) a.node_thresh[o] = -1.f;
    }
    return;
  }
  int len = 0;
  for (;;) {
    const int acc = stream_node<T, CFG, TAU1, GENERAL>(a, b, cur, c, sm);
    if (!lazy) break;
    csync(c);     // the next node reuses the shared memory; also orders the store of node_token before the read below
    const bool writer = c.rank == 0 && threadIdx.x == 0;
    int32_t* ot = a.out_tokens + static_cast<long long>(b) * a.D1;
    int32_t* on = a.out_nodes + static_cast<long long>(b) * a.D1;
    if (acc <= cur || acc >= a.N || len >= a.D1 - 1) {      // -1, or anything that is not a forward edge
      if (writer) {
        ot[len] = __ldcg(a.node_token + static_cast<long long>(b) * a.N + cur);
        on[len] = cur;
        a.accept_len[b] = len;
        for (int i = len + 1; i < a.D1; ++i) { ot[i] = -1; on[i] = -1; }
      }
      break;
    }
    cur = acc;
    if (writer) { ot[len] = a.tokens[static_cast<long long>(b) * a.N + cur]; on[len] = cur; }
    ++len;
  }
  if (c.nrank > 1) cluster_sync();     // peers may still be reading this CTA's exchange buffer
}

}  // namespace stream
}  // namespace lantern
