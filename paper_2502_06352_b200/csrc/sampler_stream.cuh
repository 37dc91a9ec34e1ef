// Stochastic static-tree drafting (Sec. 2.1) for rows that no top-k truncates: streaming kernel.
//
// The s children of a parent are the s largest keys z_j + G_j, G_j = -log(-log U_j) (Gumbel-top-s,
// sampling without replacement from p).  The drafter row is streamed from HBM once and never held
// on chip: every element gets a float32 key from fast logarithms (absolute error below kKeyEps),
// and only the elements whose key exceeds a running threshold T are appended to a short candidate
// list in shared memory.  T is a lower bound of the (s+4)-th largest key seen so far: when the
// list would overflow it is cut back to its s+4 best entries and T rises to the last of them, so
// every element left out has key <= T.  At the end the few candidates are ranked by keys
// recomputed in double precision (ties: lower token id); the result is the exact ranking as
// long as the s-th exact key clears T by kKeyEps, which is checked (LANTERN_DEV_KEY_TIES
// otherwise: more than s+4 keys within 2.5e-4 of each other at the top).  The softmax
// denominator for draft_prob comes from the same pass.
#pragma once
#include "verify_stream.cuh"

namespace lantern {
namespace stream {

constexpr int kIterElems = 4096;                 // row elements one CTA handles between two barriers
constexpr int kListCap = kIterElems + 256;       // candidate entries
constexpr int kFinal = 256;                      // candidates ranked exactly at the end
constexpr int kExtra = 4;                        // the list is cut back to s + kExtra entries
constexpr float kKeyEps = 2.5e-4f;               // bound on |fast key - exact key|

__host__ __device__ constexpr size_t sampler_stream_smem() {
  return kSmallBytes + kListCap * 8 + kFinal * 12 + 2 * 2 * SW * 8 + 16 * 8;
}

__device__ __forceinline__ float lg2_approx(float x) {
  float y;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// float32 key of one element: z - ln2 * lg2(-lg2 U) (the constant -ln(ln 2) is the same for all).
// lg2.approx is accurate to 2^-22 absolutely near 1, so for U > 0.999 (where -lg2 U is tiny) the
// callers redo the inner logarithm with logf.
__device__ __forceinline__ float fast_key(float z, float U) {
  return fmaf(-0.6931471805599453f, lg2_approx(-lg2_approx(U)), z);
}
__device__ __noinline__ float careful_key(float z, float U) {
  return fmaf(-0.6931471805599453f, lg2_approx(-logf(U) * kLog2e), z);
}

__device__ __forceinline__ bool key_before(float ka, int ia, float kb, int ib) {   // a ranks before b
  return ka > kb || (ka == kb && ia < ib);
}
__device__ __forceinline__ void warp_key_first(float& k, int& i) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ok = __shfl_xor_sync(0xffffffffu, k, o);
    const int oi = __shfl_xor_sync(0xffffffffu, i, o);
    if (key_before(ok, oi, k, i)) { k = ok; i = oi; }
  }
}

struct SampSmem {
  uint2* list;      // [kListCap] (key bits, token)
  int* cnt;         // entries in the list
  double* fkey;     // [kFinal] exact keys
  int* ftok;        // [kFinal]
  uint2* pk;        // [2][SW] warps' best entries of a selection round
  uint2* top;       // [16] winners of the rounds of a cut
};

// Cut the list back to its R best entries (key descending, token ascending).  Returns the new
// threshold: the key of the R-th entry, or `T` unchanged when the list has fewer than R entries.
__device__ __forceinline__ float cut_list(const SampSmem& s, int R, float T) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n = min(*s.cnt, kListCap);
  float pk = INFINITY;
  int pt = -1;
  int got = 0;
  for (int round = 0; round < R; ++round) {
    float bk = -INFINITY;
    int bt = 0x7fffffff;
    for (int i = tid; i < n; i += ST) {
      const uint2 en = s.list[i];
      const float k = __uint_as_float(en.x);
      const int t = static_cast<int>(en.y);
      if (key_before(pk, pt, k, t) && key_before(k, t, bk, bt)) { bk = k; bt = t; }
    }
    warp_key_first(bk, bt);
    uint2* buf = s.pk + (round & 1) * SW;
    if (lane == 0) buf[warp] = make_uint2(__float_as_uint(bk), static_cast<uint32_t>(bt));
    __syncthreads();
    float ck = -INFINITY;
    int ct = 0x7fffffff;
    if (lane < SW) { ck = __uint_as_float(buf[lane].x); ct = static_cast<int>(buf[lane].y); }
    warp_key_first(ck, ct);
    if (ct == 0x7fffffff) break;                 // fewer than R entries (the same in every thread)
    if (tid == 0) s.top[round] = make_uint2(__float_as_uint(ck), static_cast<uint32_t>(ct));
    pk = ck;
    pt = ct;
    ++got;
  }
  __syncthreads();                               // every scan of the list is over
  if (tid < got) s.list[tid] = s.top[tid];
  if (tid == 0) *s.cnt = got;
  __syncthreads();
  return got == R ? pk : T;
}

// The same cut for a short list, by warp 0 alone (no barriers inside the rounds); every thread
// calls it between two barriers' worth of quiet: nobody appends while it runs.  R <= 15.
__device__ __forceinline__ float cut_small(const SampSmem& s, int R, float T) {
  const int tid = threadIdx.x, lane = tid & 31;
  const int n = min(*s.cnt, kListCap);
  __syncthreads();                               // every thread has read the count
  if (tid < 32) {
    float pk = INFINITY;
    int pt = -1;
    int got = 0;
    for (int round = 0; round < R; ++round) {
      float bk = -INFINITY;
      int bt = 0x7fffffff;
      for (int i = lane; i < n; i += 32) {
        const uint2 en = s.list[i];
        const float k = __uint_as_float(en.x);
        const int t = static_cast<int>(en.y);
        if (key_before(pk, pt, k, t) && key_before(k, t, bk, bt)) { bk = k; bt = t; }
      }
      warp_key_first(bk, bt);
      if (bt == 0x7fffffff) break;               // fewer than R entries (the same in every lane)
      if (lane == 0) s.top[round] = make_uint2(__float_as_uint(bk), static_cast<uint32_t>(bt));
      pk = bk;
      pt = bt;
      ++got;
    }
    __syncwarp();
    if (lane < got) s.list[lane] = s.top[lane];
    if (lane == 0) {
      *s.cnt = got;
      s.top[15].x = __float_as_uint(got == R ? pk : T);
    }
  }
  __syncthreads();
  return __uint_as_float(s.top[15].x);
}

template <typename T, bool CFG, bool TAU1>
__global__ void __launch_bounds__(ST, 4) sample_stream_kernel(const SampleArgs a) {
  grid_dependency_sync();
  using IO = RowIO<T, CFG, TAU1>;
  constexpr int VN = IO::VN;
  constexpr int UV = (CFG ? 2 : 4) * 4 / VN;     // vectors per thread and iteration (ST*UV*VN <= kIterElems)
  static_assert(ST * UV * VN <= kIterElems, "iteration size");
  extern __shared__ __align__(16) unsigned char samp_smem[];
  SCtx c;
  float* small = reinterpret_cast<float*>(samp_smem);
  c.red = small;
  c.xch = c.red + 2 * SW * 4;
  c.gath = c.xch + 8;
  int* misc = reinterpret_cast<int*>(c.gath + kMaxCluster * 4);     // [32]
  SampSmem s;
  s.list = reinterpret_cast<uint2*>(samp_smem + kSmallBytes);
  s.fkey = reinterpret_cast<double*>(s.list + kListCap);
  s.ftok = reinterpret_cast<int*>(s.fkey + kFinal);
  s.pk = reinterpret_cast<uint2*>(s.ftok + kFinal);
  s.top = s.pk + 2 * SW;
  s.cnt = misc;
  c.rank = cluster_ctarank();
  c.nrank = cluster_nctarank();
  c.parity = 0;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int idx = blockIdx.x / c.nrank;
  const int b = idx % a.B;
  const int n = a.order[a.order_begin + idx / a.B];
  const int fc = a.first_child[n], nc = a.n_child[n];
  const long long row_off = static_cast<long long>(b) * a.seq_stride + static_cast<long long>(n) * a.row_stride;
  const long long out_b = static_cast<long long>(b) * a.N;
  const uint32_t row_id = static_cast<uint32_t>(out_b + n);
  const float* gum = a.gumbel ? a.gumbel + static_cast<long long>(row_id) * a.V : nullptr;
  const bool want_prob = a.draft_prob != nullptr;
  const int R = nc + kExtra;

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

  IO io;
  io.c = static_cast<const T*>(a.dc) + row_off;
  io.u = CFG ? static_cast<const T*>(a.du) + row_off : nullptr;
  io.g = a.g; io.it = a.inv_tau; io.j0 = ge.j0;

  if (tid == 0) *s.cnt = 0;
  __syncthreads();

  // Uniforms of tokens j .. j+VN-1 (j a multiple of VN); returns whether one of them exceeds 0.999.
  // Philox words become floats without an integer conversion: the 23 mantissa bits under the
  // exponent of 1.0 give 1 + i 2^-23, and subtracting 1 - 2^-24 leaves (i + 1/2) 2^-23 exactly.
  auto uniforms = [&](int j, float (&U)[VN]) -> bool {
    bool near_one = false;
    if (gum) {
#pragma unroll
      for (int e = 0; e < VN; ++e) {
        U[e] = (j + e < a.V) ? __ldcs(gum + j + e) : 0.5f;
        near_one |= U[e] > 0.999f;
      }
    } else {
#pragma unroll
      for (int q = 0; q < VN / 4; ++q) {
        const Philox4 r = philox4x32_10_keys(static_cast<uint32_t>((j >> 2) + q), row_id, static_cast<uint32_t>(a.step),
                                             (static_cast<uint32_t>(a.step >> 32) << 2) | kStreamGumbel, a.rk0, a.rk1);
        const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int e = 0; e < 4; ++e)
          U[4 * q + e] = __uint_as_float(0x3f800000u | (w[e] >> 9)) - 0.99999994f;
        near_one |= (max(max(r.x, r.y), max(r.z, r.w)) >> 9) > 8380219u;       // 0.999 * 2^23
      }
    }
    return near_one;
  };

  // One entry for the list (appends are rare after the first cut: a shared-memory atomic each)
  auto append = [&](float k, int tok) {
    const int pos = atomicAdd(s.cnt, 1);
    if (pos < kListCap) s.list[pos] = make_uint2(__float_as_uint(k), static_cast<uint32_t>(tok));
  };
  // Optimistic pass.  The first chunk's keys stay in registers until a first threshold is known: the
  // R-th best of the warps' two best keys each (distinct tokens, so a lower bound of the row's R-th
  // best key), found with one barrier; the chunk's keys above it then enter the list.  One cut of the
  // (short) list after a third of the row tightens the threshold (more cuts cost more in barriers than
  // they save in appends); the other chunks run without barriers.  If the list overflows all the same (keys that keep growing along the row), the
  // row is redone with a check after every chunk.
  float Tk = -INFINITY;                               // every element left out has key <= Tk
  float mx = -INFINITY, sx = 0.f;
  const int iters = (ge.vw + 32 * UV - 1) / (32 * UV);
  const int cut_it = max(1, iters / 3);                // the one scheduled cut of the optimistic pass
  for (int mode = 0; mode < 2; ++mode) {
    Tk = -INFINITY;
    mx = -INFINITY;
    sx = 0.f;
    for (int it = 0; it < iters; ++it) {
      const int base = vbeg + it * 32 * UV;
      uint4 rc[UV], ru[UV];
#pragma unroll
      for (int u = 0; u < UV; ++u) {
        const int vv = base + 32 * u + lane;
        if (vv < vend && vv >= ge.vi0 && vv < ge.vi1) io.load(vv, rc[u], ru[u]);
      }
      float first[UV][VN];                              // keys of the first chunk
      float tbk = -INFINITY;                            // ... and the thread's best of them
      int tbj = 0x7fffffff;
#pragma unroll
      for (int u = 0; u < UV; ++u) {
        const int vv = base + 32 * u + lane;
        const bool active = vv < vend;
        const int j = ge.j0 + vv * VN;
        float z[VN], key[VN];
#pragma unroll
        for (int e = 0; e < VN; ++e) key[e] = -INFINITY;
        if (active) {
          if (vv >= ge.vi0 && vv < ge.vi1) {
            io.z(rc[u], ru[u], z);
          } else {                                      // ragged first / last vector of the row
#pragma unroll
            for (int e = 0; e < VN; ++e) z[e] = (j + e >= ge.alo && j + e < ge.ahi) ? io.z_at(j + e) : -INFINITY;
          }
          float U[VN];
          const bool near_one = uniforms(j, U);
#pragma unroll
          for (int e = 0; e < VN; ++e) key[e] = fast_key(z[e], U[e]);
          if (near_one) {                               // rare: one vector in a hundred
#pragma unroll
            for (int e = 0; e < VN; ++e)
              if (U[e] > 0.999f) key[e] = careful_key(z[e], U[e]);
          }
          if (want_prob) acc_exp<VN>(z, mx, sx);
        }
        if (it == 0) {
#pragma unroll
          for (int e = 0; e < VN; ++e) {
            first[u][e] = key[e];
            if (key_before(key[e], j + e, tbk, tbj)) { tbk = key[e]; tbj = j + e; }
          }
        } else {
          float best = key[0];
#pragma unroll
          for (int e = 1; e < VN; ++e) best = fmaxf(best, key[e]);
          if (best > Tk) {                              // rare, and rarer after every cut
#pragma unroll
            for (int e = 0; e < VN; ++e)
              if (key[e] > Tk) append(key[e], j + e);
          }
        }
      }
      if (it == 0) {
        // the two best of every warp's thread-bests: 2 * SW keys of distinct tokens, whose R-th best is a
        // lower bound of the row's R-th best key (R <= 12 <= 2 * SW); every warp ranks them for itself
        float k1 = tbk, k2;
        int j1 = tbj, j2;
        warp_key_first(k1, j1);
        k2 = (tbj == j1) ? -INFINITY : tbk;
        j2 = (tbj == j1) ? 0x7fffffff : tbj;
        warp_key_first(k2, j2);
        if (lane == 0) {
          s.pk[2 * warp] = make_uint2(__float_as_uint(k1), static_cast<uint32_t>(j1));
          s.pk[2 * warp + 1] = make_uint2(__float_as_uint(k2), static_cast<uint32_t>(j2));
        }
        __syncthreads();
        {
          const uint2 en = s.pk[lane & (2 * SW - 1)];
          const float mk = __uint_as_float(en.x);
          const int mt = static_cast<int>(en.y);
          int rank = 0;
#pragma unroll
          for (int i = 0; i < 2 * SW; ++i) {
            const float ok = __shfl_sync(0xffffffffu, mk, i);
            const int ot = __shfl_sync(0xffffffffu, mt, i);
            rank += key_before(ok, ot, mk, mt) ? 1 : 0;
          }
          const uint32_t hit = __ballot_sync(0xffffffffu, lane < 2 * SW && rank == R - 1 && mt != 0x7fffffff && mk > -INFINITY);
          if (hit) Tk = __shfl_sync(0xffffffffu, mk, __ffs(hit) - 1);
        }
#pragma unroll
        for (int u = 0; u < UV; ++u) {
          const int j = ge.j0 + (base + 32 * u + lane) * VN;
#pragma unroll
          for (int e = 0; e < VN; ++e)
            if (first[u][e] > Tk) append(first[u][e], j + e);
        }
      } else if (it == cut_it || mode == 1) {
        __syncthreads();
        const int cn = *s.cnt;
        const bool do_cut = mode == 1 ? cn > kListCap - kIterElems : cn > R;
        __syncthreads();                                // everyone has read the count before it moves again
        if (do_cut) Tk = cn <= 1024 ? cut_small(s, R, Tk) : cut_list(s, R, Tk);
      }
    }
    __syncthreads();
    const bool overflow = *s.cnt > kListCap;
    if (!overflow) break;
    __syncthreads();                                    // (mode 1 never overflows: it cuts in time)
    if (tid == 0) *s.cnt = 0;
    __syncthreads();
  }

  // ---- softmax denominator of the row (for draft_prob)
  float gm[1] = {0.f}, gs[1] = {0.f};
  if (want_prob) {                                    // (uniform: a kernel argument)
    gm[0] = warp_max(mx);
    combine<1, true>(c, gm);
    if (gm[0] == -INFINITY) gm[0] = 0.f;
    gs[0] = warp_sum(mx == -INFINITY ? 0.f : sx * ex2_approx((mx - gm[0]) * kLog2e));
    combine<1, false>(c, gs);
  }

  // ---- candidates of all CTAs of the row -> CTA 0, exact keys, ranking
  __syncthreads();
  const int share = kFinal / static_cast<int>(c.nrank);
  if (*s.cnt > share) { __syncthreads(); Tk = cut_list(s, min(R, share), Tk); }
  float tmax[1] = {warp_max(Tk)};
  combine<1, true>(c, tmax);                          // its barriers also publish the lists
  if (c.rank == 0) {
    int nf = 0;
    for (uint32_t r = 0; r < c.nrank; ++r) {
      const uint32_t cnt_r = c.nrank > 1 ? dsmem_ld_u32(dsmem_addr(smem_u32(s.cnt), r)) : static_cast<uint32_t>(*s.cnt);
      const int m = min(static_cast<int>(cnt_r), share);
      if (tid < m) {
        uint32_t tokv;
        if (c.nrank > 1) tokv = dsmem_ld_u32(dsmem_addr(smem_u32(&s.list[tid]) + 4u, r));
        else tokv = s.list[tid].y;
        const int t = static_cast<int>(tokv);
        float U;
        if (gum) {
          U = __ldcs(gum + t);
        } else {
          const Philox4 rr = philox_stream(a.seed, a.step, row_id, kStreamGumbel, static_cast<uint32_t>(t >> 2));
          const uint32_t wv = (t & 3) == 0 ? rr.x : ((t & 3) == 1 ? rr.y : ((t & 3) == 2 ? rr.z : rr.w));
          U = uniform_open(wv);
        }
        const float zt = io.z_at(t);
        s.fkey[nf + tid] = static_cast<double>(zt) - log(-log(static_cast<double>(U)));
        s.ftok[nf + tid] = t;
      }
      nf += m;
    }
    __syncthreads();
    if (tid < nf) {
      const double k = s.fkey[tid];
      const int t = s.ftok[tid];
      int rank = 0;
      for (int i = 0; i < nf; ++i) {
        const double ki = s.fkey[i];
        rank += (ki > k || (ki == k && s.ftok[i] < t)) ? 1 : 0;
      }
      if (rank < nc) {
        a.tokens[out_b + fc + rank] = t;
        if (want_prob) {
          const float zt = io.z_at(t);
          a.draft_prob[out_b + fc + rank] = gs[0] > 0.f ? ex2_approx(fmaf(zt, kLog2e, -gm[0] * kLog2e)) / gs[0] : 0.f;
        }
        if (rank == nc - 1 && static_cast<double>(tmax[0]) + kKeyEps >= k) vflag(a.status, LANTERN_DEV_KEY_TIES);
      }
    }
    if (tid >= nf && tid < nc) {                      // fewer than s tokens with positive probability
      a.tokens[out_b + fc + tid] = -1;
      if (want_prob) a.draft_prob[out_b + fc + tid] = 0.f;
    }
    if (nf == 0 && tid == 0) vflag(a.status, LANTERN_DEV_EMPTY_ROW);
  }
  if (c.nrank > 1) cluster_sync();                    // CTA 0 may still be reading this CTA's list
}

}  // namespace stream
}  // namespace lantern
