// Relaxed verification of a static draft tree (Sec. 4; App. A.2 Eq. 1-2; Sec. 2.1).
//
// One thread-block cluster per tree node.  The node's target row (and, for an internal node,
// its drafter row) is read from HBM exactly once with 128-bit streaming loads, post-processed
// (guidance, temperature, top-k, softmax) and kept as float32 in the shared memory of the
// cluster's CTAs, each CTA owning a contiguous slice of the vocabulary.  The sibling loop, the
// residual updates and the final inverse-CDF draw run entirely on chip.
//
// Distributions are stored unnormalised: q_cur[j] = Q[j] * qs, p_cur[j] = P[j] * ps with the
// scalars qs, ps held in registers, so a renormalisation never rewrites a row.
#include "rowregs.cuh"

namespace lantern {

struct VerifyArgs {
  const void *tc, *tu, *dc, *du;
  long long row_stride, seq_stride;
  const int32_t* tokens;
  const float *u_acc, *u_res;
  const int32_t* nbr;
  int k_table, use_bulk;
  const int32_t *first_child, *n_child, *order;
  int B, N, V, SL, kpad;
  float g, inv_tau, lambda;
  int topk_t, topk_d, k, code_offset, n_codes, allow_lo, allow_hi;
  unsigned long long seed, step;
  int32_t *node_next, *node_token;
  float *node_mass, *node_thresh;
  int32_t* status;
};

constexpr int kMiscInts = 16;
constexpr int kCandInts = 40;
// fixed part of the dynamic shared memory behind the two row slices
constexpr int kTopkBytes = 2 * 256 * 4 + 2 * kCandLocal * 4 + 2 * kCandTotal * 4;
constexpr int kFixedSmemBytes = kTopkBytes + kWarps * 4 * 4 + 8 * 4 + kMaxCluster * 4 * 4 + 4 * 4 +
                                kCandInts * 4 + kMiscInts * 4 + 16;

__device__ __forceinline__ void flag(int32_t* status, int bit) {
  if (status) atomicOr(status, bit);
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

// E = row entries per thread; the CTA's slice holds SL = 256 * E entries.
template <typename T, bool CFG, int E>
__global__ void __launch_bounds__(kThreads, (E >= 16) ? 2 : 3) verify_nodes_kernel(const VerifyArgs a) {
  constexpr int VN = Vec<T>::N;
  constexpr int SL = kThreads * E;
  constexpr int NV4 = E / 4;                 // float4 per thread in a shared-memory sweep
  extern __shared__ __align__(16) unsigned char smem_raw[];
  float* Q = reinterpret_cast<float*>(smem_raw);
  float* P = Q + SL;
  TopkSmem tk;
  tk.bins = reinterpret_cast<uint32_t*>(P + SL);
  tk.candl = reinterpret_cast<float*>(tk.bins + 2 * 256);
  tk.all = tk.candl + 2 * kCandLocal;
  ClusterCtx c;
  c.hist = reinterpret_cast<uint32_t*>(tk.all);          // radix fallback only
  c.red = tk.all + 2 * kCandTotal;
  c.xch = c.red + kWarps * 4;
  c.gath = c.xch + 8;
  c.sel = reinterpret_cast<int*>(c.gath + kMaxCluster * 4);
  tk.candn = c.sel + 4;
  int* misc = tk.candn + kCandInts;
  uint64_t* mbar = reinterpret_cast<uint64_t*>(misc + kMiscInts);
  int* nbr_s = reinterpret_cast<int*>(mbar + 2);
  c.rank = cluster_ctarank();
  c.nrank = cluster_nctarank();
  c.parity = 0;
  c.hist_parity = 0;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int idx = blockIdx.x / c.nrank;
  const int b = idx % a.B;
  const int n = a.order[idx / a.B];
  const int fc = a.first_child[n], nc = a.n_child[n];
  const int lo = c.rank * SL;
  const int len = max(0, min(a.V - lo, SL));
  const long long row_off = static_cast<long long>(b) * a.seq_stride + static_cast<long long>(n) * a.row_stride;
  const int32_t* tok_b = a.tokens + static_cast<long long>(b) * a.N;
  const long long out_b = static_cast<long long>(b) * a.N;
  const uint32_t q_base = smem_u32(Q), p_base = smem_u32(P);

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
        for (int r = tid; r < a.k; r += kThreads)
          nbr_s[ci * a.kpad + r] = a.nbr[static_cast<long long>(code) * a.k_table + r];
    }
  }

  // ---- read the rows once into registers: z_q, z_p
  float zq[E], zp[E];
  load_row_regs<T, CFG, E>(static_cast<const T*>(a.tc) + row_off,
                           CFG ? static_cast<const T*>(a.tu) + row_off : nullptr, a.g, a.inv_tau, lo, len, zq);
  if (nc > 0) {
    load_row_regs<T, CFG, E>(static_cast<const T*>(a.dc) + row_off,
                             CFG ? static_cast<const T*>(a.du) + row_off : nullptr, a.g, a.inv_tau, lo, len, zp);
  } else {
#pragma unroll
    for (int e = 0; e < E; ++e) zp[e] = -INFINITY;
  }
  if (a.allow_lo > 0 || a.allow_hi < a.V) {
    mask_regs<E, VN>(zq, lo, a.allow_lo, a.allow_hi);
    mask_regs<E, VN>(zp, lo, a.allow_lo, a.allow_hi);
  }
  float mx[2] = {max_regs<E>(zq), max_regs<E>(zp)};
  cluster_reduce<2, true>(c, mx);
  if (mx[0] == -INFINITY || (nc > 0 && mx[1] == -INFINITY)) {
    if (tid == 0 && c.rank == 0) flag(a.status, LANTERN_DEV_EMPTY_ROW);
    if (mx[0] == -INFINITY) mx[0] = 0.f;
  }
  if (mx[1] == -INFINITY) mx[1] = 0.f;

  // ---- top-k truncation thresholds (exact)
  float theta[2] = {-INFINITY, -INFINITY};
  const int kth[2] = {(a.topk_t > 0 && a.topk_t < a.V) ? a.topk_t : 0,
                      (nc > 0 && a.topk_d > 0 && a.topk_d < a.V) ? a.topk_d : 0};
  const bool has_topk = kth[0] > 0 || kth[1] > 0;
  if (has_topk) {
    if (!topk_regs<E>(c, tk, zq, zp, mx, kth, theta)) {
      // too many entries tie around the k-th one: radix select over shared-memory copies
      store_regs<E, VN>(zq, Q);
      store_regs<E, VN>(zp, P);
      __syncthreads();
      float* const rows[2] = {Q, P};
      int kk[2] = {kth[0], kth[1]};
      cluster_topk_threshold<2>(c, rows, len, kk, theta);
      __syncthreads();
    }
  }

  // ---- softmax numerators -> shared memory, row sums
  float sm[2];
  if (has_topk) {
    sm[0] = exp_store_regs<E, VN, true>(zq, mx[0], theta[0], Q);
    sm[1] = exp_store_regs<E, VN, true>(zp, mx[1], theta[1], P);
  } else {
    sm[0] = exp_store_regs<E, VN, false>(zq, mx[0], 0.f, Q);
    sm[1] = nc > 0 ? exp_store_regs<E, VN, false>(zp, mx[1], 0.f, P) : 0.f;
  }
  cluster_reduce<2, false>(c, sm);     // its cluster barrier also publishes Q and P
  // q_cur[j] = Q[j] * qs,  p_cur[j] = P[j] / psum
  float qs = sm[0] > 0.f ? 1.f / sm[0] : 0.f;
  float psum = sm[1];

  // ---- neighbour rows must have landed
  if (bulk_issued) {
    bool ok = mbar_wait_bounded(mbar_a, 0);
    if (!__syncthreads_and(ok)) {
      if (tid == 0) flag(a.status, LANTERN_DEV_TIMEOUT);
      for (int ci = 0; ci < nc; ++ci) {
        int code = tok_b[fc + ci] - a.code_offset;
        if (code >= 0 && code < a.n_codes)
          for (int r = tid; r < a.k; r += kThreads)
            nbr_s[ci * a.kpad + r] = a.nbr[static_cast<long long>(code) * a.k_table + r];
      }
    }
  }
  __syncthreads();

  if (n == 0 && c.rank == 0 && tid == 0) {
    if (a.node_mass) a.node_mass[out_b] = -1.f;
    if (a.node_thresh) a.node_thresh[out_b] = -1.f;
  }

  // ---- sibling loop (Sec. 4; Eq. 1-2)
  int accepted = -1;
  for (int ci = 0; ci < nc; ++ci) {
    const int child = fc + ci;
    const int x = tok_b[child];
    bool skip = accepted >= 0 || x < 0 || x >= a.V;
    if (skip) {
      if (accepted < 0 && x >= a.V && tid == 0 && c.rank == 0) flag(a.status, LANTERN_DEV_BAD_INDEX);
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
      const uint32_t xr = static_cast<uint32_t>(x) / SL, xo = static_cast<uint32_t>(x) - xr * SL;
      const float qx = dsmem_ld_f32(dsmem_addr(q_base + xo * 4, xr)) * qs;
      const float pxraw = dsmem_ld_f32(dsmem_addr(p_base + xo * 4, xr));
      const float px = pxraw * ps;
      const float bound = a.lambda * qx;
      float cum = qx;
      int nA = 0;
      bool bad = false;
      if (has_code) {
        for (int base = 0; base < a.k; base += 32) {
          const int r = base + lane;
          float qa = 0.f;
          if (r < a.k) {
            const int t = a.code_offset + nrow[r];
            if (t >= 0 && t < a.V) {
              const uint32_t tr = static_cast<uint32_t>(t) / SL, to = static_cast<uint32_t>(t) - tr * SL;
              qa = dsmem_ld_f32(dsmem_addr(q_base + to * 4, tr)) * qs;
            } else {
              bad = true;
            }
          }
          const float incl = warp_incl_scan(qa, lane);
          const bool ok = r < a.k && (cum + incl < bound);
          const uint32_t ballot = __ballot_sync(0xffffffffu, ok);
          const int ntake = __ffs(~ballot) - 1;          // leading accepted entries; -1 when all 32
          const int take = ntake < 0 ? 32 : ntake;
          if (take > 0) cum += __shfl_sync(0xffffffffu, incl, take - 1);
          nA += take;
          if (take < 32) break;
        }
      }
      if (__any_sync(0xffffffffu, bad) && lane == 0 && c.rank == 0) flag(a.status, LANTERN_DEV_BAD_INDEX);
      const float m = cum;
      const float thr = px > 0.f ? fminf(1.f, m / px) : (m > 0.f ? 1.f : 0.f);
      float u;
      if (a.u_acc) {
        u = a.u_acc[out_b + child];
      } else {
        u = uniform_halfopen(philox_stream(a.seed, a.step, static_cast<uint32_t>(out_b + child), kStreamAccept, 0).x);
      }
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
    cluster_sync();          // every CTA has finished reading q_cur / p_cur of this round
    for (int r = tid; r < nA; r += kThreads) {
      const int t = a.code_offset + nrow[r] - lo;
      if (t >= 0 && t < len) Q[t] = 0.f;
    }
    const int xl = x - lo;                                   // position of x in this slice, if any
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
    cluster_reduce<2, false>(c, zs);
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
      cluster_reduce<2, false>(c, s2);       // leaves the per-warp and per-rank sums of Q in place
      qs = ps_old;
    }
  }

  // ---- no child accepted (or leaf): draw node_token from q_cur by inverse CDF in token order.
  // The last reduction left the per-warp sums of Q in c.red[w*2] and the per-rank sums in
  // c.gath[r*2]; the slice and the warp segment that hold the draw follow from those.
  if (accepted < 0) {
    float u;
    if (a.u_res) {
      u = a.u_res[out_b + n];
    } else {
      u = uniform_halfopen(philox_stream(a.seed, a.step, static_cast<uint32_t>(out_b + n), kStreamResample, 0).x);
    }
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
      int ow = -1, lastw = -1;
      float Ew = E_owner, Ew_owner = 0.f;
      for (int w = 0; w < kWarps; ++w) {
        const float t = c.red[w * 2];
        if (t > 0.f) lastw = w;
        if (!fallback && ow < 0 && Ew + t > target) { ow = w; Ew_owner = Ew; }
        Ew += t;
      }
      bool wfallback = fallback;
      if (ow < 0) { ow = lastw; wfallback = true; }
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
      flag(a.status, LANTERN_DEV_EMPTY_ROW);
    }
  } else if (c.rank == 0 && tid == 0) {
    a.node_token[out_b + n] = -1;
  }
  if (c.rank == 0 && tid == 0) a.node_next[out_b + n] = accepted;
  cluster_sync();    // peers may still be reading this CTA's shared memory
}

// ---- walk (Sec. 2.1): follow accepted children from the root
__global__ void walk_kernel(const int32_t* __restrict__ node_next, const int32_t* __restrict__ node_token,
                            const int32_t* __restrict__ tokens, int B, int N, int D1,
                            int32_t* __restrict__ accept_len, int32_t* __restrict__ out_tokens,
                            int32_t* __restrict__ out_nodes) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= B) return;
  const int32_t* nx = node_next + static_cast<long long>(b) * N;
  const int32_t* nt = node_token + static_cast<long long>(b) * N;
  const int32_t* tk = tokens + static_cast<long long>(b) * N;
  int32_t* ot = out_tokens + static_cast<long long>(b) * D1;
  int32_t* on = out_nodes + static_cast<long long>(b) * D1;
  int cur = 0, len = 0;
  while (len < D1 - 1) {
    int nxt = nx[cur];
    if (nxt <= cur || nxt >= N) break;      // -1, or anything that is not a forward edge
    cur = nxt;
    ot[len] = tk[cur];
    on[len] = cur;
    ++len;
  }
  ot[len] = nt[cur];
  on[len] = cur;
  accept_len[b] = len;
  for (int i = len + 1; i < D1; ++i) { ot[i] = -1; on[i] = -1; }
}

static int g_cluster_override = 0;

struct LaunchShape { int cs, e; size_t smem; };

// Choose E (row entries per thread, slice = 256*E) and the cluster size (CTAs per row).
// `min_e` is 4 for float32 rows and 8 for bfloat16 rows (one 16-byte vector per thread).
static bool choose_shape(int V, int rows, int max_children, int kpad, int min_e, LaunchShape* out) {
  auto smem_for = [&](int e) {
    return static_cast<size_t>(2) * kThreads * e * 4 + kFixedSmemBytes + static_cast<size_t>(max_children) * kpad * 4;
  };
  auto cs_for = [&](int e) { int cs = (V + kThreads * e - 1) / (kThreads * e); return cs > 8 ? (cs > 16 ? 0 : 16) : cs; };
  int e = 0;
  if (g_cluster_override > 0) {
    for (int cand = min_e; cand <= 16; cand *= 2)
      if (static_cast<long long>(kThreads) * cand * g_cluster_override >= V) { e = cand; break; }
    if (e == 0) return false;
    out->cs = g_cluster_override;
  } else {
    // largest slice first; smaller slices (more CTAs) when the launch would not fill the GPU
    for (int cand = 16; cand >= min_e; cand /= 2) {
      int cs = cs_for(cand);
      if (cs == 0) continue;
      e = cand;
      if (static_cast<long long>(rows) * cs >= 2 * 148 || cand == min_e) break;
      int cs_next = cs_for(cand / 2);
      if (cs_next == 0) break;
    }
    if (e == 0) return false;
    out->cs = cs_for(e);
  }
  out->e = e;
  out->smem = smem_for(e);
  return out->smem <= 227 * 1024;
}

template <typename T, bool CFG, int E>
static cudaError_t launch_verify_e(const VerifyArgs& a, const LaunchShape& sh, cudaStream_t st) {
  auto kern = verify_nodes_kernel<T, CFG, E>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(sh.smem));
  if (e != cudaSuccess) return e;
  if (sh.cs > 8) {
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
    if (e != cudaSuccess) return e;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(a.B) * a.N * sh.cs, 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = sh.smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = sh.cs;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, a);
}

template <typename T, bool CFG>
static cudaError_t launch_verify(const VerifyArgs& a, const LaunchShape& sh, cudaStream_t st) {
  if (sh.e == 16) return launch_verify_e<T, CFG, 16>(a, sh, st);
  if (sh.e == 8) return launch_verify_e<T, CFG, 8>(a, sh, st);
  if constexpr (Vec<T>::N <= 4) {
    if (sh.e == 4) return launch_verify_e<T, CFG, 4>(a, sh, st);
  }
  return cudaErrorInvalidValue;
}

}  // namespace lantern

using namespace lantern;

extern "C" int32_t lantern_set_cluster_size(int32_t ctas_per_row) {
  int32_t old = g_cluster_override;
  if (ctas_per_row == 0 || ctas_per_row == 1 || ctas_per_row == 2 || ctas_per_row == 4 ||
      ctas_per_row == 8 || ctas_per_row == 16)
    g_cluster_override = ctas_per_row;
  return old;
}

extern "C" size_t lantern_verify_tree_workspace(const lantern_tree* tree, int32_t batch) {
  if (!tree || batch <= 0) return 0;
  const TreeDev* t = reinterpret_cast<const TreeDev*>(tree);
  return static_cast<size_t>(2) * batch * t->n_nodes * sizeof(int32_t);
}

extern "C" lantern_status lantern_verify_tree(
    const lantern_params* p, const lantern_tree* tree, const int32_t* nbr_idx, int32_t k_table,
    const void* target_cond, const void* target_uncond, const void* draft_cond, const void* draft_uncond,
    lantern_dtype dt, int64_t row_stride, int64_t seq_stride, int32_t batch, const int32_t* tokens,
    const float* u_accept, const float* u_resample, int32_t* accept_len, int32_t* out_tokens,
    int32_t* out_nodes, int32_t* node_next, int32_t* node_token, float* node_mass, float* node_thresh,
    int32_t* device_status, void* workspace, size_t workspace_bytes, void* stream) {
  if (!p || !tree || !target_cond || !tokens || !accept_len || !out_tokens || !out_nodes)
    return LANTERN_ERR_INVALID_ARG;
  const TreeDev* t = reinterpret_cast<const TreeDev*>(tree);
  if (batch <= 0 || p->vocab <= 0 || !(p->temperature > 0.f) || !(p->lambda >= 1.f)) return LANTERN_ERR_INVALID_ARG;
  if (dt != LANTERN_F32 && dt != LANTERN_BF16) return LANTERN_ERR_INVALID_ARG;
  if (t->n_internal > 0 && !draft_cond) return LANTERN_ERR_INVALID_ARG;
  if ((target_uncond != nullptr) != (draft_uncond != nullptr) && t->n_internal > 0) return LANTERN_ERR_INVALID_ARG;
  if (p->k < 0 || p->top_k_target < 0 || p->top_k_draft < 0) return LANTERN_ERR_INVALID_ARG;
  if (p->k > 0 && (!nbr_idx || p->k > k_table || p->n_codes <= 0 || k_table > p->n_codes - 1)) return LANTERN_ERR_INVALID_ARG;
  if (p->k > 1024) return LANTERN_ERR_UNSUPPORTED;
  const int V = p->vocab;
  const int allow_lo = p->allowed_begin, allow_hi = p->allowed_end == 0 ? V : p->allowed_end;
  if (allow_lo < 0 || allow_hi > V || allow_lo >= allow_hi) return LANTERN_ERR_INVALID_ARG;
  if (p->n_codes > 0 && (p->code_offset < 0 || static_cast<int64_t>(p->code_offset) + p->n_codes > V) && p->k > 0)
    return LANTERN_ERR_INVALID_ARG;
  if (p->step >> 62) return LANTERN_ERR_INVALID_ARG;
  const size_t esz = dt == LANTERN_F32 ? 4 : 2;
  if (row_stride < V || seq_stride < 0) return LANTERN_ERR_INVALID_ARG;
  if ((row_stride * esz) % 16 || (seq_stride * esz) % 16) return LANTERN_ERR_INVALID_ARG;
  const void* ptrs[4] = {target_cond, target_uncond, draft_cond, draft_uncond};
  for (const void* q : ptrs)
    if (q && (reinterpret_cast<uintptr_t>(q) % 16)) return LANTERN_ERR_INVALID_ARG;
  if (static_cast<int64_t>(batch) * t->n_nodes > (1 << 24)) return LANTERN_ERR_UNSUPPORTED;

  if (!node_next || !node_token) {
    size_t need = lantern_verify_tree_workspace(tree, batch);
    if (!workspace || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) % 256)) return LANTERN_ERR_WORKSPACE;
    int32_t* w = static_cast<int32_t*>(workspace);
    if (!node_next) node_next = w;
    if (!node_token) node_token = w + static_cast<size_t>(batch) * t->n_nodes;
  }

  VerifyArgs a;
  a.tc = target_cond; a.tu = target_uncond; a.dc = draft_cond; a.du = draft_uncond;
  a.row_stride = row_stride; a.seq_stride = seq_stride;
  a.tokens = tokens; a.u_acc = u_accept; a.u_res = u_resample;
  a.nbr = nbr_idx; a.k_table = k_table;
  a.use_bulk = (p->k > 0 && k_table % 4 == 0 && reinterpret_cast<uintptr_t>(nbr_idx) % 16 == 0) ? 1 : 0;
  a.first_child = t->d_first_child; a.n_child = t->d_n_child; a.order = t->d_order;
  a.B = batch; a.N = t->n_nodes; a.V = V;
  a.kpad = (p->k + 3) & ~3;
  a.g = p->cfg_scale; a.inv_tau = 1.0f / p->temperature; a.lambda = p->lambda;
  a.topk_t = p->top_k_target; a.topk_d = p->top_k_draft; a.k = p->k;
  a.code_offset = p->code_offset; a.n_codes = p->n_codes; a.allow_lo = allow_lo; a.allow_hi = allow_hi;
  a.seed = p->seed; a.step = p->step;
  a.node_next = node_next; a.node_token = node_token; a.node_mass = node_mass; a.node_thresh = node_thresh;
  a.status = device_status;
  LaunchShape sh;
  if (!choose_shape(V, batch * t->n_nodes, t->max_children, a.kpad, dt == LANTERN_F32 ? 4 : 8, &sh)) return LANTERN_ERR_UNSUPPORTED;
  a.SL = kThreads * sh.e;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const bool cfg = target_uncond != nullptr;
  cudaError_t e;
  if (dt == LANTERN_F32)
    e = cfg ? launch_verify<float, true>(a, sh, st) : launch_verify<float, false>(a, sh, st);
  else
    e = cfg ? launch_verify<__nv_bfloat16, true>(a, sh, st) : launch_verify<__nv_bfloat16, false>(a, sh, st);
  if (e != cudaSuccess) return LANTERN_ERR_CUDA;
  const int D1 = t->max_depth + 1;
  walk_kernel<<<(batch + 127) / 128, 128, 0, st>>>(node_next, node_token, tokens, batch, t->n_nodes, D1,
                                                    accept_len, out_tokens, out_nodes);
  if (cudaGetLastError() != cudaSuccess) return LANTERN_ERR_CUDA;
  return LANTERN_OK;
}
