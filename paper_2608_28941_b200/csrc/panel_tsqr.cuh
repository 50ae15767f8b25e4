// Panel Householder QR (Algorithm 2 line 7, geqrt semantics) without a grid barrier per column:
// a tall-skinny QR over the row slabs followed by a reconstruction of the Householder vectors.
//
//   1. Every leaf CTA factors its own slab of the panel in shared memory by Householder QR (no
//      communication), keeping its reflectors (V, and K = T V1^T) and handing its b x b factor R up.
//   2. Node CTAs stack up to f such factors, factor the stack the same way, and hand their R up, until
//      one root is left: a tree of Householder QRs, so the whole thing is a product of orthogonal
//      transformations however ill-conditioned the panel is.
//   3. Going back down, each node applies its reflectors to the b x b block X it received from its
//      parent (the root starts from the identity) and passes one b x b block to every child.  At a
//      leaf, Q_slab = Q_leaf [X; 0] are that slab's rows of the explicit orthonormal factor Q.
//   4. The reflectors of the panel itself are recovered from Q: with S the diagonal sign matrix of the
//      Householder convention, Q - [S; 0] = V U is an LU factorisation (V unit lower trapezoidal,
//      U upper triangular) whose L factor is exactly the matrix of Householder vectors of the panel,
//      and T = -U S V1^{-T} (V1 = top b x b block of V).  For ANY sign matrix S the result is orthogonal
//      (T^{-1} + T^{-T} = V^T V holds identically) and maps [S; 0] to Q; choosing S_jj = -sign of the
//      pivot met at step j of the elimination reproduces LAPACK's convention beta = -sign(alpha) ||x||,
//      because a reflector does not change when its column is scaled.  The first sign is taken from the
//      panel's own (0, 0) entry so that an exactly zero pivot keeps the sign of its zero.
//      Only the top b x b block needs the elimination (leaf 0); every other row is V = Q_row U^{-1}.
//
// Grid barriers: one per tree level up, one per level down, one after the elimination
// (2 * levels - 1 in all, plus two for the look-ahead fix-up), against one per column before.
// When a column below the diagonal is exactly zero LAPACK takes H = I (tau = 0); here that column of Q
// is completed orthogonally instead, which gives another valid factorisation of the same panel.
#pragma once

#include "panel.cuh"

namespace rrf {

// Optional phase trace (compiled in with -DRRF_TSQR_TRACE only; used to time the phases of the tree kernel)
#ifdef RRF_TSQR_TRACE
__device__ unsigned long long g_tsqr_trace[64];
__device__ __forceinline__ void tsqr_stamp(int slot, bool who) {
  if (who && threadIdx.x == 0) {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    g_tsqr_trace[slot] = t;
  }
}
#define RRF_STAMP(slot, who) tsqr_stamp(slot, who)
#define RRF_CSTAMP(slot, who) if ((who) && threadIdx.x == 0) g_tsqr_trace[slot] = (unsigned long long)clock64()
#define RRF_CSTAMP_T(slot, who, thr) if ((who) && threadIdx.x == (thr)) g_tsqr_trace[slot] = (unsigned long long)clock64()
#else
#define RRF_CSTAMP_T(slot, who, thr)
#define RRF_STAMP(slot, who)
#define RRF_CSTAMP(slot, who)
#endif

// log2(b) rounds that turn tau (diagonal of Ts) and the Gram entries v_c^T v_j (strictly lower part of
// Ts, pitch b + 1) into the compact-WY factor T in the upper triangle of Ts (see tfactor_kernel).
__device__ __forceinline__ void tfactor_rounds(double* Ts, double* Ms, int b) {
  const int pitch = b + 1, mp = b / 2 + 1;
  const int tid = threadIdx.x, nthr = blockDim.x;
  for (int s = 1; s < b; s <<= 1) {
    const int per_level = b * s / 2;
    const int ls = 31 - __clz(s);
    for (int idx = tid; idx < per_level; idx += nthr) {
      const int q = idx >> (2 * ls), rc = idx & (s * s - 1), r = rc >> ls, c = rc & (s - 1);
      const int o = 2 * s * q;
      const double* ga = Ts + (size_t)(o + s) * pitch + (o + r);
      const double* tb = Ts + (size_t)(o + s) * pitch + (o + s + c);
      double a0 = 0.0, a1 = 0.0;
      int k = 0;
      for (; k + 1 <= c; k += 2) {
        a0 += ga[k * pitch] * tb[k * pitch];
        a1 += ga[(k + 1) * pitch] * tb[(k + 1) * pitch];
      }
      if (k <= c) a0 += ga[k * pitch] * tb[k * pitch];
      Ms[(s * q + r) * mp + c] = a0 + a1;
    }
    __syncthreads();
    for (int idx = tid; idx < per_level; idx += nthr) {
      const int q = idx >> (2 * ls), rc = idx & (s * s - 1), r = rc >> ls, c = rc & (s - 1);
      const int o = 2 * s * q;
      const double* ta = Ts + (size_t)(o + r) * pitch + o;
      const double* mb = Ms + (size_t)(s * q) * mp + c;
      double a0 = 0.0, a1 = 0.0;
      int k = r;
      for (; k + 1 < s; k += 2) {
        a0 += ta[k] * mb[k * mp];
        a1 += ta[k + 1] * mb[(k + 1) * mp];
      }
      if (k < s) a0 += ta[k] * mb[k * mp];
      Ts[(o + r) * pitch + (o + s + c)] = -(a0 + a1);
    }
    __syncthreads();
  }
}

// In-place inverses of both triangles of a b x b array A (pitch pa) that holds a unit lower triangular
// L strictly below the diagonal and an upper triangular U on and above it: on return the strictly lower
// part is that of L^{-1} and the upper part is U^{-1}.  Recursive doubling: with the diagonal blocks of
// size s inverted, the off-diagonal block of each pair of them is -inv11 * A12 * inv22 (upper) or
// -inv22 * A21 * inv11 (lower).  `tmp` holds 2 * (b/2) * (b/2 + 1) doubles.
__device__ __forceinline__ void tri_inverse_both(double* A, int pa, double* tmp, int b) {
  const int tid = threadIdx.x, nthr = blockDim.x;
  const int mp = b / 2 + 1;
  double* Mu = tmp;
  double* Ml = tmp + (size_t)(b / 2) * mp;
  for (int i = tid; i < b; i += nthr) A[i * pa + i] = 1.0 / A[i * pa + i];
  __syncthreads();
  for (int s = 1; s < b; s <<= 1) {
    const int per_level = b * s / 2;
    const int ls = 31 - __clz(s);
    // Mu = A12 * inv22 (upper), Ml = A21 * inv11 (lower; inv11 has a unit diagonal)
    for (int idx = tid; idx < per_level; idx += nthr) {
      const int q = idx >> (2 * ls), rc = idx & (s * s - 1), r = rc >> ls, c = rc & (s - 1);
      const int o = 2 * s * q;
      double au = 0.0;
      for (int k = 0; k <= c; ++k) au += A[(o + r) * pa + (o + s + k)] * A[(o + s + k) * pa + (o + s + c)];
      Mu[(s * q + r) * mp + c] = au;
      double al = A[(o + s + r) * pa + (o + c)];                 // k = c: unit diagonal of inv11
      for (int k = c + 1; k < s; ++k) al += A[(o + s + r) * pa + (o + k)] * A[(o + k) * pa + (o + c)];
      Ml[(s * q + r) * mp + c] = al;
    }
    __syncthreads();
    for (int idx = tid; idx < per_level; idx += nthr) {
      const int q = idx >> (2 * ls), rc = idx & (s * s - 1), r = rc >> ls, c = rc & (s - 1);
      const int o = 2 * s * q;
      double au = 0.0;
      for (int k = r; k < s; ++k) au += A[(o + r) * pa + (o + k)] * Mu[(s * q + k) * mp + c];
      double al = Ml[(s * q + r) * mp + c];                      // k = r: unit diagonal of inv22
      for (int k = 0; k < r; ++k) al += A[(o + s + r) * pa + (o + s + k)] * Ml[(s * q + k) * mp + c];
      A[(o + r) * pa + (o + s + c)] = -au;
      A[(o + s + r) * pa + (o + c)] = -al;
    }
    __syncthreads();
  }
}

// ------------------------------------------------------------------------------------------
// Householder QR of a matrix that one CTA holds in shared memory: S is column-major with pitch Rp and
// RS = 32 * QMAX * RH rows, zero filled below its last row; the pivot of column j is row row0 + j and
// rows above row0 are left alone.  Same formulation as the grid-wide kernel (one pass per column gives
// the norm, the products for the reflector's application and a row of V^T V), with the sums staying
// inside the CTA.  On return S holds V (explicit ones and zeros), Ts (pitch b + 1) holds tau on its
// diagonal and v_c^T v_j (c < j) below it, and Rout (global, row-major b x b) holds R.
// ------------------------------------------------------------------------------------------
template <int QMAX, int RH>
__device__ __forceinline__ void cta_qr(double* S, int Rp, int b, int row0, double* w_s, double* p_s, double* sc_s,
                                       double* Ts, double* __restrict__ Rout) {
  constexpr int NT = kPanelThreads, NW = NT / 32;
  constexpr int NWC = NW / RH;
  constexpr int CG = 4;
  constexpr int RS = 32 * QMAX * RH;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int rg = warp / NWC, wc = warp - rg * NWC;
  const int tp = b + 1;
  double tau_prev = 0.0;
  for (int j = 0; j < b; ++j) {
    const int pr = row0 + j;
    double* Sj = S + (size_t)j * Rp;
    const double* Sjm1 = S + (size_t)(j > 0 ? j - 1 : 0) * Rp;
    RRF_CSTAMP(40, j == 8 && blockIdx.x == 0);
    if (j > 0 && tau_prev != 0.0) {
      const double f = tau_prev * w_s[j];
      for (int r = tid; r < RS; r += NT)
        if (r >= pr) Sj[r] -= f * Sjm1[r];
    }
    __syncthreads();
    RRF_CSTAMP(41, j == 8 && blockIdx.x == 0);
    {
      double yj[QMAX], vp[QMAX];
      const int rbase = rg * (32 * QMAX) + lane;
#pragma unroll
      for (int q = 0; q < QMAX; ++q) {
        const int r = rbase + 32 * q;
        yj[q] = r > pr ? Sj[r] : 0.0;
        vp[q] = r >= pr ? Sjm1[r] : 0.0;
      }
      const bool pending = (j > 0) && (tau_prev != 0.0);
      for (int c0 = wc; c0 < b; c0 += NWC * CG) {
        double x[CG][QMAX], acc[CG];
#pragma unroll
        for (int u = 0; u < CG; ++u) {
          const int c = c0 + u * NWC;
          const double* Sc = S + (size_t)(c < b ? c : 0) * Rp + rbase;
#pragma unroll
          for (int q = 0; q < QMAX; ++q) x[u][q] = Sc[32 * q];
        }
#pragma unroll
        for (int u = 0; u < CG; ++u) {
          const int c = c0 + u * NWC;
          const bool upd = pending && c > j && c < b;
          double a = 0.0;
          if (upd) {
            const double f = tau_prev * w_s[c];
            double* Sc = S + (size_t)c * Rp + rbase;
#pragma unroll
            for (int q = 0; q < QMAX; ++q) {
              const double xv = x[u][q] - f * vp[q];
              Sc[32 * q] = xv;
              a += yj[q] * xv;
            }
          } else {
#pragma unroll
            for (int q = 0; q < QMAX; ++q) a += yj[q] * x[u][q];
          }
          acc[u] = c < b ? a : 0.0;
        }
        const double tot = warp_sum4(acc, lane);
        const int u = ((lane >> 4) << 1) | ((lane >> 3) & 1);
        if ((lane & 7) == 0 && c0 + u * NWC < b) p_s[rg * b + c0 + u * NWC] = tot;
      }
    }
    RRF_CSTAMP(42, j == 8 && blockIdx.x == 0);
    __syncthreads();
    RRF_CSTAMP(43, j == 8 && blockIdx.x == 0);
    // scalars of reflector j, computed by every thread that needs them (no further exchange)
    if (tid < b) {
      double pj = p_s[j], pc = p_s[tid];
#pragma unroll
      for (int h = 1; h < RH; ++h) {
        pj += p_s[h * b + j];
        pc += p_s[h * b + tid];
      }
      const double alpha = Sj[pr], piv = S[(size_t)tid * Rp + pr];
      double tau = 0.0, rdenom = 0.0, beta = alpha;
      if (pj != 0.0) {
        beta = -copysign(sqrt(alpha * alpha + pj), alpha);
        tau = (beta - alpha) / beta;
        rdenom = 1.0 / (alpha - beta);
      }
      const double wv = piv + pc * rdenom;
      double rv;
      if (tid == j) {
        sc_s[0] = tau;
        sc_s[1] = rdenom;
        Ts[j * tp + j] = tau;
        rv = beta;
      } else {
        w_s[tid] = wv;
        if (tid < j) Ts[j * tp + tid] = wv;
        rv = tid < j ? 0.0 : piv - tau * wv;
      }
      Rout[(size_t)j * b + tid] = rv;
    }
    RRF_CSTAMP(44, j == 8 && blockIdx.x == 0);
    __syncthreads();
    RRF_CSTAMP(45, j == 8 && blockIdx.x == 0);
    const double rdenom = sc_s[1];
    for (int r = tid; r < RS; r += NT) Sj[r] = r > pr ? Sj[r] * rdenom : (r == pr ? 1.0 : 0.0);
    tau_prev = sc_s[0];
    __syncthreads();
    RRF_CSTAMP(46, j == 8 && blockIdx.x == 0);
  }
}

// ------------------------------------------------------------------------------------------
// Look-ahead fix-up (the paper's "Update Panel"): S <- P - Vp (Tp^T (Vp^T P)) for the slabs of the GL
// leaf CTAs, on the tensor cores (FP64 m16n8k8), with two grid barriers (`gb`) between its three
// phases.  `aux` holds panel_fix_doubles(b) doubles.  CTAs that hold no slab pass leaf = false and only
// take part in the barriers.
// ------------------------------------------------------------------------------------------
template <typename T, typename Barrier>
__device__ __forceinline__ bool panel_fixup(double* S, int Rp, int nloc, int gr0, int b, int GL, int cta, bool leaf,
                                            const PanelFix& fix, double* aux, Barrier gb) {
  constexpr int NT = kPanelThreads, NW = NT / 32;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, t = lane & 3;
  const int lb = 31 - __clz(b);
  double* Vst = aux;                                   // [kFixChunk][b + 8] or [kFixChunk][b + 4]
  double* Mst = Vst + (size_t)kFixChunk * (b + 8);     // [b][b + 8]: Tp (pitch b + 1), then M
  const T* Vp = reinterpret_cast<const T*>(fix.Vp);
  const T* Tp = reinterpret_cast<const T*>(fix.Tp);
  const int nch = leaf ? (nloc + kFixChunk - 1) / kFixChunk : 0;
  constexpr int EPT = 4;                               // kFixChunk * 64 / NT staged elements per thread
  T pre[EPT];
  auto fetch = [&](int ch) {                           // rows of Vp for chunk ch, into registers
#pragma unroll
    for (int e = 0; e < EPT; ++e) {
      const int idx = tid + e * NT, rr = idx >> lb, c = idx & (b - 1), r = ch * kFixChunk + rr;
      pre[e] = (rr < kFixChunk && r < nloc) ? Vp[(size_t)(gr0 + r) * fix.ldvp + c] : T(0);
    }
  };
  auto stash = [&](int pitch) {                        // registers -> Vst[rr][c]
#pragma unroll
    for (int e = 0; e < EPT; ++e) {
      const int idx = tid + e * NT, rr = idx >> lb, c = idx & (b - 1);
      if (rr < kFixChunk) Vst[rr * pitch + c] = (double)pre[e];
    }
  };
  if (leaf) {
    // Tp into shared memory (pitch b + 1), zero below the diagonal
    for (int idx = tid; idx < b * b; idx += NT) {
      const int l = idx >> lb, k = idx & (b - 1);
      Mst[l * (b + 1) + k] = l <= k ? (double)Tp[(size_t)l * fix.ldtp + k] : 0.0;
    }
    // Phase 1: Gpart[cta] = Vp[slab]^T S.  Warp (mt, np) owns G[16 mt .., 16 np ..] (two n-tiles).
    const int nmt = b >> 4;
    const bool act = warp < nmt * nmt;
    const int mt = act ? warp / nmt : 0, np = act ? warp - mt * nmt : 0;
    const int PV = b + 8;
    double acc[2][4];
#pragma unroll
    for (int i = 0; i < 2; ++i)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[i][e] = 0.0;
    if (nch > 0) fetch(0);
    for (int ch = 0; ch < nch; ++ch) {
      __syncthreads();
      stash(PV);
      __syncthreads();
      if (ch + 1 < nch) fetch(ch + 1);
      if (act) {
        const int rc = ch * kFixChunk;
#pragma unroll
        for (int ks = 0; ks < kFixChunk / 8; ++ks) {
          const double* va = Vst + (ks * 8 + t) * PV + mt * 16 + g;
          const double af[4] = {va[0], va[8], va[4 * PV], va[4 * PV + 8]};
#pragma unroll
          for (int i = 0; i < 2; ++i) {
            const double* sb = S + (size_t)((np * 2 + i) * 8 + g) * Rp + rc + ks * 8 + t;
            const double bf[2] = {sb[0], sb[4]};
            mma16x8x8(acc[i], af, bf);
          }
        }
      }
    }
    if (act) {
      double* gp = fix.Gpart + (size_t)cta * b * b;
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        const int col = (np * 2 + i) * 8 + 2 * t, row = mt * 16 + g;
        gp[(size_t)row * b + col] = acc[i][0];
        gp[(size_t)row * b + col + 1] = acc[i][1];
        gp[(size_t)(row + 8) * b + col] = acc[i][2];
        gp[(size_t)(row + 8) * b + col + 1] = acc[i][3];
      }
    }
  }
  if (!gb()) return false;
  // Phase 2: leaf c owns columns c, c + GL, ... of G = sum of the partials (in CTA order) and of
  // M = Tp^T G, column by column: M[k][c2] = sum_{l <= k} Tp[l][k] G[l][c2].
  if (leaf) {
    const int ncol = cta < b ? (b - cta + GL - 1) / GL : 0;
    double* Gs = Vst;                                  // up to kFixChunk columns of G at a time
    for (int q0 = 0; q0 < ncol; q0 += kFixChunk) {
      const int nq = min(kFixChunk, ncol - q0);
      __syncthreads();
      for (int idx = tid; idx < nq * b; idx += NT) {
        const int q = idx >> lb, l = idx & (b - 1), c2 = cta + (q0 + q) * GL;
        const double* gp = fix.Gpart + (size_t)l * b + c2;
        double sum = 0.0;
        int x = 0;
        for (; x + 8 <= GL; x += 8) {
          double v[8];
#pragma unroll
          for (int e = 0; e < 8; ++e) v[e] = __ldcg(gp + (size_t)(x + e) * b * b);
#pragma unroll
          for (int e = 0; e < 8; ++e) sum += v[e];
        }
        for (; x < GL; ++x) sum += __ldcg(gp + (size_t)x * b * b);
        Gs[q * b + l] = sum;
      }
      __syncthreads();
      for (int idx = tid; idx < nq * b; idx += NT) {
        const int q = idx >> lb, k = idx & (b - 1), c2 = cta + (q0 + q) * GL;
        double s0 = 0.0, s1 = 0.0;
        int l = 0;
        for (; l + 1 <= k; l += 2) {
          s0 += Mst[l * (b + 1) + k] * Gs[q * b + l];
          s1 += Mst[(l + 1) * (b + 1) + k] * Gs[q * b + l + 1];
        }
        if (l <= k) s0 += Mst[l * (b + 1) + k] * Gs[q * b + l];
        fix.M[(size_t)k * b + c2] = s0 + s1;
      }
    }
  }
  if (!gb()) return false;
  // Phase 3: S -= Vp[slab] M.  A task is a 16-row x 8-column tile of a chunk.
  if (leaf) {
    const int PV = b + 4, PM = b + 8;
    for (int idx = tid; idx < b * b; idx += NT) Mst[(idx >> lb) * PM + (idx & (b - 1))] = __ldcg(fix.M + idx);
    const int ntask = (kFixChunk / 16) * (b >> 3);
    if (nch > 0) fetch(0);
    for (int ch = 0; ch < nch; ++ch) {
      __syncthreads();
      stash(PV);
      __syncthreads();
      if (ch + 1 < nch) fetch(ch + 1);
      const int rc = ch * kFixChunk;
      for (int task = warp; task < ntask; task += NW) {
        const int r0 = (task & 1) * 16, n0 = (task >> 1) * 8;
        double acc[4] = {0.0, 0.0, 0.0, 0.0};
        for (int k0 = 0; k0 < b; k0 += 8) {
          const double* va = Vst + (r0 + g) * PV + k0 + t;
          const double af[4] = {va[0], va[8 * PV], va[4], va[8 * PV + 4]};
          const double* mb = Mst + (k0 + t) * PM + n0 + g;
          const double bf[2] = {mb[0], mb[4 * PM]};
          mma16x8x8(acc, af, bf);
        }
        double* s0 = S + (size_t)(n0 + 2 * t) * Rp + rc + r0 + g;
        s0[0] -= acc[0];
        s0[Rp] -= acc[1];
        s0[8] -= acc[2];
        s0[Rp + 8] -= acc[3];
      }
    }
    __syncthreads();
  }
  return true;
}

// ------------------------------------------------------------------------------------------
// Small dense helpers on the FP64 tensor cores (m16n8k8).  Operands are fetched element by element
// through functors, so a triangular or implicit operand is just a functor that returns zeros and ones.
// ------------------------------------------------------------------------------------------
// C (b x b) = A (b x b) * B (b x b); tiles of 16 x 8 are dealt to the warps of the CTA.
template <typename FA, typename FB, typename ST>
__device__ __forceinline__ void small_mma(int b, FA fa, FB fb, ST st) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, g = lane >> 2, t = lane & 3;
  const int nnt = b >> 3, ntile = (b >> 4) * nnt;
  for (int tile = warp; tile < ntile; tile += kPanelThreads / 32) {
    const int m0 = (tile / nnt) * 16, n0 = (tile % nnt) * 8;
    double acc[4] = {0.0, 0.0, 0.0, 0.0};
    for (int k0 = 0; k0 < b; k0 += 8) {
      const double af[4] = {fa(m0 + g, k0 + t), fa(m0 + g + 8, k0 + t), fa(m0 + g, k0 + t + 4), fa(m0 + g + 8, k0 + t + 4)};
      const double bf[2] = {fb(k0 + t, n0 + g), fb(k0 + t + 4, n0 + g)};
      mma16x8x8(acc, af, bf);
    }
    st(m0 + g, n0 + 2 * t, acc[0], acc[1]);
    st(m0 + g + 8, n0 + 2 * t, acc[2], acc[3]);
  }
}

// For the rows [r_begin, r_end) (multiples of 16) of a matrix held column-major in shared memory (pitch
// Rp, b columns): epi(r, n, acc) with acc = sum_c S[r][c] * Mb[c][n], Mb in shared memory with pitch pm.
// A warp reads all of its 16 rows into registers before it calls epi, so epi may overwrite them.
template <typename EPI>
__device__ __forceinline__ void slab_mma(const double* S, int Rp, int r_begin, int r_end, int b, const double* Mb, int pm,
                                         EPI epi) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, g = lane >> 2, t = lane & 3;
  const int nks = b >> 3;
  for (int r0 = r_begin + 16 * warp; r0 < r_end; r0 += 16 * (kPanelThreads / 32)) {
    double a[8][4];
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
      if (ks < nks) {
        const double* p = S + (size_t)(ks * 8 + t) * Rp + r0 + g;
        a[ks][0] = p[0];
        a[ks][1] = p[8];
        a[ks][2] = p[4 * (size_t)Rp];
        a[ks][3] = p[4 * (size_t)Rp + 8];
      }
    }
    for (int n0 = 0; n0 < b; n0 += 8) {
      double acc[4] = {0.0, 0.0, 0.0, 0.0};
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        if (ks < nks) {
          const double* mb = Mb + (ks * 8 + t) * pm + n0 + g;
          const double bf[2] = {mb[0], mb[4 * pm]};
          mma16x8x8(acc, a[ks], bf);
        }
      }
      epi(r0 + g, n0 + 2 * t, acc[0], acc[1]);
      epi(r0 + g + 8, n0 + 2 * t, acc[2], acc[3]);
    }
  }
}

// Shape of the reduction tree and the scratch of the kernel below.  CTAs [off[l], off[l] + cnt[l]) form
// level l (0: leaves, nlev - 1: the root); node q of level l > 0 stacks the factors of nodes
// q*f .. q*f + f - 1 of level l - 1.  var[l]: shared-memory tiling of that level's factorisation.
struct TsqrPlan {
  int nlev, f, R;          // levels, fan-in, rows of a leaf slab
  int off[6], cnt[6], var[6];
};
struct TsqrScratch {
  double* Rbuf;            // [CTA][b*b]: the CTA's R factor on the way up; a leaf's M = K X on the way down
  double* Xbuf;            // [CTA][b*b]: the block of the orthonormal factor handed down to the CTA
  double* Kbuf;            // [CTA][b*b]: K^T with K = T V1^T of the CTA's own reflectors; later X U^{-1}
  double* Ubuf;            // [2][b*b]: U^{-1}, U of the reconstruction
};

__device__ __forceinline__ void cta_qr_variant(int var, double* S, int Rp, int b, int row0, double* w_s, double* p_s,
                                               double* sc_s, double* Ts, double* Rout) {
#ifdef RRF_ONE_VARIANT
  cta_qr<5, 2>(S, Rp, b, row0, w_s, p_s, sc_s, Ts, Rout);
  return;
#endif
  switch (var) {
    case 0: cta_qr<2, 1>(S, Rp, b, row0, w_s, p_s, sc_s, Ts, Rout); break;
    case 1: cta_qr<4, 1>(S, Rp, b, row0, w_s, p_s, sc_s, Ts, Rout); break;
    case 2: cta_qr<7, 1>(S, Rp, b, row0, w_s, p_s, sc_s, Ts, Rout); break;
    case 3: cta_qr<5, 2>(S, Rp, b, row0, w_s, p_s, sc_s, Ts, Rout); break;
    default: cta_qr<8, 2>(S, Rp, b, row0, w_s, p_s, sc_s, Ts, Rout); break;
  }
}
__host__ __device__ constexpr int tsqr_variant_rows(int var) {
  return var == 0 ? 64 : var == 1 ? 128 : var == 2 ? 224 : var == 3 ? 320 : 512;
}

// ------------------------------------------------------------------------------------------
// The kernel.  Cooperative launch, one CTA per leaf slab and per tree node, all co-resident.  Dynamic
// shared memory: the slab / stack S [b][Rp], an auxiliary region of panel_fix_doubles(b) doubles (fix-up
// staging, then T's workspace, then the small matrices of the way down), and 5 b + 4 scalars.
// ------------------------------------------------------------------------------------------
__host__ __device__ constexpr int tsqr_small_doubles(int b) { return 5 * b + 4; }

template <typename T>
__global__ void __launch_bounds__(kPanelThreads)
    panel_tsqr_kernel(const T* __restrict__ Y, PanelSource src_fused, PanelSource src_alt, const int* __restrict__ fused_flag,
                      int rows, int b, int Rp, T* __restrict__ V, long long ldv, TsqrPlan plan, TsqrScratch sc,
                      unsigned* bar, Ctrl* ctrl, const int* done_flag, PanelFix fix, unsigned bar_base,
                      T* __restrict__ Tout, long long ldt) {
  if (*reinterpret_cast<const volatile int*>(done_flag) || *reinterpret_cast<const volatile int*>(&ctrl->status) < 0) return;
  const bool use_alt = fused_flag != nullptr && *fused_flag == 0;
  const PanelSource src = use_alt ? src_alt : src_fused;
  extern __shared__ double psm[];
  double* S = psm;                                   // [b][Rp]
  double* aux = S + (size_t)b * Rp;                  // panel_fix_doubles(b)
  double* w_s = aux + panel_fix_doubles(b);          // [b]
  double* p_s = w_s + b;                             // [2][b]
  double* sgn_s = p_s + 2 * b;                       // [b]: signs of the reconstruction
  double* sc_s = sgn_s + b;                          // [4]

  constexpr int NT = kPanelThreads;
  const int tid = threadIdx.x;
  const int id = blockIdx.x, ncta = gridDim.x;
  const int lb = 31 - __clz(b);
  const int bb = b * b;
  int lv = 0;
  while (lv + 1 < plan.nlev && id >= plan.off[lv + 1]) ++lv;
  const int q = id - plan.off[lv];                   // index within the level
  const bool leaf = lv == 0;
  const int GL = plan.cnt[0];
  const int row0 = fix.enabled ? b : 0;              // slab rows are numbered from b rows above the panel
  const int ext = rows + row0;
  const int gr0 = q * plan.R;                        // leaves: first row of the slab
  const int nloc = leaf ? max(0, min(plan.R, ext - gr0)) : 0;
  const int lrow0 = (leaf && q == 0) ? row0 : 0;     // pivot offset of this CTA's own factorisation
  const int RS = tsqr_variant_rows(plan.var[lv]);
  unsigned nbar = 0;
  auto gb = [&]() { return grid_barrier(bar, bar_base + (++nbar) * (unsigned)ncta, ctrl); };
  double y00 = 0.0;

  if (leaf) {
    for (int idx = tid; idx < nloc * b; idx += NT) {
      const int r = idx >> lb, c = idx & (b - 1);
      S[(size_t)c * Rp + r] = panel_entry(Y, src, gr0 + r - row0, c, b);
    }
    const int npad = RS - nloc;
    for (int idx = tid; idx < npad * b; idx += NT) {
      const int c = idx / npad, r = nloc + (idx - c * npad);
      S[(size_t)c * Rp + r] = 0.0;
    }
    __syncthreads();
  }
  if (fix.enabled && !panel_fixup<T>(S, Rp, nloc, gr0, b, GL, q, leaf, fix, aux, gb)) return;
  if (leaf && q == 0) y00 = S[row0];                 // the panel's (0, 0) entry decides the first sign
  RRF_STAMP(0, id == 0);

  double* Ts = aux;                                  // [b][b + 1]
  double* Ms = Ts + (size_t)b * (b + 1);             // [b/2][b/2 + 1]
  double* myR = sc.Rbuf + (size_t)id * bb;
  double* myK = sc.Kbuf + (size_t)id * bb;
  const double* myX = sc.Xbuf + (size_t)id * bb;
  int nc = 0;                                        // nodes: number of children

  // ---- up: factor the slab (leaves), then level by level the stacks of R factors
  for (int l = 0; l < plan.nlev; ++l) {
    if (lv == l) {
      if (l > 0) {
        nc = min(plan.f, plan.cnt[l - 1] - q * plan.f);
        const double* ch = sc.Rbuf + (size_t)(plan.off[l - 1] + q * plan.f) * bb;
        for (int idx = tid; idx < nc * bb; idx += NT) {
          const int r = idx >> lb, c = idx & (b - 1);          // r = child * b + row
          S[(size_t)c * Rp + r] = __ldcg(ch + idx);
        }
        const int npad = RS - nc * b;
        for (int idx = tid; idx < npad * b; idx += NT) {
          const int c = idx / npad, r = nc * b + (idx - c * npad);
          S[(size_t)c * Rp + r] = 0.0;
        }
        __syncthreads();
      }
      cta_qr_variant(plan.var[l], S, Rp, b, lrow0, w_s, p_s, sc_s, Ts, myR);
      RRF_STAMP(1 + 4 * l, q == 0);
      tfactor_rounds(Ts, Ms, b);
      RRF_STAMP(2 + 4 * l, q == 0);
      // K = T V1^T (upper triangular), stored transposed
      small_mma(b,
                [&](int c, int i) { return i >= c ? Ts[c * (b + 1) + i] : 0.0; },
                [&](int i, int r) { return S[(size_t)i * Rp + lrow0 + r]; },
                [&](int c, int r, double v0, double v1) {
                  myK[(size_t)r * b + c] = v0;
                  myK[(size_t)(r + 1) * b + c] = v1;
                });
      __syncthreads();
    }
    RRF_STAMP(3 + 4 * l, lv == l && q == 0);
    if (l + 1 < plan.nlev && !gb()) return;
    RRF_STAMP(4 + 4 * l, id == 0);
  }

  // ---- down: every node turns the block it received into one block per child
  double* Mb = aux;                                  // [b][b + 8]
  const int pm = b + 8;
  const bool root = lv == plan.nlev - 1;
  for (int l = plan.nlev - 1; l >= 1; --l) {
    if (lv == l) {
      // M = K X (X = I at the root)
      small_mma(b,
                [&](int c, int i) { return myK[(size_t)i * b + c]; },
                [&](int i, int n) { return root ? (i == n ? 1.0 : 0.0) : __ldcg(myX + (size_t)i * b + n); },
                [&](int c, int n, double v0, double v1) {
                  Mb[c * pm + n] = v0;
                  Mb[c * pm + n + 1] = v1;
                });
      __syncthreads();
      double* chX = sc.Xbuf + (size_t)(plan.off[l - 1] + q * plan.f) * bb;
      slab_mma(S, Rp, 0, nc * b, b, Mb, pm, [&](int r, int n, double a0, double a1) {
        double x0 = 0.0, x1 = 0.0;
        if (r < b) {
          if (root) {
            x0 = r == n ? 1.0 : 0.0;
            x1 = r == n + 1 ? 1.0 : 0.0;
          } else {
            x0 = __ldcg(myX + (size_t)r * b + n);
            x1 = __ldcg(myX + (size_t)r * b + n + 1);
          }
        }
        chX[(size_t)r * b + n] = x0 - a0;              // row r of the stack = row r % b of child r / b
        chX[(size_t)r * b + n + 1] = x1 - a1;
      });
    }
    if (!gb()) return;
    RRF_STAMP(24 + l, id == 0);
  }

  // ---- leaves: M = K X; leaf 0 recovers the top block of the Householder vectors, U and T
  const bool xid = plan.nlev == 1;                   // a single leaf is its own root: X = I
  const double* Ui = sc.Ubuf;                        // U^{-1}
  double* Ug = sc.Ubuf + bb;                         // U
  if (leaf) {
    const double r00 = __ldcg(sc.Rbuf + (size_t)plan.off[plan.nlev - 1] * bb);   // R[0][0] of the whole panel
    __syncthreads();
    small_mma(b,
              [&](int c, int i) { return myK[(size_t)i * b + c]; },
              [&](int i, int n) { return xid ? (i == n ? 1.0 : 0.0) : __ldcg(myX + (size_t)i * b + n); },
              [&](int c, int n, double v0, double v1) {
                myR[(size_t)c * b + n] = v0;
                myR[(size_t)c * b + n + 1] = v1;
              });
    __syncthreads();
    if (q == 0) {
      const int pa = b + 1;
      double* A = aux;                               // [b][b + 1]
      double* tmp = A + (size_t)b * pa;              // 2 * (b/2) * (b/2 + 1)
      // Q1 = X - V1 M: the top b x b block of the orthonormal factor
      small_mma(b,
                [&](int r, int c) { return S[(size_t)c * Rp + row0 + r]; },
                [&](int c, int n) { return myR[(size_t)c * b + n]; },
                [&](int r, int n, double v0, double v1) {
                  const double x0 = xid ? (r == n ? 1.0 : 0.0) : __ldcg(myX + (size_t)r * b + n);
                  const double x1 = xid ? (r == n + 1 ? 1.0 : 0.0) : __ldcg(myX + (size_t)r * b + n + 1);
                  A[r * pa + n] = x0 - v0;
                  A[r * pa + n + 1] = x1 - v1;
                });
      __syncthreads();
      RRF_STAMP(32, true);
      // Q1 - S = L1 U with S_jj = -sign(pivot) chosen as the elimination goes
      for (int j = 0; j < b; ++j) {
        const double a = A[j * pa + j];
        const double s = j == 0 ? -copysign(1.0, y00) * copysign(1.0, r00) : -copysign(1.0, a);
        const double piv = a - s;
        const double rcp = 1.0 / piv;
        __syncthreads();                             // everyone has read the pivot
        for (int i = j + 1 + tid; i < b; i += NT) A[i * pa + j] *= rcp;
        if (tid == 0) {
          A[j * pa + j] = piv;
          sgn_s[j] = s;
        }
        __syncthreads();
        const int nn = b - 1 - j;
        for (int idx = tid; idx < nn * nn; idx += NT) {
          const int i = j + 1 + idx / nn, c = j + 1 + idx % nn;
          A[i * pa + c] -= A[i * pa + j] * A[j * pa + c];
        }
        __syncthreads();
      }
      for (int idx = tid; idx < bb; idx += NT) {
        const int r = idx >> lb, c = idx & (b - 1);
        V[(size_t)r * ldv + c] = c < r ? (T)A[r * pa + c] : (c == r ? T(1) : T(0));
        Ug[idx] = c >= r ? A[r * pa + c] : 0.0;
      }
      __syncthreads();
      RRF_STAMP(33, true);
      tri_inverse_both(A, pa, tmp, b);
      RRF_STAMP(34, true);
      for (int idx = tid; idx < bb; idx += NT) {
        const int r = idx >> lb, c = idx & (b - 1);
        sc.Ubuf[idx] = c >= r ? A[r * pa + c] : 0.0;
      }
      // T = -U S L1^{-T}
      small_mma(b,
                [&](int r, int i) { return i >= r ? Ug[(size_t)r * b + i] * sgn_s[i] : 0.0; },
                [&](int i, int c) { return i < c ? A[c * pa + i] : (i == c ? 1.0 : 0.0); },
                [&](int r, int c, double v0, double v1) {
                  Tout[(size_t)r * ldt + c] = c >= r ? (T)(-v0) : T(0);
                  Tout[(size_t)r * ldt + c + 1] = c + 1 >= r ? (T)(-v1) : T(0);
                });
    }
  }
  RRF_STAMP(35, id == 0);
  if (!gb()) return;
  if (!leaf) return;
  RRF_STAMP(36, id == 0);

  // ---- every leaf: V[slab] = Q[slab] U^{-1} = [X U^{-1}; 0] - V_leaf (M U^{-1})
  small_mma(b,
            [&](int c, int k) { return myR[(size_t)c * b + k]; },
            [&](int k, int n) { return __ldcg(Ui + (size_t)k * b + n); },
            [&](int c, int n, double v0, double v1) {
              Mb[c * pm + n] = v0;
              Mb[c * pm + n + 1] = v1;
            });
  small_mma(b,
            [&](int r, int k) { return xid ? (r == k ? 1.0 : 0.0) : __ldcg(myX + (size_t)r * b + k); },
            [&](int k, int n) { return __ldcg(Ui + (size_t)k * b + n); },
            [&](int r, int n, double v0, double v1) {
              myK[(size_t)r * b + n] = v0;
              myK[(size_t)r * b + n + 1] = v1;
            });
  __syncthreads();
  RRF_STAMP(37, id == 0);
  const int first_out = lrow0 + (q == 0 ? b : 0);    // leaf 0 wrote its top block from L1
  slab_mma(S, Rp, 0, (nloc + 15) & ~15, b, Mb, pm, [&](int r, int n, double a0, double a1) {
    if (r < first_out || r >= nloc) return;
    double x0 = 0.0, x1 = 0.0;
    if (r - lrow0 < b) {
      x0 = myK[(size_t)(r - lrow0) * b + n];
      x1 = myK[(size_t)(r - lrow0) * b + n + 1];
    }
    T* dst = V + (size_t)(gr0 + r - row0) * ldv + n;
    dst[0] = (T)(x0 - a0);
    dst[1] = (T)(x1 - a1);
  });
  RRF_STAMP(38, id == 0);
}

}  // namespace rrf
