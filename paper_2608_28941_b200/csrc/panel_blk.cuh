// Panel Householder QR (Algorithm 2 line 7, geqrt semantics), blocked: the panel's columns are factored in
// micro-panels of eight.
//
// The plain column-by-column kernel (panel.cuh) reads and writes the whole trailing slab for every column
// (a BLAS-2 pass bound by shared-memory bandwidth) and pays a grid barrier plus an all-to-all read of b partial
// sums per column.  Here a column step touches only the eight columns of its micro-panel:
//   column j of micro-panel [j0, j0+8):  finish column j with the pending reflector, one pass over the slab's
//   eight columns (applies the pending reflector and takes the dot products of column j with all eight), one
//   exchange of eight partial sums per CTA, the reflector's scalars, scaling of column j.
// After its eighth column the micro-panel is applied to the rest of the panel as a block reflector on the FP64
// tensor cores:  D = X^T V8 (every column against the eight new vectors; for finished columns these are the
// entries of V^T V that the T factor needs), one two-stage exchange, C = T8^T D, X -= V8 C.
//
// Exchanges replace the grid barrier: every CTA writes its values as flagged words (see ll_store: the value and
// the tag of the round in the same 64-bit words) into its own slots of a global buffer; every CTA reads all slots,
// spinning until the round's tag is there, and sums them in CTA order, so all CTAs hold the same bits.  A slot is
// reused two rounds later, which is safe because a CTA can only write round r+2 after it has read every CTA's
// round r+1, i.e. after every CTA has finished reading round r.  All CTAs must be co-resident (cooperative
// launch); every wait is bounded.  The slab can live in shared memory or, for panels that do not fit there, in a
// stretch of global memory private to the CTA.
#pragma once

#include "panel_tsqr.cuh"

namespace rrf {

constexpr int kMB = 8;                       // columns of a micro-panel

struct BlkScratch {
  unsigned long long* Lw;  // [2][16][Gp][2]: per-column exchange, flagged words (see ll_store); Gp = G rounded up to 32
  unsigned long long* Pw;  // [8 b][Gp][2]: per-CTA partial D of a block step, flagged words, CTA index innermost
  unsigned long long* Rw;  // [16 b][2]: C = T8^T D and D summed over the CTAs, flagged words
  double* Cg;              // [G][8 b]: a CTA's own copy of C when shared memory has no room for it
};
constexpr int kBlkDw = 2048;                 // doubles of the D partials of the K-split warps (overlaid on the fix-up staging)

// Flagged words: a double travels as two 64-bit words, each carrying 32 bits of the value and the 32-bit tag of
// the round.  An aligned 64-bit word is written and read as one piece, so a reader that finds the round's tag in
// both words has the value: one trip through L2 instead of a flag wait followed by a data read, no fences.
__device__ __forceinline__ void ll_store(unsigned long long* p, double v, unsigned tag) {
  const unsigned long long bits = (unsigned long long)__double_as_longlong(v);
  const unsigned long long w0 = (bits & 0xffffffffull) | ((unsigned long long)tag << 32);
  const unsigned long long w1 = (bits >> 32) | ((unsigned long long)tag << 32);
  asm volatile("st.relaxed.gpu.global.v2.u64 [%0], {%1, %2};" ::"l"(p), "l"(w0), "l"(w1) : "memory");
}
__device__ __forceinline__ bool ll_try(const unsigned long long* p, unsigned tag, double* out) {
  unsigned long long w0, w1;
  asm volatile("ld.relaxed.gpu.global.v2.u64 {%0, %1}, [%2];" : "=l"(w0), "=l"(w1) : "l"(p) : "memory");
  if ((unsigned)(w0 >> 32) != tag || (unsigned)(w1 >> 32) != tag) return false;
  *out = __longlong_as_double((long long)((w0 & 0xffffffffull) | (w1 << 32)));
  return true;
}
// Sum of value `row` of this round over all CTAs: lane x takes CTAs x, x + 32, ... (all its reads in flight
// together), then the fixed shuffle tree.  Returns false if a tag never came.
constexpr int kBlkMaxRounds = kPanelMaxG / 32;
__device__ __forceinline__ bool ll_sum(const unsigned long long* rowp, int G, unsigned tag, int lane, Ctrl* ctrl, double* sum) {
  double v[kBlkMaxRounds];
  bool have[kBlkMaxRounds];
#pragma unroll
  for (int q = 0; q < kBlkMaxRounds; ++q) {
    v[q] = 0.0;
    have[q] = lane + 32 * q >= G;
  }
  bool ok = true;
  const long long t0 = clock64();
  while (true) {
    bool all = true;
#pragma unroll
    for (int q = 0; q < kBlkMaxRounds; ++q) {
      if (!have[q]) have[q] = ll_try(rowp + 2 * (size_t)(lane + 32 * q), tag, &v[q]);
      all = all && have[q];
    }
    if (all) break;
    __nanosleep(40);                         // leave the SM's memory pipeline to the stores the others wait for
    if (clock64() - t0 > kWaitLimitClocks) {
      atomicExch(&ctrl->status, (int)RRF_ERR_TIMEOUT);
      atomicExch(&ctrl->done, 1);
      ok = false;
      break;
    }
  }
  double a = 0.0;
#pragma unroll
  for (int q = 0; q < kBlkMaxRounds; ++q) a += v[q];
  *sum = warp_sum(a);
  return ok;
}

// ------------------------------------------------------------------------------------------
// The kernel.  Slab rows are numbered from the first row the kernel touches (with the look-ahead fix-up: b rows
// above the panel).  R rows per CTA, RS >= R rows allocated (a multiple of 16, zero filled), pitch Rp.
// `ksplit`: warps that share the rows of one tile in the D product (1: no shared-memory staging of D);
// `c_in_smem`: C of the block step is staged in shared memory (else read from global memory, for slabs that
// leave no room).  `gslab`: the slabs themselves live in global memory (any height, any number of CTAs).
// ------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(kPanelThreads)
    panel_blk_kernel(const T* __restrict__ Y, PanelSource src_fused, PanelSource src_alt, const int* __restrict__ fused_flag,
                     int rows, int b, int R, int Rp, int RS, T* __restrict__ V, long long ldv,
                     double* __restrict__ gram, double* __restrict__ tau_out, BlkScratch bs, unsigned seq_base,
                     int ksplit, int c_in_smem, unsigned* bar, Ctrl* ctrl, const int* done_flag, PanelFix fix,
                     unsigned bar_base, T* __restrict__ Tout, long long ldt, double* __restrict__ csq,
                     double* __restrict__ gslab) {      // non-NULL: the slabs live in global memory ([CTA][b][Rp])
  if (*reinterpret_cast<const volatile int*>(done_flag) || *reinterpret_cast<const volatile int*>(&ctrl->status) < 0) return;
  const bool use_alt = fused_flag != nullptr && *fused_flag == 0;
  const PanelSource src = use_alt ? src_alt : src_fused;
  extern __shared__ double psm[];
  __shared__ int ok_s;
  constexpr int NT = kPanelThreads, NW = NT / 32;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;
  const int G = gridDim.x, cta = blockIdx.x;
  const int Gp = (G + 31) & ~31;
  const int row0 = fix.enabled ? b : 0;
  const int ext = rows + row0;
  const int gr0 = cta * R;
  const int nloc = max(0, min(R, ext - gr0));
  const int lb = 31 - __clz(b);
  const int aux_n = max(fix.enabled ? panel_fix_doubles(b) : 0, ksplit > 1 ? kBlkDw : 0);
  const int cp = b + 8;
  // The slab [b][Rp]: in shared memory, or - for slabs taller than shared memory holds, or to confine a tall
  // panel to a few SMs - in this CTA's own stretch of global memory (served by L1 / L2; nobody else touches it).
  double* S = gslab != nullptr ? gslab + (size_t)blockIdx.x * b * Rp : psm;
  double* aux = gslab != nullptr ? psm : psm + (size_t)b * Rp;   // fix-up staging, then the D partials of the K-split warps
  double* Cs = aux + aux_n;                         // [8][b + 8] (c_in_smem)
  double* p_s = Cs + (c_in_smem ? kMB * cp : 0);    // [2][8]
  double* pr_s = p_s + 16;                          // [8] pivot row of the micro-panel's columns
  double* tot_s = pr_s + 8;                         // [8] grid-wide sums
  double* w8_s = tot_s + 8;                         // [8] v^T y_c of the pending reflector
  double* Gm = w8_s + 8;                            // [8][8] v_l^T v_i of the micro-panel (l < i)
  double* T8 = Gm + 64;                             // [8][8]
  double* tauq = T8 + 64;                           // [8]
  double* sc_s = tauq + 8;                          // [8]
  unsigned nbar = 0;
  auto gb = [&]() { return grid_barrier(bar, bar_base + (++nbar) * (unsigned)G, ctrl); };

  for (int idx = tid; idx < nloc * b; idx += NT) {
    const int r = idx >> lb, c = idx & (b - 1);
    S[(size_t)c * Rp + r] = panel_entry(Y, src, gr0 + r - row0, c, b);
  }
  {
    const int npad = RS - nloc;
    for (int idx = tid; idx < npad * b; idx += NT) {
      const int c = idx / npad, r = nloc + (idx - c * npad);
      S[(size_t)c * Rp + r] = 0.0;
    }
  }
  if (tid == 0) ok_s = 1;
  __syncthreads();
  if (fix.enabled && !panel_fixup<T>(S, Rp, nloc, gr0, b, G, cta, true, fix, aux, gb)) return;
  if (csq != nullptr) {
    for (int c = warp; c < b; c += NW) {
      double a = 0.0;
      for (int r = lane; r < nloc; r += 32) {
        const double v = (gr0 + r >= row0) ? S[(size_t)c * Rp + r] : 0.0;
        a += v * v;
      }
      a = warp_sum(a);
      if (lane == 0) csq[(size_t)c * Gp + cta] = a;
    }
  }

  for (int j0 = 0; j0 < b; j0 += kMB) {
    double tau_prev = 0.0;
    // ---------------------------------------------------------------- the eight columns of the micro-panel
    for (int jj = 0; jj < kMB; ++jj) {
      const int j = j0 + jj, pr = row0 + j, par = j & 1;
      const unsigned want = seq_base + 1u + (unsigned)j;
      double* Sj = S + (size_t)j * Rp;
      const double* Sjm1 = S + (size_t)(jj > 0 ? j - 1 : j) * Rp;
      const bool pending = jj > 0 && tau_prev != 0.0;      // column j itself was finished with the scaling of v_{j-1}
      {
        // one warp per (column of the micro-panel, half of the rows): pending reflector, then y_j^T x_c
        const int cc = warp & 7, h = warp >> 3;
        const int half = ((RS >> 1) + 15) & ~15, rbeg = h * half, rend = min(RS, rbeg + half);
        double* Sc = S + (size_t)(j0 + cc) * Rp;
        const bool upd = pending && cc > jj;
        const double f = upd ? tau_prev * w8_s[cc] : 0.0;
        double a = 0.0;
        for (int r = rbeg + lane; r < rend; r += 32) {
          const int grow = gr0 + r;
          const double y = grow > pr ? Sj[r] : 0.0;
          double x = Sc[r];
          if (upd) {
            x -= f * (grow >= pr ? Sjm1[r] : 0.0);
            Sc[r] = x;
          }
          a += y * x;
        }
        a = warp_sum(a);
        if (lane == 0) p_s[h * 8 + cc] = a;
      }
      __syncthreads();
      // exchange: warp 0 publishes this CTA's line, warps 1..8 sum one value each over all CTAs, warp 9 fetches
      // the pivot row from the CTA that owns it
      // Each gathering warp first publishes this CTA's share of its value, then reads everybody's: a store issued
      // ahead of the warp's own polling loads is not held up behind them in the SM's memory pipeline.
      if (warp >= 1 && warp <= 8) {
        const int i = warp - 1;
        if (lane == 0) ll_store(bs.Lw + (((size_t)par * 16 + i) * Gp + cta) * 2, p_s[i] + p_s[8 + i], want);
        double a;
        const bool ok = ll_sum(bs.Lw + ((size_t)par * 16 + i) * Gp * 2, G, want, lane, ctrl, &a);
        if (lane == 0) tot_s[i] = a;
        if (!ok) ok_s = 0;
      } else if (warp == 9) {
        const int ow = pr / R, lr = pr - gr0;
        if (lane < 8) {
          if (ow == cta) ll_store(bs.Lw + (((size_t)par * 16 + 8 + lane) * Gp + cta) * 2, S[(size_t)(j0 + lane) * Rp + lr], want);
          const unsigned long long* p = bs.Lw + (((size_t)par * 16 + 8 + lane) * Gp + ow) * 2;
          double v = 0.0;
          const long long t0 = clock64();
          while (!ll_try(p, want, &v)) {
            if (clock64() - t0 > kWaitLimitClocks) {
              atomicExch(&ctrl->status, (int)RRF_ERR_TIMEOUT);
              atomicExch(&ctrl->done, 1);
              ok_s = 0;
              break;
            }
          }
          pr_s[lane] = v;
        }
      }
      __syncthreads();
      if (!ok_s) return;
      if (tid < kMB) {
        const double alpha = pr_s[jj], s2 = tot_s[jj];
        double tau = 0.0, rdenom = 0.0;
        if (s2 != 0.0) {
          const double beta = -copysign(sqrt(alpha * alpha + s2), alpha);
          tau = (beta - alpha) / beta;
          rdenom = 1.0 / (alpha - beta);
        }
        const double wv = pr_s[tid] + tot_s[tid] * rdenom;
        if (tid == jj) {
          sc_s[0] = tau;
          sc_s[1] = rdenom;
          tauq[jj] = tau;
          if (cta == 0) tau_out[j] = tau;
        } else if (tid > jj) {
          w8_s[tid] = wv;
        } else {
          Gm[jj * 8 + tid] = wv;
          if (cta == 0) gram[(size_t)j * b + j0 + tid] = wv;
        }
      }
      __syncthreads();
      // column j becomes v_j (unit lower trapezoidal, explicit ones and zeros); the same sweep finishes column
      // j + 1 with the new reflector (each thread touches only its own rows of both columns)
      const double tau = sc_s[0], rdenom = sc_s[1];
      const bool fin = jj + 1 < kMB && tau != 0.0;
      const double fnx = fin ? tau * w8_s[jj + 1] : 0.0;
      double* Sn = S + (size_t)(fin ? j + 1 : j) * Rp;
      for (int r = tid; r < RS; r += NT) {
        const int grow = gr0 + r;
        const double vj = grow > pr ? Sj[r] * rdenom : (grow == pr ? 1.0 : 0.0);
        Sj[r] = vj;
        if (fin && grow > pr) Sn[r] -= fnx * vj;
      }
      tau_prev = tau;
      __syncthreads();
    }
    if (b == kMB) break;
    // ---------------------------------------------------------------- block step
    const int P = j0 / kMB;
    const unsigned wantb = seq_base + 1u + (unsigned)P;
    // T8 of the micro-panel: T8[0:i, i] = -tau_i T8[0:i, 0:i] (V8[:, 0:i]^T v_i); thread r owns row r (in registers)
    if (tid < kMB) {
      const int r = tid;
      double trow[kMB];
#pragma unroll
      for (int i = 0; i < kMB; ++i) {
        double tv = 0.0;
        if (i == r) {
          tv = tauq[i];
        } else if (i > r) {
          double s = 0.0;
#pragma unroll
          for (int l = 0; l < kMB; ++l)
            if (l >= r && l < i) s += trow[l] * Gm[i * 8 + l];
          tv = -tauq[i] * s;
        }
        trow[i] = tv;
        T8[r * 8 + i] = tv;
      }
    }
    // D = X^T V8 for this CTA's rows (every column of the panel against the eight new vectors), m16n8k8:
    // A = X^T (16 columns x 8 rows), B = V8 (8 rows x 8 vectors).  Warp = (tile of 16 columns, share of the rows).
    {
      const int mt = b >> 4, nks = RS >> 3, per = (nks + ksplit - 1) / ksplit;
      const int mi = warp % mt, sp = warp / mt;
      if (sp < ksplit) {
        double acc[4] = {0.0, 0.0, 0.0, 0.0};
        const int ke = min(nks, (sp + 1) * per);
        for (int ks = sp * per; ks < ke; ++ks) {
          const double* pa = S + (size_t)(mi * 16 + g) * Rp + ks * 8 + t;
          const double af[4] = {pa[0], pa[8 * (size_t)Rp], pa[4], pa[8 * (size_t)Rp + 4]};
          const double* pb = S + (size_t)(j0 + g) * Rp + ks * 8 + t;
          const double bf[2] = {pb[0], pb[4]};
          mma16x8x8(acc, af, bf);
        }
        // c0: (column mi*16 + g, vector 2t), c1: vector 2t+1, c2/c3: column + 8
        const int e0 = (mi * 16 + g) * 8 + 2 * t;         // entry (column, vector) = column * 8 + vector
        if (ksplit > 1) {
          double* dw = aux + (size_t)sp * (b * 8) + e0;
          dw[0] = acc[0];
          dw[1] = acc[1];
          dw[64] = acc[2];
          dw[65] = acc[3];
        } else {
          unsigned long long* pw = bs.Pw + ((size_t)e0 * Gp + cta) * 2;
          ll_store(pw, acc[0], wantb);
          ll_store(pw + (size_t)Gp * 2, acc[1], wantb);
          ll_store(pw + (size_t)64 * Gp * 2, acc[2], wantb);
          ll_store(pw + (size_t)65 * Gp * 2, acc[3], wantb);
        }
      }
    }
    __syncthreads();
    if (ksplit > 1) {                                   // every (tile, share) warp has written its slice, zeros included
      for (int e = tid; e < b * 8; e += NT) {
        double s = 0.0;
        for (int sp = 0; sp < ksplit; ++sp) s += aux[(size_t)sp * (b * 8) + e];
        ll_store(bs.Pw + ((size_t)e * Gp + cta) * 2, s, wantb);
      }
    }
    // stage 2: CTA x sums the partials of its columns over all CTAs (fixed order), applies T8^T and publishes
    // C[:, c] = T8^T D[:, c] and D[:, c]
    {
      const int ncs = (b + G - 1) / G;                 // columns per reducing CTA
      const int c_lo = cta * ncs, c_hi = min(b, c_lo + ncs);
      double* dsum = sc_s;                             // [8]
      for (int c = c_lo; c < c_hi; ++c) {
        if (warp < kMB) {
          double a;
          const bool ok = ll_sum(bs.Pw + (size_t)(c * 8 + warp) * Gp * 2, G, wantb, lane, ctrl, &a);
          if (lane == 0) dsum[warp] = a;
          if (!ok) ok_s = 0;
        }
        __syncthreads();
        if (tid < kMB) {
          double cv = 0.0;
          for (int l = 0; l <= tid; ++l) cv += T8[l * 8 + tid] * dsum[l];
          ll_store(bs.Rw + ((size_t)tid * b + c) * 2, cv, wantb);
          ll_store(bs.Rw + ((size_t)(kMB + tid) * b + c) * 2, dsum[tid], wantb);
        }
        __syncthreads();
      }
      // stage 3: every CTA takes C (and CTA 0 the entries of V^T V against finished columns)
      const int nwant = kMB * b + (cta == 0 ? kMB * b : 0);
      double* Cg = bs.Cg + (size_t)cta * kMB * b;
      for (int e = tid; e < nwant; e += NT) {
        double v = 0.0;
        const unsigned long long* p = bs.Rw + (size_t)e * 2;
        const long long t0 = clock64();
        while (!ll_try(p, wantb, &v)) {
          if (clock64() - t0 > kWaitLimitClocks) {
            atomicExch(&ctrl->status, (int)RRF_ERR_TIMEOUT);
            atomicExch(&ctrl->done, 1);
            ok_s = 0;
            break;
          }
        }
        if (e < kMB * b) {
          if (c_in_smem) Cs[(e >> lb) * cp + (e & (b - 1))] = v;
          else Cg[e] = v;
        } else {
          const int i = (e - kMB * b) >> lb, c = e & (b - 1);
          if (c < j0) gram[(size_t)(j0 + i) * b + c] = v;
        }
      }
    }
    __syncthreads();
    if (!ok_s) return;
    // X[:, c] -= V8 C[:, c] for the columns behind the micro-panel: A = V8 (16 rows x 8), B = C (8 x 8 columns)
    {
      const double* Cgc = bs.Cg + (size_t)cta * kMB * b;
      const int ntc = (b - j0 - kMB) >> 3, nrt = RS >> 4;
      for (int task = warp; task < nrt * ntc; task += NW) {
        const int rt = task / ntc, ct = task - rt * ntc;
        const int r0 = rt * 16, c0 = j0 + kMB + ct * 8;
        const double* pa = S + (size_t)(j0 + t) * Rp + r0 + g;
        const double af[4] = {pa[0], pa[8], pa[4 * (size_t)Rp], pa[4 * (size_t)Rp + 8]};
        double bf[2];
        if (c_in_smem) {
          bf[0] = Cs[t * cp + c0 + g];
          bf[1] = Cs[(t + 4) * cp + c0 + g];
        } else {                                          // written by this CTA before the barrier above
          bf[0] = __ldcg(Cgc + (size_t)t * b + c0 + g);
          bf[1] = __ldcg(Cgc + (size_t)(t + 4) * b + c0 + g);
        }
        double acc[4] = {0.0, 0.0, 0.0, 0.0};
        mma16x8x8(acc, af, bf);
        double* px = S + (size_t)(c0 + 2 * t) * Rp + r0 + g;
        px[0] -= acc[0];
        px[Rp] -= acc[1];
        px[8] -= acc[2];
        px[Rp + 8] -= acc[3];
      }
    }
    __syncthreads();
  }

  for (int idx = tid; idx < nloc * b; idx += NT) {
    const int r = idx >> lb, c = idx & (b - 1);
    if (gr0 + r >= row0) V[(size_t)(gr0 + r - row0) * ldv + c] = (T)S[(size_t)c * Rp + r];
  }
  if (Tout != nullptr && cta == 0) {
    __syncthreads();
    tfactor_block<T>(gram, tau_out, b, Tout, ldt, psm);
  }
}

}  // namespace rrf
