// Persistent ("stream-K") versions of the two large contractions of a block step.
//
// Both kernels run one CTA per SM they are given (every SM under the sequential schedule; all but the
// SMs of the panel kernel under the look-ahead schedule, where they run beside it).  The tiles of the problem are numbered along the
// direction in which an accumulator can stay in registers, and CTA p owns the contiguous
// range [p*tpc, (p+1)*tpc) of them, so every SM gets the same amount of work whatever the
// trailing matrix's height.  When a CTA's range crosses from one accumulator to the next it
// writes a partial result to slot (p + index of the accumulator): consecutive (CTA,
// accumulator) pairs differ in p, in the index, or in both, so the slot is unique, and the
// consumer of the partials (panel loader, Z reduction) sums the slots of one accumulator in
// CTA order - a fixed order, so results are reproducible bit for bit.
//
// TMA loads are issued by one extra warp (vtw) or by one lane of the first warp (upd); the consumer
// warps never wait for each other (full/empty mbarriers per stage, every wait bounded).
//
//   vtw_sk_kernel   Z = V_i^T W[r0:, :]                      (Algorithm 2 line 8, first product)
//   upd_sk_kernel   W[r0:, :] -= V_i Zt^T, norms of line 9, and - fused, from the updated tile
//                   still in registers - a later panel Y = W_new Omega_j (line 7 of a later pass:
//                   j = i+1 under the sequential schedule, j = i+2 under look-ahead), which saves
//                   one full read of W per block step.
#pragma once

#include "gemm.cuh"

namespace rrf {

__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

template <typename T, int MT, int NT>
__device__ __forceinline__ void flush_tile(T (&acc)[MT][NT][4], T* __restrict__ dst, int ld, int row0, int col0,
                                           int g, int t) {
#pragma unroll
  for (int a = 0; a < MT; ++a)
#pragma unroll
    for (int cc = 0; cc < NT; ++cc) {
      const int r = row0 + a * 16 + g;
      const int col = col0 + cc * 8 + 2 * t;
      store2(dst + (size_t)r * ld + col, acc[a][cc][0], acc[a][cc][1]);
      store2(dst + (size_t)(r + 8) * ld + col, acc[a][cc][2], acc[a][cc][3]);
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[a][cc][e] = T(0);
    }
}

// ------------------------------------------------------------------------------------------
// Z partials.  Tiles: L = c*KT + kt (column tile c of BN columns, K chunk kt of BK rows).
// Slot (p + c) of Zpart holds a B x BN partial of column tile c.
// ------------------------------------------------------------------------------------------
template <typename T, int B, int BN, int BK, int WM, int WN, int STAGES>
__global__ void __launch_bounds__((WM * WN + 1) * 32)
    vtw_sk_kernel(const __grid_constant__ CUtensorMap tmV,  // V [m][ldv], box [BK][KE]
                  const __grid_constant__ CUtensorMap tmC,  // C [m][ncols], box [BK][KE]
                  T* __restrict__ Zpart, int r0, int cv0, int KT, int total, int tpc, Ctrl* ctrl) {
  if (*reinterpret_cast<volatile int*>(&ctrl->done)) return;
  constexpr int KE = Elem<T>::KE;
  constexpr int NCW = WM * WN;
  constexpr int TM = B / WM, TN = BN / WN, MT = TM / 16, NT = TN / 8;
  static_assert(TM % 16 == 0 && TN % 8 == 0 && B % KE == 0 && BN % KE == 0 && BK % 8 == 0, "tile");
  constexpr int NBV = B / KE, NBC = BN / KE;
  constexpr int BOX_BYTES = BK * 128;
  constexpr int V_BYTES = NBV * BOX_BYTES, C_BYTES = NBC * BOX_BYTES, STAGE_BYTES = V_BYTES + C_BYTES;

  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = align1024(smem_raw);
  __shared__ uint64_t full[STAGES], empty[STAGES];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int p = blockIdx.x;
  const int L0 = p * tpc;
  const int ntile = min(total, L0 + tpc) - L0;

  if (tid == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&empty[s], NCW);
    }
    mbar_fence_init();
  }
  __syncthreads();

  if (warp == NCW) {
    if (lane == 0) {
      for (int i = 0; i < ntile; ++i) {
        const int st = i % STAGES;
        if (i >= STAGES && !mbar_wait(&empty[st], ((i / STAGES) - 1) & 1, ctrl)) return;
        const int L = L0 + i, c = L / KT, kt = L - c * KT;
        unsigned char* sV = smem + st * STAGE_BYTES;
        const int y = r0 + kt * BK;
        mbar_expect_tx(&full[st], STAGE_BYTES);
#pragma unroll
        for (int v = 0; v < NBV; ++v) tma_load_2d(sV + v * BOX_BYTES, &tmV, cv0 + v * KE, y, &full[st]);
#pragma unroll
        for (int cb = 0; cb < NBC; ++cb)
          tma_load_2d(sV + V_BYTES + cb * BOX_BYTES, &tmC, c * BN + cb * KE, y, &full[st]);
      }
    }
    return;
  }

  const int wm = warp / WN, wn = warp % WN;
  T acc[MT][NT][4];
#pragma unroll
  for (int a = 0; a < MT; ++a)
#pragma unroll
    for (int c = 0; c < NT; ++c)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[a][c][e] = T(0);

  // per-thread byte offsets of the fragment elements inside a stage (rows 2t and 2t+1 of each box)
  uint32_t offA[MT][4], offB[NT][2];
  {
    const uint32_t x0 = ((uint32_t)(2 * t) & 7u) << 4, x1 = ((uint32_t)(2 * t + 1) & 7u) << 4;
    const uint32_t r0b = (uint32_t)(2 * t) * 128u, r1b = r0b + 128u;
#pragma unroll
    for (int a = 0; a < MT; ++a) {
      const int j = wm * TM + a * 16 + g;
      const uint32_t b_lo = (uint32_t)(j / KE) * BOX_BYTES, b_hi = (uint32_t)((j + 8) / KE) * BOX_BYTES;
      const uint32_t c_lo = (uint32_t)(j % KE) * sizeof(T), c_hi = (uint32_t)((j + 8) % KE) * sizeof(T);
      offA[a][0] = b_lo + r0b + (c_lo ^ x0);
      offA[a][1] = b_hi + r0b + (c_hi ^ x0);
      offA[a][2] = b_lo + r1b + (c_lo ^ x1);
      offA[a][3] = b_hi + r1b + (c_hi ^ x1);
    }
#pragma unroll
    for (int cc = 0; cc < NT; ++cc) {
      const int nn = wn * TN + cc * 8 + g;
      const uint32_t bb = (uint32_t)(nn / KE) * BOX_BYTES, co = (uint32_t)(nn % KE) * sizeof(T);
      offB[cc][0] = bb + r0b + (co ^ x0);
      offB[cc][1] = bb + r1b + (co ^ x1);
    }
  }
  int cur_c = L0 / KT;
  int c = cur_c, kt = L0 - cur_c * KT, st = 0;
  uint32_t ph = 0;
  for (int i = 0; i < ntile; ++i) {
    if (c != cur_c) {
      flush_tile<T, MT, NT>(acc, Zpart + (size_t)(p + cur_c) * (size_t)(B * BN), BN, wm * TM, wn * TN, g, t);
      cur_c = c;
    }
    if (!mbar_wait(&full[st], ph, ctrl)) return;
    const unsigned char* sV = smem + st * STAGE_BYTES;
    const unsigned char* sC = sV + V_BYTES;
    // Rows k = 8*ks + 2t and k + 1 of a box: the swizzle XORs the 16-byte chunk index with k & 7,
    // which is 2t or 2t + 1 whatever ks is, so every fragment address is a per-thread constant
    // plus ks * 1024 bytes.
#pragma unroll
    for (int ks = 0; ks < BK / 8; ++ks) {
      Op<T> af[MT][4], bf[NT][2];
#pragma unroll
      for (int a = 0; a < MT; ++a) {
        af[a][0] = prep(*reinterpret_cast<const T*>(sV + offA[a][0] + ks * 1024));
        af[a][1] = prep(*reinterpret_cast<const T*>(sV + offA[a][1] + ks * 1024));
        af[a][2] = prep(*reinterpret_cast<const T*>(sV + offA[a][2] + ks * 1024));
        af[a][3] = prep(*reinterpret_cast<const T*>(sV + offA[a][3] + ks * 1024));
      }
#pragma unroll
      for (int cc = 0; cc < NT; ++cc) {
        bf[cc][0] = prep(*reinterpret_cast<const T*>(sC + offB[cc][0] + ks * 1024));
        bf[cc][1] = prep(*reinterpret_cast<const T*>(sC + offB[cc][1] + ks * 1024));
      }
#pragma unroll
      for (int a = 0; a < MT; ++a)
#pragma unroll
        for (int cc = 0; cc < NT; ++cc)
          mma_op(acc[a][cc], af[a][0], af[a][1], af[a][2], af[a][3], bf[cc][0], bf[cc][1]);
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&empty[st]);
    if (++st == STAGES) { st = 0; ph ^= 1u; }
    if (++kt == KT) { kt = 0; ++c; }
  }
  if (ntile > 0)
    flush_tile<T, MT, NT>(acc, Zpart + (size_t)(p + cur_c) * (size_t)(B * BN), BN, wm * TM, wn * TN, g, t);
}

// ------------------------------------------------------------------------------------------
// Fused update + next sample.  Tiles: L = s*NC + c (row slab s of BM rows, column tile c of BN
// columns); a CTA keeps V[slab] in shared memory and the slab's Y accumulator in registers.
//   P     = V[slab, :] * Zt[col tile, :]^T                 (K = B)
//   Wnew  = W[slab, col tile] - P   -> global (block row B_i to `top`, the rest back to C)
//   Y    += Wnew * OmegaT[j0 .. j0+B, col tile]^T          (K = BN; only if j0 >= 0)
// The accumulator fragment of Wnew is used directly as the A operand of the second product:
// within one 128-byte group of columns, thread t of a quad holds the KE/4 consecutive columns
// (KE/4)*t ..., i.e. n-tile u of the group covers columns (KE/4)*t + 2u + {0, 1}, which are
// exactly k-slots (t, t+4) of one m16n8k8 step whose B operand is read from OmegaT with the
// same chunk rule as every other K-contiguous operand.  No shuffles, no shared-memory round trip.
// Slot ((p + s)*WN + wn) of Ypart holds the BM x B partial of slab s from CTA p, warp column wn.
// ------------------------------------------------------------------------------------------
// PW: a dedicated producer warp issues the TMA loads.  Without it (PW = false) lane 0 of consumer
// warp 0 issues them at the top of each tile, which leaves the CTA at eight warps - two per SM
// sub-partition, hence up to 255 registers per thread for the widest block size.
template <typename T, int B, int BM, int BNB, int WM, int WN, int STAGES, bool PW>
__global__ void __launch_bounds__((WM * WN + (PW ? 1 : 0)) * 32, 1)
    upd_sk_kernel(const __grid_constant__ CUtensorMap tmV,  // V [m][ldv], box [BM][KE]
                  const __grid_constant__ CUtensorMap tmZ,  // Zt [npad][B], box [BN][KE]
                  const __grid_constant__ CUtensorMap tmC,  // C [m][ncols], box [BM][KE]
                  const __grid_constant__ CUtensorMap tmO,  // OmegaT [max_rank][n], box [B][KE]
                  T* __restrict__ C, long long ldc, T* __restrict__ top, long long ldtop,
                  int r0, int rows, int ncols, int cv0, int top_rows, int j0,
                  T* __restrict__ Ypart, double* __restrict__ norm_part,
                  int NC, int total, int tpc, Ctrl* ctrl,
                  const int* __restrict__ samp_flag,     // non-NULL: sample only if *samp_flag != 0
                  int p0, int Lb) {                      // this launch is CTAs p0 ... of the pass and starts at tile Lb
  if (*reinterpret_cast<volatile int*>(&ctrl->done)) return;
  constexpr int KE = Elem<T>::KE, NV = Elem<T>::NV, KS = Elem<T>::KS;
  constexpr int U = KE / 8;            // n-tiles per 128-byte column group
  constexpr int NCW = WM * WN;
  constexpr int BN = BNB * KE;
  constexpr int KB = B / KE;           // 128-byte K boxes of V and Zt
  constexpr int TM = BM / WM, MT = TM / 16;
  constexpr int QW = BNB / WN;         // column groups per warp
  constexpr int NTB = B / 8;           // n-tiles of the Y accumulator
  static_assert(TM % 16 == 0 && BNB % WN == 0 && B % KE == 0, "tile");
  constexpr int V_BOX = BM * 128, W_BOX = BM * 128, Z_BOX = BN * 128, O_BOX = B * 128;
  constexpr int V_BYTES = KB * V_BOX;
  constexpr int W_BYTES = BNB * W_BOX, Z_BYTES = KB * Z_BOX, O_BYTES = BNB * O_BOX;
  constexpr int STAGE_BYTES = W_BYTES + Z_BYTES + O_BYTES;

  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = align1024(smem_raw);
  unsigned char* sVs = smem;
  unsigned char* sStage = smem + V_BYTES;
  __shared__ uint64_t full[STAGES], empty[STAGES], v_full, v_empty;
  __shared__ double red[64];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  // A pass may be split over two launches (the second one, on the SMs a finished panel kernel has left, takes the
  // tiles from Lb on): CTA numbers, which name the partial-result slots, run on from the first launch's.
  // (the widest block is never split: its instantiation has no register to spare)
  const int p = (B >= 128 ? 0 : p0) + blockIdx.x;
  const int L0 = (B >= 128 ? 0 : Lb) + blockIdx.x * tpc;
  const int ntile = B >= 128 ? min(total, L0 + tpc) - L0 : max(0, min(total, L0 + tpc) - L0);
  // the widest block size and single precision keep the host's decision (those instantiations are at
  // the register limit and lose 3-4 % with the extra test)
  constexpr bool kPredicted = B < 128 && sizeof(T) == 8;
  const bool do_sample = j0 >= 0 && (!kPredicted || samp_flag == nullptr || *samp_flag != 0);
  if (kPredicted && do_sample && samp_flag != nullptr && p == 0 && tid == 0) atomicAdd(&ctrl->fused_samples, 1);

  if (tid == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&empty[s], NCW);
    }
    mbar_init(&v_full, 1);
    mbar_init(&v_empty, NCW);
    mbar_fence_init();
  }
  __syncthreads();

  double s_top = 0.0, s_trail = 0.0;

  // loads of one tile (and of V when the tile opens a new row slab); called by one thread
  auto load_slab = [&](int s) {
    mbar_expect_tx(&v_full, V_BYTES);
#pragma unroll
    for (int kb = 0; kb < KB; ++kb) tma_load_2d(sVs + kb * V_BOX, &tmV, cv0 + kb * KE, r0 + s * BM, &v_full);
  };
  auto load_tile = [&](int i, int s, int c) {
    const int st = i % STAGES;
    unsigned char* sW = sStage + st * STAGE_BYTES;
    mbar_expect_tx(&full[st], do_sample ? STAGE_BYTES : W_BYTES + Z_BYTES);
#pragma unroll
    for (int q = 0; q < BNB; ++q) tma_load_2d(sW + q * W_BOX, &tmC, c * BN + q * KE, r0 + s * BM, &full[st]);
#pragma unroll
    for (int kb = 0; kb < KB; ++kb) tma_load_2d(sW + W_BYTES + kb * Z_BOX, &tmZ, kb * KE, c * BN, &full[st]);
    if (do_sample) {
#pragma unroll
      for (int q = 0; q < BNB; ++q)
        tma_load_2d(sW + W_BYTES + Z_BYTES + q * O_BOX, &tmO, c * BN + q * KE, j0, &full[st]);
    }
  };

  if (PW && warp == NCW) {
    // ------------------------------------------------------------ producer warp
    if (lane == 0) {
      int cur_s = -1, nslab = 0;
      int s = L0 / NC, c = L0 - s * NC;
      for (int i = 0; i < ntile; ++i, c = (c + 1 == NC ? 0 : c + 1), s += (c == 0)) {
        if (s != cur_s) {
          if (nslab > 0 && !mbar_wait(&v_empty, (nslab - 1) & 1, ctrl)) break;
          load_slab(s);
          cur_s = s;
          ++nslab;
        }
        if (i >= STAGES && !mbar_wait(&empty[i % STAGES], ((i / STAGES) - 1) & 1, ctrl)) break;
        load_tile(i, s, c);
      }
    }
  } else {
    // ------------------------------------------------------------ consumer warps
    const int wm = warp / WN, wn = warp % WN;
    T accY[MT][NTB][4];
#pragma unroll
    for (int a = 0; a < MT; ++a)
#pragma unroll
      for (int nb = 0; nb < NTB; ++nb)
#pragma unroll
        for (int e = 0; e < 4; ++e) accY[a][nb][e] = T(0);

    int cur_s = -1, nslab = 0;
    bool ok = true;
    int s = L0 / NC, c = L0 - s * NC, st = 0;
    uint32_t ph = 0;
    // state of the inline producer (PW = false; used by lane 0 of warp 0 only)
    int nxt = 0, p_s = s, p_c = c, p_cur_s = -1, p_nslab = 0;
    // per slab: where this thread's rows go, and to which norm they count (hoisted out of the tile loop)
    T* rowp[MT][2];
    bool rtop[MT][2];
    for (int i = 0; i < ntile && ok; ++i) {
      if (s != cur_s && cur_s >= 0) {
        if (do_sample)
          flush_tile<T, MT, NTB>(accY, Ypart + ((size_t)(p + cur_s) * WN + wn) * (size_t)(BM * B), B, wm * TM, 0, g, t);
        __syncwarp();
        if (lane == 0) mbar_arrive(&v_empty);
      }
      if (!PW) {
        if (warp == 0 && lane == 0) {
          // issue every tile up to STAGES-1 ahead; a tile that opens a new slab waits until the
          // consumers stand at it (the V buffer is single)
          while (nxt < ntile && nxt <= i + STAGES - 1) {
            if (p_s != p_cur_s) {
              if (nxt != i) break;
              if (p_nslab > 0 && !mbar_wait(&v_empty, (p_nslab - 1) & 1, ctrl)) break;
              load_slab(p_s);
              p_cur_s = p_s;
              ++p_nslab;
            }
            if (nxt >= STAGES && !mbar_wait(&empty[nxt % STAGES], ((nxt / STAGES) - 1) & 1, ctrl)) break;
            load_tile(nxt, p_s, p_c);
            ++nxt;
            if (++p_c == NC) { p_c = 0; ++p_s; }
          }
        }
        __syncwarp();
      }
      if (s != cur_s) {
        if (!mbar_wait(&v_full, nslab & 1, ctrl)) { ok = false; break; }
        cur_s = s;
        ++nslab;
#pragma unroll
        for (int a = 0; a < MT; ++a)
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            const int lr = s * BM + wm * TM + a * 16 + g + 8 * h;     // row relative to r0
            rtop[a][h] = lr < top_rows;
            rowp[a][h] = lr >= rows ? nullptr : (rtop[a][h] ? top + (size_t)lr * ldtop : C + (size_t)(r0 + lr) * ldc);
          }
      }
      if (!mbar_wait(&full[st], ph, ctrl)) { ok = false; break; }
      const unsigned char* sW = sStage + st * STAGE_BYTES;
      const unsigned char* sZ = sW + W_BYTES;
      const unsigned char* sO = sZ + Z_BYTES;

      if constexpr (sizeof(T) == 8) {
        // ---- P = V * Zt^T for this warp's rows and column groups
        T acc[MT][QW][U][4];
#pragma unroll
        for (int a = 0; a < MT; ++a)
#pragma unroll
          for (int q = 0; q < QW; ++q)
#pragma unroll
            for (int u = 0; u < U; ++u)
#pragma unroll
              for (int e = 0; e < 4; ++e) acc[a][q][u][e] = T(0);
#pragma unroll
        for (int kb = 0; kb < KB; ++kb) {
#pragma unroll
          for (int s2 = 0; s2 < 2; ++s2) {
            T ra[MT][2][NV];
#pragma unroll
            for (int a = 0; a < MT; ++a) {
              const int rlo = wm * TM + a * 16 + g;
              const uint32_t chunk = ((uint32_t)(2 * t + s2) ^ (uint32_t)g) << 4;
              VecLoad16<T>::ld(sVs + kb * V_BOX + rlo * 128 + chunk, ra[a][0]);
              VecLoad16<T>::ld(sVs + kb * V_BOX + (rlo + 8) * 128 + chunk, ra[a][1]);
            }
#pragma unroll
            for (int q = 0; q < QW; ++q)
#pragma unroll
              for (int u = 0; u < U; ++u) {
                // n-slot g of tile u is column (KE/4)*(g/2) + 2u + (g&1) of the group
                const int zr = (wn * QW + q) * KE + (KE / 4) * (g >> 1) + 2 * u + (g & 1);
                T rb[NV];
                VecLoad16<T>::ld(sZ + kb * Z_BOX + zr * 128 + (((uint32_t)(2 * t + s2) ^ (uint32_t)(zr & 7)) << 4), rb);
#pragma unroll
                for (int ks = 0; ks < KS; ++ks) {
                  const T bf[2] = {rb[2 * ks], rb[2 * ks + 1]};
#pragma unroll
                  for (int a = 0; a < MT; ++a) {
                    const T af[4] = {ra[a][0][2 * ks], ra[a][1][2 * ks], ra[a][0][2 * ks + 1], ra[a][1][2 * ks + 1]};
                    mma16x8x8(acc[a][q][u], af, bf);
                  }
                }
              }
          }
        }

        // ---- Wnew = W - P: store, norms, and keep as the A operand of the sample product
        const int col_base = c * BN;
        const bool interior = col_base + BN <= ncols;      // no column guards needed
#pragma unroll
        for (int a = 0; a < MT; ++a)
#pragma unroll
          for (int q = 0; q < QW; ++q) {
            const int grp = wn * QW + q;
            const int col = col_base + grp * KE + (KE / 4) * t;   // first of this thread's KE/4 consecutive columns
#pragma unroll
            for (int h = 0; h < 2; ++h) {
              const int rl = wm * TM + a * 16 + g + 8 * h;     // row inside the slab
              T wv[2][NV];
#pragma unroll
              for (int s2 = 0; s2 < 2; ++s2)
                VecLoad16<T>::ld(sW + grp * W_BOX + rl * 128 + (((uint32_t)(2 * t + s2) ^ (uint32_t)g) << 4), wv[s2]);
              T* dst = rowp[a][h];
              double q0 = 0.0, q1 = 0.0;
#pragma unroll
              for (int s2 = 0; s2 < 2; ++s2)
#pragma unroll
                for (int ks = 0; ks < KS; ++ks) {
                  const int u = s2 * KS + ks;
                  const T y0 = wv[s2][2 * ks] - acc[a][q][u][2 * h];
                  const T y1 = wv[s2][2 * ks + 1] - acc[a][q][u][2 * h + 1];
                  acc[a][q][u][2 * h] = y0;
                  acc[a][q][u][2 * h + 1] = y1;
                  const int cc = col + 2 * u;
                  if (dst != nullptr) {
                    if (interior || cc + 1 < ncols) {
                      store2(dst + cc, y0, y1);
                      q0 += (double)y0 * (double)y0;
                      q1 += (double)y1 * (double)y1;
                    } else if (cc < ncols) {
                      dst[cc] = y0;
                      q0 += (double)y0 * (double)y0;
                    }
                  }
                }
              const double qs = q0 + q1;
              s_top += rtop[a][h] ? qs : 0.0;
              s_trail += rtop[a][h] ? 0.0 : qs;
            }
          }

        // ---- Y += Wnew * OmegaT^T (K = this warp's columns)
        if (do_sample) {
#pragma unroll
          for (int q = 0; q < QW; ++q) {
            const int grp = wn * QW + q;
#pragma unroll
            for (int s2 = 0; s2 < 2; ++s2) {
#pragma unroll
              for (int nb = 0; nb < NTB; ++nb) {
                const int jr = nb * 8 + g;
                T rb[NV];
                VecLoad16<T>::ld(sO + grp * O_BOX + jr * 128 + (((uint32_t)(2 * t + s2) ^ (uint32_t)g) << 4), rb);
#pragma unroll
                for (int ks = 0; ks < KS; ++ks) {
                  const int u = s2 * KS + ks;
                  const T bf[2] = {rb[2 * ks], rb[2 * ks + 1]};
#pragma unroll
                  for (int a = 0; a < MT; ++a) {
                    const T af[4] = {acc[a][q][u][0], acc[a][q][u][2], acc[a][q][u][1], acc[a][q][u][3]};
                    mma16x8x8(accY[a][nb], af, bf);
                  }
                }
              }
            }
          }
        }
      } else {
        // The tile runs as a pipeline over this warp's QW column groups so that the tensor pipe always
        // has a product to work on while the element-wise part of another group is in flight:
        //   VZ(0) | VZ(1) + EPI(0) | S(0) + EPI(1) | S(1)          (QW = 2)
        // Single precision only (three TF32 products and their splitting per MMA leave issue slots for
        // this to pay: 11 % on the 4096 x 11008 workload); in double precision the plain order above is
        // faster by 4 %.
        // VZ(q): P = V * Zt^T for group q.  EPI(q): Wnew = W - P, store, norms (2 MT pieces, one per 8
        // rows).  S(q): Y += Wnew * OmegaT^T with the accumulator fragment of Wnew as the A operand.
        // The pieces of EPI are placed between the unrolled MMA iterations of the neighbouring product.
        T acc[MT][QW][U][4];
        const int col_base = c * BN;
        const bool interior = col_base + BN <= ncols;      // no column guards needed
        constexpr int NP = 2 * MT;                          // pieces of one group's epilogue
#define RRF_VZ_ITER(qa_, qb_, it_)                                                                                   \
        {                                                                                                         \
          const int kb_ = (it_) >> 1, s2_ = (it_) & 1;                                                            \
          Op<T> oa_[MT][2][NV];                                                                                   \
          _Pragma("unroll") for (int a = 0; a < MT; ++a) {                                                        \
            const int rlo = wm * TM + a * 16 + g;                                                                 \
            const uint32_t chunk = ((uint32_t)(2 * t + s2_) ^ (uint32_t)g) << 4;                                  \
            T ra0_[NV], ra1_[NV];                                                                                 \
            VecLoad16<T>::ld(sVs + kb_ * V_BOX + rlo * 128 + chunk, ra0_);                                        \
            VecLoad16<T>::ld(sVs + kb_ * V_BOX + (rlo + 8) * 128 + chunk, ra1_);                                  \
            _Pragma("unroll") for (int e = 0; e < NV; ++e) {                                                      \
              oa_[a][0][e] = prep(ra0_[e]);                                                                       \
              oa_[a][1][e] = prep(ra1_[e]);                                                                       \
            }                                                                                                     \
          }                                                                                                       \
          _Pragma("unroll") for (int q_ = (qa_); q_ < (qb_); ++q_)                                                \
          _Pragma("unroll") for (int u = 0; u < U; ++u) {                                                         \
            /* n-slot g of tile u is column (KE/4)*(g/2) + 2u + (g&1) of the group */                             \
            const int zr = (wn * QW + (q_)) * KE + (KE / 4) * (g >> 1) + 2 * u + (g & 1);                         \
            T rb_[NV];                                                                                            \
            VecLoad16<T>::ld(sZ + kb_ * Z_BOX + zr * 128 + (((uint32_t)(2 * t + s2_) ^ (uint32_t)(zr & 7)) << 4), rb_); \
            _Pragma("unroll") for (int ks = 0; ks < KS; ++ks) {                                                   \
              const Op<T> b0_ = prep(rb_[2 * ks]), b1_ = prep(rb_[2 * ks + 1]);                                   \
              _Pragma("unroll") for (int a = 0; a < MT; ++a)                                                      \
                mma_op(acc[a][q_][u], oa_[a][0][2 * ks], oa_[a][1][2 * ks], oa_[a][0][2 * ks + 1],                \
                       oa_[a][1][2 * ks + 1], b0_, b1_);                                                          \
            }                                                                                                     \
          }                                                                                                       \
        }
#define RRF_EPI_PIECE(q_, e_)                                                                                  \
        {                                                                                                         \
          const int a_ = (e_) >> 1, h_ = (e_) & 1;                                                                \
          const int grp = wn * QW + (q_);                                                                         \
          const int col = col_base + grp * KE + (KE / 4) * t;   /* first of this thread's KE/4 consecutive columns */ \
          const int rl = wm * TM + a_ * 16 + g + 8 * h_;        /* row inside the slab */                         \
          T wv[2][NV];                                                                                            \
          _Pragma("unroll") for (int s2 = 0; s2 < 2; ++s2)                                                        \
            VecLoad16<T>::ld(sW + grp * W_BOX + rl * 128 + (((uint32_t)(2 * t + s2) ^ (uint32_t)g) << 4), wv[s2]); \
          T* dst = rowp[a_][h_];                                                                                  \
          double q0 = 0.0, q1 = 0.0;                                                                              \
          _Pragma("unroll") for (int s2 = 0; s2 < 2; ++s2)                                                        \
            _Pragma("unroll") for (int ks = 0; ks < KS; ++ks) {                                                   \
              const int u = s2 * KS + ks;                                                                         \
              const T y0 = wv[s2][2 * ks] - acc[a_][q_][u][2 * h_];                                               \
              const T y1 = wv[s2][2 * ks + 1] - acc[a_][q_][u][2 * h_ + 1];                                       \
              acc[a_][q_][u][2 * h_] = y0;                                                                        \
              acc[a_][q_][u][2 * h_ + 1] = y1;                                                                    \
              const int cc = col + 2 * u;                                                                         \
              if (dst != nullptr) {                                                                               \
                if (interior || cc + 1 < ncols) {                                                                 \
                  store2(dst + cc, y0, y1);                                                                       \
                  q0 += (double)y0 * (double)y0;                                                                  \
                  q1 += (double)y1 * (double)y1;                                                                  \
                } else if (cc < ncols) {                                                                          \
                  dst[cc] = y0;                                                                                   \
                  q0 += (double)y0 * (double)y0;                                                                  \
                }                                                                                                 \
              }                                                                                                   \
            }                                                                                                     \
          const double qs = q0 + q1;                                                                              \
          s_top += rtop[a_][h_] ? qs : 0.0;                                                                       \
          s_trail += rtop[a_][h_] ? 0.0 : qs;                                                                     \
        }
#define RRF_S_ITER(q_, it_)                                                                                    \
        {                                                                                                         \
          const int s2_ = (it_) / NTB, nb_ = (it_) % NTB;                                                         \
          const int grp = wn * QW + (q_);                                                                         \
          const int jr = nb_ * 8 + g;                                                                             \
          T rb_[NV];                                                                                              \
          VecLoad16<T>::ld(sO + grp * O_BOX + jr * 128 + (((uint32_t)(2 * t + s2_) ^ (uint32_t)g) << 4), rb_);    \
          _Pragma("unroll") for (int ks = 0; ks < KS; ++ks) {                                                     \
            const int u = s2_ * KS + ks;                                                                          \
            const Op<T> b0_ = prep(rb_[2 * ks]), b1_ = prep(rb_[2 * ks + 1]);                                     \
            _Pragma("unroll") for (int a = 0; a < MT; ++a)                                                        \
              mma_op(accY[a][nb_], oW[a][u][0], oW[a][u][2], oW[a][u][1], oW[a][u][3], b0_, b1_);                 \
          }                                                                                                       \
        }
        /* the updated tile of group q_ as the A operand of the sample product, split once for all its n-tiles */ \
#define RRF_SPLIT_W(q_)                                                                                           \
        _Pragma("unroll") for (int a = 0; a < MT; ++a)                                                            \
          _Pragma("unroll") for (int u = 0; u < U; ++u)                                                           \
            _Pragma("unroll") for (int e = 0; e < 4; ++e) oW[a][u][e] = prep(acc[a][q_][u][e]);
        Op<T> oW[MT][U][4];
#pragma unroll
        for (int a = 0; a < MT; ++a)
#pragma unroll
          for (int q = 0; q < QW; ++q)
#pragma unroll
            for (int u = 0; u < U; ++u)
#pragma unroll
              for (int e = 0; e < 4; ++e) acc[a][q][u][e] = T(0);
        constexpr int NVZ = 2 * KB, NSI = 2 * NTB;          // unrolled iterations of VZ and of S(q)
        static_assert(QW == 1 || QW == 2, "column groups per warp");
          constexpr bool kSplitVZ = true;
        if (QW == 2 && kSplitVZ) {
#pragma unroll
          for (int it = 0; it < NVZ; ++it) RRF_VZ_ITER(0, 1, it)
#pragma unroll
          for (int it = 0; it < NVZ; ++it) {
            RRF_VZ_ITER(QW - 1, QW, it)
#pragma unroll
            for (int e = 0; e < NP; ++e)
              if (it == (((e + 1) * NVZ) / (NP + 1) > 0 ? ((e + 1) * NVZ) / (NP + 1) - 1 : 0)) RRF_EPI_PIECE(0, e)
          }
        } else {
#pragma unroll
          for (int it = 0; it < NVZ; ++it) RRF_VZ_ITER(0, QW, it)
#pragma unroll
          for (int e = 0; e < NP; ++e) RRF_EPI_PIECE(0, e)
        }
        if (QW == 2 && !do_sample) {
#pragma unroll
          for (int e = 0; e < NP; ++e) RRF_EPI_PIECE(QW - 1, e)
        }
        if (do_sample) {
          RRF_SPLIT_W(0)
#pragma unroll
          for (int it = 0; it < NSI; ++it) {
            RRF_S_ITER(0, it)
            if (QW == 2) {
#pragma unroll
              for (int e = 0; e < NP; ++e)
                if (it == ((e + 1) * NSI) / (NP + 1) - 1) RRF_EPI_PIECE(QW - 1, e)
            }
          }
          if (QW == 2) {
            RRF_SPLIT_W(QW - 1)
#pragma unroll
            for (int it = 0; it < NSI; ++it) RRF_S_ITER(QW - 1, it)
          }
        }
#undef RRF_SPLIT_W
#undef RRF_VZ_ITER
#undef RRF_EPI_PIECE
#undef RRF_S_ITER
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty[st]);
      if (++st == STAGES) { st = 0; ph ^= 1u; }
      if (++c == NC) { c = 0; ++s; }
    }
    if (ok && cur_s >= 0 && do_sample)
      flush_tile<T, MT, NTB>(accY, Ypart + ((size_t)(p + cur_s) * WN + wn) * (size_t)(BM * B), B, wm * TM, 0, g, t);
  }

  // per-CTA norm partials (all warps join; the producer contributes zeros)
  const double bt = block_sum(s_top, red);
  const double br = block_sum(s_trail, red + 32);
  if (tid == 0 && norm_part != nullptr) {
    norm_part[2 * p] = bt;
    norm_part[2 * p + 1] = br;
  }
}

}  // namespace rrf
