// The three dense contractions of one block step of Algorithm 2 as TMA-staged tensor-core
// kernels (f64: DMMA m16n8k8; f32: 3xTF32 on the same fragment layout).
//
//   sample_kernel   Y  = W[r0:, :] * Omega_i            (Algorithm 2 line 7, "Sample Panel")
//   vtw_kernel      Z  = V_i^T * W[r0:, :]              (line 8, first product of the WY update)
//   update_kernel   W[r0:, :] -= V_i * Zt^T  + norms    (line 8, second product; line 9's ||B_i||_F^2)
//
// Shared-memory tiles are written by TMA with the 128-byte swizzle.  Two operand forms occur:
//   K-contiguous  (a row of the tile is 128 bytes along the contraction index): each thread
//       fetches one 16-byte chunk per row, chunk (2t + s) ^ (row & 7), and feeds its elements to
//       k-slots (t, t+4) of consecutive m16n8k8 steps.  The contraction index may be permuted
//       freely as long as both operands use the same permutation, which they do.
//   MN-contiguous (a row of the tile is one contraction index, 128 bytes along M or N):
//       scalar loads at rows k = 8*ks + 2t (+1).
// Both access patterns are bank-conflict free under the swizzle.
#pragma once

#include "common.cuh"

namespace rrf {

template <typename T>
struct Elem {
  static constexpr int KE = 128 / (int)sizeof(T);       // elements per 128-byte line
  static constexpr int NV = 16 / (int)sizeof(T);        // elements per 16-byte chunk
  static constexpr int KS = NV / 2;                     // m16n8k8 steps fed by one chunk
};

__device__ __forceinline__ unsigned char* align1024(unsigned char* p) {
  return reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(p) + 1023) & ~uintptr_t(1023));
}

template <typename T>
__device__ __forceinline__ void store2(T* p, T a, T b);
template <>
__device__ __forceinline__ void store2<double>(double* p, double a, double b) {
  *reinterpret_cast<double2*>(p) = make_double2(a, b);
}
template <>
__device__ __forceinline__ void store2<float>(float* p, float a, float b) {
  *reinterpret_cast<float2*>(p) = make_float2(a, b);
}

// ------------------------------------------------------------------------------------------
// Y_part[seg] = W[r0 + slab*BM ..., k-range(seg)] * OmegaT[j0 .. j0+B, k-range(seg)]^T
// grid = (row slabs, K segments); both operands K-contiguous.
// ------------------------------------------------------------------------------------------
template <typename T, int B, int BM, int WM, int WN, int STAGES>
__global__ void __launch_bounds__(WM* WN * 32)
    sample_kernel(const __grid_constant__ CUtensorMap tmW,  // W [m][n], box [BM][KE]
                  const __grid_constant__ CUtensorMap tmO,  // OmegaT [max_rank][n], box [B][KE]
                  T* __restrict__ Ypart,                    // [nseg][rows][B]
                  int r0, int rows, int n, int j0, int kt_per_seg, Ctrl* ctrl) {
  if (*reinterpret_cast<volatile int*>(&ctrl->done)) return;
  constexpr int KE = Elem<T>::KE, NV = Elem<T>::NV, KS = Elem<T>::KS;
  constexpr int TM = BM / WM, TN = B / WN, MT = TM / 16, NT = TN / 8;
  static_assert(TM % 16 == 0 && TN % 8 == 0, "warp tile");
  constexpr int A_BYTES = BM * 128, B_BYTES = B * 128, STAGE_BYTES = A_BYTES + B_BYTES;

  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = align1024(smem_raw);
  __shared__ uint64_t full[STAGES];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int wm = warp / WN, wn = warp % WN;
  const int slab = blockIdx.x, seg = blockIdx.y;
  const int KT = (n + KE - 1) / KE;
  const int kt0 = seg * kt_per_seg;
  const int nkt = max(0, min(KT, kt0 + kt_per_seg) - kt0);
  const int grow0 = r0 + slab * BM;

  if (tid == 0) {
    for (int s = 0; s < STAGES; ++s) mbar_init(&full[s], 1);
    mbar_fence_init();
  }
  __syncthreads();

  auto issue = [&](int i) {
    const int st = i % STAGES;
    unsigned char* sA = smem + st * STAGE_BYTES;
    mbar_expect_tx(&full[st], STAGE_BYTES);
    tma_load_2d(sA, &tmW, (kt0 + i) * KE, grow0, &full[st]);
    tma_load_2d(sA + A_BYTES, &tmO, (kt0 + i) * KE, j0, &full[st]);
  };
  if (tid == 0)
    for (int i = 0; i < STAGES - 1 && i < nkt; ++i) issue(i);

  T acc[MT][NT][4];
#pragma unroll
  for (int a = 0; a < MT; ++a)
#pragma unroll
    for (int c = 0; c < NT; ++c)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[a][c][e] = T(0);

  for (int i = 0; i < nkt; ++i) {
    if (tid == 0 && i + STAGES - 1 < nkt) issue(i + STAGES - 1);
    const int st = i % STAGES;
    if (!mbar_wait(&full[st], (i / STAGES) & 1, ctrl)) return;
    const unsigned char* sA = smem + st * STAGE_BYTES;
    const unsigned char* sB = sA + A_BYTES;
#pragma unroll
    for (int s2 = 0; s2 < 2; ++s2) {
      const uint32_t chunk = ((uint32_t)(2 * t + s2) ^ (uint32_t)g) << 4;
      T ra[MT][2][NV], rb[NT][NV];
#pragma unroll
      for (int a = 0; a < MT; ++a) {
        const int rlo = wm * TM + a * 16 + g;
        VecLoad16<T>::ld(sA + rlo * 128 + chunk, ra[a][0]);
        VecLoad16<T>::ld(sA + (rlo + 8) * 128 + chunk, ra[a][1]);
      }
#pragma unroll
      for (int c = 0; c < NT; ++c) {
        const int rn = wn * TN + c * 8 + g;
        VecLoad16<T>::ld(sB + rn * 128 + chunk, rb[c]);
      }
#pragma unroll
      for (int ks = 0; ks < KS; ++ks)
#pragma unroll
        for (int a = 0; a < MT; ++a) {
          const T af[4] = {ra[a][0][2 * ks], ra[a][1][2 * ks], ra[a][0][2 * ks + 1], ra[a][1][2 * ks + 1]};
#pragma unroll
          for (int c = 0; c < NT; ++c) {
            const T bf[2] = {rb[c][2 * ks], rb[c][2 * ks + 1]};
            mma16x8x8(acc[a][c], af, bf);
          }
        }
    }
    __syncthreads();  // everyone is done with stage st before it is refilled
  }

  T* Y = Ypart + (size_t)seg * (size_t)rows * B;
#pragma unroll
  for (int a = 0; a < MT; ++a)
#pragma unroll
    for (int c = 0; c < NT; ++c) {
      const int row = slab * BM + wm * TM + a * 16 + g;
      const int col = wn * TN + c * 8 + 2 * t;
      if (row < rows) store2(Y + (size_t)row * B + col, acc[a][c][0], acc[a][c][1]);
      if (row + 8 < rows) store2(Y + (size_t)(row + 8) * B + col, acc[a][c][2], acc[a][c][3]);
    }
}

// ------------------------------------------------------------------------------------------
// Z_part[seg][0:B, col tile] = V[r0 + k-range(seg), cv0 .. cv0+B]^T * C[r0 + k-range(seg), col tile]
// grid = (column tiles, K segments); both operands MN-contiguous (K runs over matrix rows).
// ------------------------------------------------------------------------------------------
template <typename T, int B, int BN, int BK, int WM, int WN, int STAGES>
__global__ void __launch_bounds__(WM* WN * 32)
    vtw_kernel(const __grid_constant__ CUtensorMap tmV,  // V [m][ldv], box [BK][KE]
               const __grid_constant__ CUtensorMap tmC,  // C [m][ncols], box [BK][KE]
               T* __restrict__ Zpart,                    // [nseg][B][npad]
               int r0, int rows, int cv0, int npad, int kt_per_seg, Ctrl* ctrl) {
  if (*reinterpret_cast<volatile int*>(&ctrl->done)) return;
  constexpr int KE = Elem<T>::KE;
  constexpr int TM = B / WM, TN = BN / WN, MT = TM / 16, NT = TN / 8;
  static_assert(TM % 16 == 0 && TN % 8 == 0 && B % KE == 0 && BN % KE == 0 && BK % 8 == 0, "tile");
  constexpr int NBV = B / KE, NBC = BN / KE;
  constexpr int BOX_BYTES = BK * 128;
  constexpr int V_BYTES = NBV * BOX_BYTES, C_BYTES = NBC * BOX_BYTES, STAGE_BYTES = V_BYTES + C_BYTES;

  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = align1024(smem_raw);
  __shared__ uint64_t full[STAGES];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int wm = warp / WN, wn = warp % WN;
  const int col0 = blockIdx.x * BN, seg = blockIdx.y;
  const int KT = (rows + BK - 1) / BK;
  const int kt0 = seg * kt_per_seg;
  const int nkt = max(0, min(KT, kt0 + kt_per_seg) - kt0);

  if (tid == 0) {
    for (int s = 0; s < STAGES; ++s) mbar_init(&full[s], 1);
    mbar_fence_init();
  }
  __syncthreads();

  auto issue = [&](int i) {
    const int st = i % STAGES;
    unsigned char* sV = smem + st * STAGE_BYTES;
    const int y = r0 + (kt0 + i) * BK;
    mbar_expect_tx(&full[st], STAGE_BYTES);
#pragma unroll
    for (int v = 0; v < NBV; ++v) tma_load_2d(sV + v * BOX_BYTES, &tmV, cv0 + v * KE, y, &full[st]);
#pragma unroll
    for (int c = 0; c < NBC; ++c) tma_load_2d(sV + V_BYTES + c * BOX_BYTES, &tmC, col0 + c * KE, y, &full[st]);
  };
  if (tid == 0)
    for (int i = 0; i < STAGES - 1 && i < nkt; ++i) issue(i);

  T acc[MT][NT][4];
#pragma unroll
  for (int a = 0; a < MT; ++a)
#pragma unroll
    for (int c = 0; c < NT; ++c)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[a][c][e] = T(0);

  // The last K tile may reach past `rows` only when r0 + rows == m, where TMA zero-fills.
  for (int i = 0; i < nkt; ++i) {
    if (tid == 0 && i + STAGES - 1 < nkt) issue(i + STAGES - 1);
    const int st = i % STAGES;
    if (!mbar_wait(&full[st], (i / STAGES) & 1, ctrl)) return;
    const unsigned char* sV = smem + st * STAGE_BYTES;
    const unsigned char* sC = sV + V_BYTES;
#pragma unroll
    for (int ks = 0; ks < BK / 8; ++ks) {
      const uint32_t k = ks * 8 + 2 * t;
      T af[MT][4], bf[NT][2];
#pragma unroll
      for (int a = 0; a < MT; ++a) {
        const int j = wm * TM + a * 16 + g;
        const unsigned char* box_lo = sV + (j / KE) * BOX_BYTES;
        const unsigned char* box_hi = sV + ((j + 8) / KE) * BOX_BYTES;
        const uint32_t c_lo = (j % KE) * sizeof(T), c_hi = ((j + 8) % KE) * sizeof(T);
        af[a][0] = *reinterpret_cast<const T*>(box_lo + swz128(k * 128 + c_lo));
        af[a][1] = *reinterpret_cast<const T*>(box_hi + swz128(k * 128 + c_hi));
        af[a][2] = *reinterpret_cast<const T*>(box_lo + swz128((k + 1) * 128 + c_lo));
        af[a][3] = *reinterpret_cast<const T*>(box_hi + swz128((k + 1) * 128 + c_hi));
      }
#pragma unroll
      for (int c = 0; c < NT; ++c) {
        const int nn = wn * TN + c * 8 + g;
        const unsigned char* box = sC + (nn / KE) * BOX_BYTES;
        const uint32_t cc = (nn % KE) * sizeof(T);
        bf[c][0] = *reinterpret_cast<const T*>(box + swz128(k * 128 + cc));
        bf[c][1] = *reinterpret_cast<const T*>(box + swz128((k + 1) * 128 + cc));
      }
#pragma unroll
      for (int a = 0; a < MT; ++a)
#pragma unroll
        for (int c = 0; c < NT; ++c) mma16x8x8(acc[a][c], af[a], bf[c]);
    }
    __syncthreads();
  }

  T* Z = Zpart + (size_t)seg * (size_t)B * npad;
#pragma unroll
  for (int a = 0; a < MT; ++a)
#pragma unroll
    for (int c = 0; c < NT; ++c) {
      const int j = wm * TM + a * 16 + g;
      const int col = col0 + wn * TN + c * 8 + 2 * t;  // < npad by construction
      store2(Z + (size_t)j * npad + col, acc[a][c][0], acc[a][c][1]);
      store2(Z + (size_t)(j + 8) * npad + col, acc[a][c][2], acc[a][c][3]);
    }
}

// ------------------------------------------------------------------------------------------
// C[r0 + row tile, col tile] -= V[r0 + row tile, cv0 .. cv0+B] * Zt[col tile, 0:B]^T
// Rows r0 .. r0+top_rows-1 of the result go to `top` (the finished block row B_i), the rest
// back to C.  Also emits the two squared Frobenius norms of those row groups, per CTA.
// grid = (column tiles, row tiles); both operands K-contiguous, K = B in one shot.
// ------------------------------------------------------------------------------------------
template <typename T, int B, int BM, int BN, int WM, int WN>
__global__ void __launch_bounds__(WM* WN * 32)
    update_kernel(const __grid_constant__ CUtensorMap tmV,  // V [m][ldv], box [BM][KE]
                  const __grid_constant__ CUtensorMap tmZ,  // Zt [npad][B], box [BN][KE]
                  T* __restrict__ C, long long ldc, T* __restrict__ top, long long ldtop,
                  int r0, int rows, int ncols, int cv0, int top_rows,
                  double* __restrict__ norm_part, Ctrl* ctrl) {
  if (*reinterpret_cast<volatile int*>(&ctrl->done)) return;
  constexpr int KE = Elem<T>::KE, NV = Elem<T>::NV, KS = Elem<T>::KS;
  constexpr int TM = BM / WM, TN = BN / WN, MT = TM / 16, NT = TN / 8;
  constexpr int NKB = B / KE;  // 128-byte K boxes
  static_assert(B % KE == 0, "block size must fill whole 128-byte lines");
  constexpr int A_BOX = BM * 128, B_BOX = BN * 128;
  constexpr int TOTAL = NKB * (A_BOX + B_BOX);

  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = align1024(smem_raw);
  __shared__ uint64_t full;
  __shared__ double red[64];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int wm = warp / WN, wn = warp % WN;
  const int col0 = blockIdx.x * BN, lrow0 = blockIdx.y * BM;

  if (tid == 0) {
    mbar_init(&full, 1);
    mbar_fence_init();
  }
  __syncthreads();
  if (tid == 0) {
    mbar_expect_tx(&full, TOTAL);
#pragma unroll
    for (int kb = 0; kb < NKB; ++kb) {
      tma_load_2d(smem + kb * A_BOX, &tmV, cv0 + kb * KE, r0 + lrow0, &full);
      tma_load_2d(smem + NKB * A_BOX + kb * B_BOX, &tmZ, kb * KE, col0, &full);
    }
  }

  // C tile straight into the accumulator layout while the operands are in flight
  T cw[MT][NT][4];
#pragma unroll
  for (int a = 0; a < MT; ++a)
#pragma unroll
    for (int c = 0; c < NT; ++c) {
      const int lrow = lrow0 + wm * TM + a * 16 + g;
      const int col = col0 + wn * TN + c * 8 + 2 * t;
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int lr = lrow + 8 * h;
        T x0 = T(0), x1 = T(0);
        if (lr < rows) {
          const T* p = C + (size_t)(r0 + lr) * ldc + col;
          if (col < ncols) x0 = p[0];
          if (col + 1 < ncols) x1 = p[1];
        }
        cw[a][c][2 * h] = x0;
        cw[a][c][2 * h + 1] = x1;
      }
    }

  T acc[MT][NT][4];
#pragma unroll
  for (int a = 0; a < MT; ++a)
#pragma unroll
    for (int c = 0; c < NT; ++c)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[a][c][e] = T(0);

  if (!mbar_wait(&full, 0, ctrl)) return;

#pragma unroll
  for (int kb = 0; kb < NKB; ++kb) {
    const unsigned char* sA = smem + kb * A_BOX;
    const unsigned char* sB = smem + NKB * A_BOX + kb * B_BOX;
#pragma unroll
    for (int s2 = 0; s2 < 2; ++s2) {
      const uint32_t chunk = ((uint32_t)(2 * t + s2) ^ (uint32_t)g) << 4;
      T ra[MT][2][NV], rb[NT][NV];
#pragma unroll
      for (int a = 0; a < MT; ++a) {
        const int rlo = wm * TM + a * 16 + g;
        VecLoad16<T>::ld(sA + rlo * 128 + chunk, ra[a][0]);
        VecLoad16<T>::ld(sA + (rlo + 8) * 128 + chunk, ra[a][1]);
      }
#pragma unroll
      for (int c = 0; c < NT; ++c) {
        const int rn = wn * TN + c * 8 + g;
        VecLoad16<T>::ld(sB + rn * 128 + chunk, rb[c]);
      }
#pragma unroll
      for (int ks = 0; ks < KS; ++ks)
#pragma unroll
        for (int a = 0; a < MT; ++a) {
          const T af[4] = {ra[a][0][2 * ks], ra[a][1][2 * ks], ra[a][0][2 * ks + 1], ra[a][1][2 * ks + 1]};
#pragma unroll
          for (int c = 0; c < NT; ++c) {
            const T bf[2] = {rb[c][2 * ks], rb[c][2 * ks + 1]};
            mma16x8x8(acc[a][c], af, bf);
          }
        }
    }
  }

  double s_top = 0.0, s_trail = 0.0;
#pragma unroll
  for (int a = 0; a < MT; ++a)
#pragma unroll
    for (int c = 0; c < NT; ++c) {
      const int lrow = lrow0 + wm * TM + a * 16 + g;
      const int col = col0 + wn * TN + c * 8 + 2 * t;
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int lr = lrow + 8 * h;
        if (lr >= rows) continue;
        const T y0 = cw[a][c][2 * h] - acc[a][c][2 * h];
        const T y1 = cw[a][c][2 * h + 1] - acc[a][c][2 * h + 1];
        const bool is_top = lr < top_rows;
        T* p = is_top ? top + (size_t)lr * ldtop + col : C + (size_t)(r0 + lr) * ldc + col;
        double q = 0.0;
        if (col + 1 < ncols) {
          store2(p, y0, y1);
          q = (double)y0 * (double)y0 + (double)y1 * (double)y1;
        } else if (col < ncols) {
          p[0] = y0;
          q = (double)y0 * (double)y0;
        }
        if (is_top) s_top += q; else s_trail += q;
      }
    }
  const double bt = block_sum(s_top, red);
  const double br = block_sum(s_trail, red + 32);
  if (tid == 0 && norm_part != nullptr) {
    const size_t blk = (size_t)blockIdx.y * gridDim.x + blockIdx.x;
    norm_part[2 * blk] = bt;
    norm_part[2 * blk + 1] = br;
  }
}

}  // namespace rrf
