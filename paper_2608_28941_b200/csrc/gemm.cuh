// Dense contractions of Algorithm 2 as TMA-staged tensor-core kernels (f64: DMMA m16n8k8;
// f32: 3xTF32 on the same fragment layout).  This file holds the shared tile conventions and
//
//   sample_kernel   Y  = W[r0:, :] * Omega_i            (Algorithm 2 line 7, "Sample Panel")
//
// which runs once per call, for the first block; the persistent kernels of the block loop
// are in gemm_sk.cuh.
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
// Items (row slab, K segment), walked by one CTA per SM; both operands K-contiguous.
// ------------------------------------------------------------------------------------------
// KBS 128-byte K boxes of both operands form one pipeline stage.
template <typename T, int B, int BM, int WM, int WN, int STAGES, int KBS>
__global__ void __launch_bounds__(WM* WN * 32)
    sample_kernel(const __grid_constant__ CUtensorMap tmW,  // W [m][n], box [BM][KE]
                  const __grid_constant__ CUtensorMap tmO,  // OmegaT [max_rank][n], box [B][KE]
                  T* __restrict__ Ypart,                    // [nseg][rows][B]
                  int r0, int rows, int n, int j0, int nslabs, int nseg, int kt_per_seg, Ctrl* ctrl,
                  const int* __restrict__ only_if_zero,     // non-NULL: run only where the fused update skipped this panel
                  double* __restrict__ sq_part) {           // non-NULL: also per-CTA partial sums of squares of W
  if (*reinterpret_cast<volatile int*>(&ctrl->done)) return;
  if (only_if_zero != nullptr) {
    if (*only_if_zero != 0) return;
    if (blockIdx.x == 0 && threadIdx.x == 0) atomicAdd(&ctrl->extra_samples, 1);
  }
  constexpr int KE = Elem<T>::KE, NV = Elem<T>::NV, KS = Elem<T>::KS;
  constexpr int TM = BM / WM, TN = B / WN, MT = TM / 16, NT = TN / 8;
  static_assert(TM % 16 == 0 && TN % 8 == 0, "warp tile");
  constexpr int A_BYTES = BM * 128, B_BYTES = B * 128, STAGE_BYTES = KBS * (A_BYTES + B_BYTES);

  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = align1024(smem_raw);
  __shared__ uint64_t full[STAGES];
  __shared__ double red[32];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int wm = warp / WN, wn = warp % WN;
  const int KT = (n + KBS * KE - 1) / (KBS * KE);    // K tiles of KBS boxes
  // ||W||_F^2 on the side (Algorithm 2 line 2): the warps of warp column 0 between them load every element
  // of a W tile exactly once, and the items of the launch partition W
  const bool take_sq = sq_part != nullptr && wn == 0;
  double sq = 0.0;

  if (tid == 0) {
    for (int s = 0; s < STAGES; ++s) mbar_init(&full[s], 1);
    mbar_fence_init();
  }
  __syncthreads();

  // One CTA per SM walks the (row slab, K segment) items; `base` counts the K tiles this CTA has been
  // through, which is what the stage ring and the barrier phases follow across items.
  int base = 0;
  for (int item = blockIdx.x; item < nslabs * nseg; item += gridDim.x) {
    const int slab = item % nslabs, seg = item / nslabs;
    const int kt0 = seg * kt_per_seg;
    const int nkt = max(0, min(KT, kt0 + kt_per_seg) - kt0);
    const int grow0 = r0 + slab * BM;

    auto issue = [&](int i) {
      const int st = (base + i) % STAGES;
      unsigned char* sA = smem + st * STAGE_BYTES;
      mbar_expect_tx(&full[st], STAGE_BYTES);
#pragma unroll
      for (int kb = 0; kb < KBS; ++kb) {
        tma_load_2d(sA + kb * A_BYTES, &tmW, ((kt0 + i) * KBS + kb) * KE, grow0, &full[st]);
        tma_load_2d(sA + KBS * A_BYTES + kb * B_BYTES, &tmO, ((kt0 + i) * KBS + kb) * KE, j0, &full[st]);
      }
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
      const int st = (base + i) % STAGES;
      if (!mbar_wait(&full[st], ((base + i) / STAGES) & 1, ctrl)) return;
#pragma unroll
      for (int kb = 0; kb < KBS; ++kb) {
        const unsigned char* sA = smem + st * STAGE_BYTES + kb * A_BYTES;
        const unsigned char* sB = smem + st * STAGE_BYTES + KBS * A_BYTES + kb * B_BYTES;
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
          if (take_sq) {
#pragma unroll
            for (int a = 0; a < MT; ++a)
#pragma unroll
              for (int h = 0; h < 2; ++h)
#pragma unroll
                for (int e = 0; e < NV; ++e) sq += (double)ra[a][h][e] * (double)ra[a][h][e];
          }
#pragma unroll
          for (int c = 0; c < NT; ++c) {
            const int rn = wn * TN + c * 8 + g;
            VecLoad16<T>::ld(sB + rn * 128 + chunk, rb[c]);
          }
          Op<T> oa[MT][2][NV], ob[NT][NV];     // split once, used by NT (resp. MT) products each
#pragma unroll
          for (int a = 0; a < MT; ++a)
#pragma unroll
            for (int e = 0; e < NV; ++e) {
              oa[a][0][e] = prep(ra[a][0][e]);
              oa[a][1][e] = prep(ra[a][1][e]);
            }
#pragma unroll
          for (int c = 0; c < NT; ++c)
#pragma unroll
            for (int e = 0; e < NV; ++e) ob[c][e] = prep(rb[c][e]);
#pragma unroll
          for (int ks = 0; ks < KS; ++ks)
#pragma unroll
            for (int a = 0; a < MT; ++a)
#pragma unroll
              for (int c = 0; c < NT; ++c)
                mma_op(acc[a][c], oa[a][0][2 * ks], oa[a][1][2 * ks], oa[a][0][2 * ks + 1], oa[a][1][2 * ks + 1],
                       ob[c][2 * ks], ob[c][2 * ks + 1]);
        }
      }
      __syncthreads();  // everyone is done with stage st before it is refilled
    }
    base += nkt;

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
  if (sq_part != nullptr) {
    const double tot = block_sum(sq, red);     // fixed order within the CTA; the CTA's items in their order
    if (tid == 0) sq_part[blockIdx.x] = tot;
  }
}

}  // namespace rrf
