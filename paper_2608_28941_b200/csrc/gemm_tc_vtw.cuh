// Single-precision Z = V_i^T W[r0:, :] (Algorithm 2 line 8, first product) on the fifth-generation tensor
// cores: tcgen05.mma kind::tf32, accumulator and LEFT operand in tensor memory.
//
// Same tiling, same stream-K ranges and the same partial-result slots as vtw_sk_kernel, so the consumer of the
// partials does not know which of the two ran.  The instruction computes D[128 x N] (+)= A[128 x 8] B[8 x N] with
// A = (W tile)^T and B = V tile; a K step is two instructions, A_hi [V_hi | V_lo] (N = 2B) and A_lo V_hi (N = B).
//   * Both tiles arrive by TMA with a 128-byte line holding one contraction index (a row of the matrices) and 32
//     consecutive columns.  For V that is the instruction's transposed ("MN-major") shared-memory operand, which for
//     32-bit data needs the swizzle with 32-byte atoms; its hi and lo planes are written by the split warps to a
//     second ring at the same offsets within a box, V_lo right behind V_hi so that one descriptor covers both.
//   * The 128 x 32 tile of W never goes back to shared memory: each of the eight split warps reads its part of it
//     transposed (lane = column of W, sixteen rows per thread; a warp reads whole 128-byte lines, so any swizzle is
//     conflict free), splits it and stores the planes with tcgen05.st as the left operand (lane = row of D, one
//     tensor-memory column per contraction index).  With W as a shared-memory operand the kernel ran at the
//     bandwidth of shared memory (152 KB of traffic per 24 KB stage; 88 KB this way) and was 7 % slower.
//   * `chunk` bounds how many 64-row tiles are summed inside tensor memory before the split warps add the
//     accumulator into registers with round-to-nearest adds (0: a whole accumulator stays in tensor memory).
//
// Warp roles: 0-7 split operands and drain the accumulator (warp w owns tensor-memory lanes 32 (w % 4) ..., i.e.
// those columns of the tile, rows 16 (w / 4) ... of a stage, and half w / 4 of the B rows of Z), 8 issues TMA
// loads, 9 issues the MMAs.  Tensor-memory columns: [D: 2B | A stage 0: hi 32, lo 32 | A stage 1 ...].
#pragma once

#include "gemm_tc_upd.cuh"

namespace rrf {

// right operand in shared memory with the contraction index as rows (32-byte-atom swizzle), left operand in tensor memory
__host__ __device__ constexpr uint32_t tc_idesc_tf32_ts_mn(int M, int N) {
  return (1u << 4) | (2u << 7) | (2u << 10) | (1u << 16) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
__device__ __forceinline__ float lds32(uint32_t a) {
  float v;
  asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(a));
  return v;
}

template <int B, int RS, int OS>
struct TcCfg {
  static constexpr int NBV = B / 32, NBC = kTcBN / 32;
  static constexpr int BOX = kTcSub * 128;
  static constexpr int RAW = (NBV + NBC) * BOX;       // one stage of the TMA ring: V boxes, then W boxes
  static constexpr int OPS = 2 * NBV * BOX;           // one stage of the plane ring: V_hi boxes, V_lo boxes
  static constexpr int SMEM = RS * RAW + OS * OPS + 1024;
  static constexpr int TA = 2 * B;                    // first tensor-memory column of the A stages (64 columns each)
  static constexpr int COLS = (TA + OS * 64 <= 256) ? 256 : 512;
  static_assert(TA + OS * 64 <= 512, "tensor memory");
};

template <int B, int RS, int OS>
__global__ void __launch_bounds__(kTcThreads, 1)
    vtw_tc_kernel(const __grid_constant__ CUtensorMap tmV,  // V [m][ldv], box [32][32], 32-byte-atom swizzle
                   const __grid_constant__ CUtensorMap tmC,  // C [m][ncols], box [32][32], 32-byte-atom swizzle
                   float* __restrict__ Zpart, int r0, int cv0, int KT, int total, int tpc, int chunk, Ctrl* ctrl) {
  if (*reinterpret_cast<volatile int*>(&ctrl->done)) return;
  using Cfg = TcCfg<B, RS, OS>;
  constexpr int NBV = Cfg::NBV, NBC = Cfg::NBC, BOX = Cfg::BOX, RAW = Cfg::RAW, OPS = Cfg::OPS, TA = Cfg::TA;
  static_assert(B == 32 || B == 64 || B == 128, "block sizes");
  static_assert(BOX / 16 == kTcConv * 32, "one 16-byte chunk of a box per split thread");

  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = align1024(smem_raw);
  unsigned char* ops = smem + RS * RAW;
  __shared__ uint64_t raw_full[RS], raw_empty[RS], op_full[OS], op_empty[OS], acc_full, acc_empty;
  __shared__ uint32_t tmem_slot;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int p = blockIdx.x;
  const int L0 = p * tpc;
  const int ntile = min(total, L0 + tpc) - L0;
  const int nsub = 2 * ntile;

  if (tid == 0) {
    for (int s = 0; s < RS; ++s) {
      mbar_init(&raw_full[s], 1);
      mbar_init(&raw_empty[s], kTcConv);
    }
    for (int s = 0; s < OS; ++s) {
      mbar_init(&op_full[s], kTcConv);
      mbar_init(&op_empty[s], 1);
    }
    mbar_init(&acc_full, 1);
    mbar_init(&acc_empty, kTcConv);
    mbar_fence_init();
  }
  __syncthreads();
  if (warp == 0) tmem_alloc(&tmem_slot, Cfg::COLS);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(&tmem_slot);

  auto drain_after = [&](int i, bool* last_of_acc) {
    const int L = L0 + i, c = L / KT, kt = L - c * KT;
    *last_of_acc = (i == ntile - 1) || (kt == KT - 1);
    return *last_of_acc || (chunk > 0 && (kt + 1) % chunk == 0);
  };

  if (warp == kTcConv) {
    // ---------------------------------------------------------------- TMA producer
    if (lane == 0) {
      for (int q = 0; q < nsub; ++q) {
        const int s = q % RS;
        if (q >= RS && !mbar_wait(&raw_empty[s], ((q / RS) - 1) & 1, ctrl)) break;
        const int L = L0 + (q >> 1), c = L / KT, kt = L - c * KT;
        const int y = r0 + kt * 64 + (q & 1) * kTcSub;
        unsigned char* dst = smem + s * RAW;
        mbar_expect_tx(&raw_full[s], RAW);
#pragma unroll
        for (int v = 0; v < NBV; ++v) tma_load_2d(dst + v * BOX, &tmV, cv0 + v * 32, y, &raw_full[s]);
#pragma unroll
        for (int cb = 0; cb < NBC; ++cb)
          tma_load_2d(dst + (NBV + cb) * BOX, &tmC, c * kTcBN + cb * 32, y, &raw_full[s]);
      }
    }
  } else if (warp == kTcConv + 1) {
    // ---------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc2 = tc_idesc_tf32_ts_mn(kTcBN, 2 * B), idesc1 = tc_idesc_tf32_ts_mn(kTcBN, B);
      uint32_t fresh = 1;
      int ndrain = 0;
      for (int q = 0; q < nsub; ++q) {
        const int o = q % OS;
        if (!mbar_wait(&op_full[o], (q / OS) & 1, ctrl)) break;
        if (fresh && ndrain > 0 && !mbar_wait(&acc_empty, (ndrain - 1) & 1, ctrl)) break;
        tc_fence_after();
        const uint32_t vH = smem_u32(ops + o * OPS);
        const uint32_t aH = tmem + TA + o * 64, aL = aH + 32;
#pragma unroll
        for (int ks = 0; ks < kTcSub / 8; ++ks) {
          const uint64_t vd = tc_desc(vH + ks * 1024, BOX);        // [V_hi | V_lo], or its first half
          tc_mma_tf32_ts(tmem, aH + ks * 8, vd, idesc2, fresh ^ 1u);
          tc_mma_tf32_ts(tmem, aL + ks * 8, vd, idesc1, 1u);
          fresh = 0;
        }
        tc_commit(&op_empty[o]);
        bool last;
        if ((q & 1) && drain_after(q >> 1, &last)) {
          tc_commit(&acc_full);
          fresh = 1;
          ++ndrain;
        }
      }
    }
  } else {
    // ---------------------------------------------------------------- split (W to tensor memory, V to planes), drain
    constexpr int HB = B / 2;
    const int quad = warp & 3, half = warp >> 2;
    const uint32_t tlane = tmem + ((uint32_t)(quad * 32) << 16);
    float acc[HB];
#pragma unroll
    for (int j = 0; j < HB; ++j) acc[j] = 0.f;
    int ndrain = 0;
    const uint32_t raw0 = smem_u32(smem), op0 = smem_u32(ops) + tid * 16;
    for (int q = 0; q < nsub; ++q) {
      const int s = q % RS, o = q % OS;
      if (!mbar_wait(&raw_full[s], (q / RS) & 1, ctrl)) break;
      if (q >= OS && !mbar_wait(&op_empty[o], ((q / OS) - 1) & 1, ctrl)) break;
      tc_fence_after();
      // W: column quad * 32 + lane of the tile (box `quad`), rows half * 16 ... of the stage
      {
        const uint32_t wbox = raw0 + s * RAW + (NBV + quad) * BOX + (lane & 7) * 4;
        float hi[16], lo[16];
#pragma unroll
        for (int kk = 0; kk < 16; ++kk) {
          const int k = half * 16 + kk;
          const float x = lds32(wbox + k * 128 + ((((uint32_t)lane >> 3) ^ ((uint32_t)k & 3u)) << 5));
          hi[kk] = tf32_rn(x);
          lo[kk] = tf32_rn(x - hi[kk]);
        }
        tmem_st16(tlane + TA + o * 64 + half * 16, hi);
        tmem_st16(tlane + TA + o * 64 + 32 + half * 16, lo);
      }
      // V: one 16-byte chunk per box and thread, planes at the same offsets
      {
        const uint32_t src = raw0 + s * RAW + tid * 16, dst = op0 + o * OPS;
        float4 x[NBV];
#pragma unroll
        for (int bx = 0; bx < NBV; ++bx) x[bx] = lds128(src + bx * BOX);
#pragma unroll
        for (int bx = 0; bx < NBV; ++bx) {
          float4 h, l;
          h.x = tf32_rn(x[bx].x);
          h.y = tf32_rn(x[bx].y);
          h.z = tf32_rn(x[bx].z);
          h.w = tf32_rn(x[bx].w);
          l.x = tf32_rn(x[bx].x - h.x);
          l.y = tf32_rn(x[bx].y - h.y);
          l.z = tf32_rn(x[bx].z - h.z);
          l.w = tf32_rn(x[bx].w - h.w);
          sts128(dst + bx * BOX, h);
          sts128(dst + (NBV + bx) * BOX, l);
        }
      }
      tmem_st_wait();
      tc_fence_before();
      proxy_fence_async_smem();
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(&op_full[o]);
        mbar_arrive(&raw_empty[s]);     // every value read from the stage has been used by the stores above
      }
      bool last;
      if ((q & 1) && drain_after(q >> 1, &last)) {
        if (!mbar_wait(&acc_full, ndrain & 1, ctrl)) break;
        ++ndrain;
        tc_fence_after();
        const uint32_t taddr = tlane + half * HB;
#pragma unroll
        for (int jj = 0; jj < HB / 16; ++jj) {
          float v[16], w[16];
          tmem_ld16(taddr + jj * 16, v);
          tmem_ld16(taddr + B + jj * 16, w);
#pragma unroll
          for (int e = 0; e < 16; ++e) acc[jj * 16 + e] += v[e] + w[e];
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&acc_empty);
        if (last) {
          const int c = (L0 + (q >> 1)) / KT;
          float* out = Zpart + (size_t)(p + c) * (size_t)(B * kTcBN) + (size_t)(half * HB) * kTcBN + quad * 32 + lane;
#pragma unroll
          for (int j = 0; j < HB; ++j) {
            out[(size_t)j * kTcBN] = acc[j];
            acc[j] = 0.f;
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, Cfg::COLS);
}

}  // namespace rrf
