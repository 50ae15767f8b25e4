// Single-precision fused update of a block step (Algorithm 2 line 8, second product, with the norms
// of line 9 and the next sample of line 7) on the fifth-generation tensor cores.
//
// Same tiles (row slab of 128, column tile of 64), same stream-K ranges, same output slots and the
// same norm partials as upd_sk_kernel.  Per tile:
//   P     = V[slab, :] Zt[tile, :]^T                  K = B      (GEMM 1)
//   Wnew  = W[slab, tile] - P  -> back into the W tile's place in shared memory and from there to global memory
//                                 by a TMA store (whole 128-byte lines); sums of squares for the norms
//   Y    += Wnew OmegaT[j0 .. j0+B, tile]^T           K = 64     (GEMM 2, only if j0 >= 0)
// The left operand of both products sits in TENSOR MEMORY (lane = row of the slab, one column per
// contraction index): V is written there once per slab, Wnew once per tile by the very threads that
// compute it, each split into its two TF32 planes on the way.  The right operands are Zt and OmegaT
// rows, which arrive by TMA already split (split_planes_kernel wrote the planes to global memory:
// both are small and stay in L2), K-contiguous with the ordinary 128-byte swizzle.  So shared memory
// carries only what TMA brings - W, Zt planes, OmegaT planes - and is read once by the tensor core
// and (W) once by the epilogue: about 220 KB of shared-memory traffic per 64 KB of HBM traffic.
//
// 3xTF32 as everywhere, D += A_lo B_hi + A_hi B_lo + A_hi B_hi, but in two instructions per K step: the
// hi and lo planes of the right operand lie one after the other in shared memory, so one instruction
// with twice the columns forms A_hi [B_hi | B_lo] and a second one adds A_lo B_hi to the first half;
// the halves are added when the accumulator is read.  (One thread issues a dependent tf32 instruction
// every 52 to 64 clocks whether it has 64 or 128 columns - 128 is where the tensor core itself needs
// 64 - so the wider instruction is free.)  The accumulator of P lives for one tile (K = B), that of Y
// for `chunk` tiles before it is added, rounded to nearest, into registers.
//
// Warp roles: 0-7 epilogue (warp w owns tensor-memory lanes 32 (w % 4) ... = those rows of the slab,
// and columns 32 (w / 4) ... of the tile = one TMA box of W), 8 TMA producer of W, 9 MMA issuer,
// 10 and 11 TMA producers of the Zt and OmegaT planes.
// Tensor-memory columns: [V_hi V_lo | Wnew_hi Wnew_lo | P, P's hi x lo part | Y, Y's hi x lo part].
#pragma once

#include "gemm_tc.cuh"
#include "panel_tsqr.cuh"

namespace rrf {

// dst[0][r][c] = tf32(src[r][c]), dst[1][r][c] = tf32(src[r][c] - dst[0][r][c]); dst planes have leading dimension ldd
__global__ void split_planes_kernel(const float* __restrict__ src, long long lds, int rows, int cols,
                                    float* __restrict__ dst, long long ldd, const int* __restrict__ done_flag) {
  if (done_flag != nullptr && *done_flag) return;
  const long long total = (long long)rows * cols;
  const size_t plane = (size_t)rows * (size_t)ldd;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    const int r = (int)(i / cols), c = (int)(i - (long long)r * cols);
    const float x = src[(size_t)r * lds + c];
    const float h = tf32_rn(x);
    dst[(size_t)r * ldd + c] = h;
    dst[plane + (size_t)r * ldd + c] = tf32_rn(x - h);
  }
}

// K-contiguous shared-memory operand with the 128-byte swizzle: rows of 128 bytes, groups of eight rows 1024 bytes apart
__device__ __forceinline__ uint64_t tc_desc_k(uint32_t addr) {
  return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024u >> 4) << 32) | (1ull << 46) |
         (2ull << 61);
}
__host__ __device__ constexpr uint32_t tc_idesc_tf32_k(int M, int N) {
  return (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
// D (+)= A B with A in tensor memory (lane = row, column = contraction index)
__device__ __forceinline__ void tc_mma_tf32_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::tf32 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b), "r"(idesc), "r"(accumulate)
      : "memory");
}
// 16 consecutive columns of this thread's tensor-memory lane <- registers
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const float (&v)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
      ::"r"(taddr), "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])),
        "r"(__float_as_uint(v[3])), "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])),
        "r"(__float_as_uint(v[7])), "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])),
        "r"(__float_as_uint(v[11])), "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])),
        "r"(__float_as_uint(v[15]))
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
// 2-D tiled TMA store: box in shared memory -> element coordinates (x = innermost, y); rows and columns outside the
// tensor are not written
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t smem_src, int x, int y) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
               ::"l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(smem_src)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// Optional cycle accounting of one CTA's waits (compiled in with -DRRF_TSQR_TRACE only)
#ifdef RRF_TSQR_TRACE
#define UTC_TRACE_DECL long long utc_acc[8] = {0, 0, 0, 0, 0, 0, 0, 0}; const bool utc_on = blockIdx.x == 5 && (threadIdx.x & 31) == 0 && do_sample
#define UTC_T(slot, ...) { const long long utc_t0 = clock64(); __VA_ARGS__; utc_acc[slot] += clock64() - utc_t0; }
#define UTC_DUMP(base) if (utc_on) { for (int q_ = 0; q_ < 8; ++q_) g_tsqr_trace[(base) + q_] = (unsigned long long)utc_acc[q_]; }
#else
#define UTC_TRACE_DECL
#define UTC_T(slot, ...) { __VA_ARGS__; }
#define UTC_DUMP(base)
#endif

constexpr int kUtcBM = 128, kUtcBN = 64;
constexpr int kUtcEpi = 8;
// The sampled panel Y is summed in tensor memory over this many times more 64-element pieces of its contraction
// index than Z is (the chunk length of rrf_set_single_engine): an error in Y moves the sample, not the accuracy
// of the factorisation, and every drain of Y stalls both the issuer and the epilogue warps for one product.
constexpr int kUtcYChunkFactor = 8;
constexpr int kUtcThreads = (kUtcEpi + 4) * 32;     // + W producer, MMA issuer, Zt producer, OmegaT producer

// Shared memory is three independent TMA rings, because the three inputs of a tile are given back at
// different times: the W tile once the epilogue warps have it in registers, the Zt planes once the
// first product is complete, the OmegaT planes once the second is.  W comes from DRAM and gets the
// deepest ring; the planes come from L2.
template <int B>
struct UtcCfg {
  static constexpr int W_BOX = kUtcBM * 128;            // 128 rows x 32 columns
  static constexpr int W_BYTES = 2 * W_BOX;
  static constexpr int Z_BOX = kUtcBN * 128;            // 64 rows of Zt (columns of the tile) x 32 contraction indices
  static constexpr int KBZ = B / 32;
  static constexpr int Z_BYTES = KBZ * 2 * Z_BOX;       // per K box: hi rows, then lo rows
  static constexpr int O_BOX = B * 128;                 // B rows of OmegaT x 32 columns of the tile
  static constexpr int O_BYTES = 2 * 2 * O_BOX;         // per K box (two of them): hi rows, then lo rows
  static constexpr int NW = 3, NZ = (B == 64) ? 2 : 3, NO = (B == 64) ? 2 : 3;
  static constexpr int SMEM = NW * W_BYTES + NZ * Z_BYTES + NO * O_BYTES + 1024;
  // tensor-memory columns: [V_hi V_lo | Wnew_hi Wnew_lo | P and its hi x lo part | Y and its hi x lo part]
  static constexpr int TV = 0, TW = 2 * B, TD = TW + 2 * kUtcBN, TY = TD + 2 * kUtcBN;
  static constexpr int COLS = 512;
  static_assert(TY + 2 * B <= COLS, "tensor memory");
  static_assert(SMEM + 2048 <= 232448, "shared memory");
};

template <int B>
__global__ void __launch_bounds__(kUtcThreads, 1)
    upd_tc_kernel(const __grid_constant__ CUtensorMap tmC,   // C [m][ncols], box [128][32]
                  const __grid_constant__ CUtensorMap tmZs,  // Zt planes [2 npad][B], box [64][32]
                  const __grid_constant__ CUtensorMap tmOs,  // OmegaT planes [2 B][n], box [B][32]
                  const __grid_constant__ CUtensorMap tmCs,  // C as written [r0 + rows][ncols], box [32][32]
                  const __grid_constant__ CUtensorMap tmTs,  // rows of B being formed [top_rows][ncols], box [32][32]
                  const float* __restrict__ V, long long ldv, int r0, int rows, int ncols, int cv0, int top_rows,
                  int sample, int npad, float* __restrict__ Ypart, double* __restrict__ norm_part,
                  int NC, int total, int tpc, int chunk, Ctrl* ctrl) {
  if (*reinterpret_cast<volatile int*>(&ctrl->done)) return;
  using Cfg = UtcCfg<B>;
  constexpr int NW = Cfg::NW, NZ = Cfg::NZ, NO = Cfg::NO, W_BOX = Cfg::W_BOX, W_BYTES = Cfg::W_BYTES, Z_BOX = Cfg::Z_BOX,
                Z_BYTES = Cfg::Z_BYTES, O_BOX = Cfg::O_BOX, O_BYTES = Cfg::O_BYTES, KBZ = Cfg::KBZ;
  constexpr int TV = Cfg::TV, TW = Cfg::TW, TD = Cfg::TD, TY = Cfg::TY;
  constexpr int BN = kUtcBN, BM = kUtcBM;
  static_assert(B == 32 || B == 64, "block sizes with a 128-row slab");

  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = align1024(smem_raw);
  unsigned char* ringW = smem;
  unsigned char* ringZ = ringW + NW * W_BYTES;
  unsigned char* ringO = ringZ + NZ * Z_BYTES;
  __shared__ uint64_t wfull[NW], wempty[NW], zfull[NZ], zempty[NZ], ofull[NO], oempty[NO];
  __shared__ uint64_t v_ready, d_full, d_empty, w_ready, w_empty, y_full, y_empty;
  __shared__ uint32_t tmem_slot;
  __shared__ double red[64];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int p = blockIdx.x;
  const int L0 = p * tpc;
  const int ntile = min(total, L0 + tpc) - L0;
  const bool do_sample = sample != 0;

  if (tid == 0) {
    for (int s = 0; s < NW; ++s) {
      mbar_init(&wfull[s], 1);
      mbar_init(&wempty[s], kUtcEpi);
    }
    for (int s = 0; s < NZ; ++s) {
      mbar_init(&zfull[s], 1);
      mbar_init(&zempty[s], 1);
    }
    for (int s = 0; s < NO; ++s) {
      mbar_init(&ofull[s], 1);
      mbar_init(&oempty[s], 1);
    }
    mbar_init(&v_ready, kUtcEpi);
    mbar_init(&d_full, 1);
    mbar_init(&d_empty, kUtcEpi);
    mbar_init(&w_ready, kUtcEpi);
    mbar_init(&w_empty, 1);
    mbar_init(&y_full, 1);
    mbar_init(&y_empty, kUtcEpi);
    mbar_fence_init();
  }
  __syncthreads();
  if (warp == 0) tmem_alloc(&tmem_slot, Cfg::COLS);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(&tmem_slot);

  // The Y accumulator is drained after the tile in column c of a slab if that tile ends the slab (or this CTA's
  // range), or closes a chunk.  Writer and reader of the accumulator both use this rule.
  auto drain_after = [&](int i, bool* last) {
    const int L = L0 + i, s = L / NC, c = L - s * NC;
    *last = (i == ntile - 1) || (c == NC - 1);
    return *last || (chunk > 0 && (c + 1) % chunk == 0);
  };

  double s_top = 0.0, s_trail = 0.0;

  if (warp == kUtcEpi) {
    // ---------------------------------------------------------------- TMA producer: W tiles
    if (lane == 0) {
      for (int i = 0; i < ntile; ++i) {
        const int st = i % NW;
        if (i >= NW && !mbar_wait(&wempty[st], ((i / NW) - 1) & 1, ctrl)) break;
        const int L = L0 + i, s = L / NC, c = L - s * NC;
        unsigned char* sW = ringW + st * W_BYTES;
        mbar_expect_tx(&wfull[st], W_BYTES);
#pragma unroll
        for (int q = 0; q < 2; ++q) tma_load_2d(sW + q * W_BOX, &tmC, c * BN + q * 32, r0 + s * BM, &wfull[st]);
      }
    }
  } else if (warp == kUtcEpi + 2) {
    // ---------------------------------------------------------------- TMA producer: Zt planes
    if (lane == 0) {
      for (int i = 0; i < ntile; ++i) {
        const int st = i % NZ;
        if (i >= NZ && !mbar_wait(&zempty[st], ((i / NZ) - 1) & 1, ctrl)) break;
        const int L = L0 + i, s = L / NC, c = L - s * NC;
        unsigned char* sZ = ringZ + st * Z_BYTES;
        mbar_expect_tx(&zfull[st], Z_BYTES);
#pragma unroll
        for (int kb = 0; kb < KBZ; ++kb) {
          tma_load_2d(sZ + kb * 2 * Z_BOX, &tmZs, kb * 32, c * BN, &zfull[st]);
          tma_load_2d(sZ + kb * 2 * Z_BOX + Z_BOX, &tmZs, kb * 32, npad + c * BN, &zfull[st]);
        }
      }
    }
  } else if (warp == kUtcEpi + 3) {
    // ---------------------------------------------------------------- TMA producer: OmegaT planes
    if (lane == 0 && do_sample) {
      for (int i = 0; i < ntile; ++i) {
        const int st = i % NO;
        if (i >= NO && !mbar_wait(&oempty[st], ((i / NO) - 1) & 1, ctrl)) break;
        const int L = L0 + i, s = L / NC, c = L - s * NC;
        unsigned char* sO = ringO + st * O_BYTES;
        mbar_expect_tx(&ofull[st], O_BYTES);
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          tma_load_2d(sO + q * 2 * O_BOX, &tmOs, c * BN + q * 32, 0, &ofull[st]);
          tma_load_2d(sO + q * 2 * O_BOX + O_BOX, &tmOs, c * BN + q * 32, B, &ofull[st]);
        }
      }
    }
  } else if (warp == kUtcEpi + 1) {
    // ---------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      constexpr uint32_t idescP2 = tc_idesc_tf32_k(BM, 2 * BN), idescP1 = tc_idesc_tf32_k(BM, BN);
      constexpr uint32_t idescY2 = tc_idesc_tf32_k(BM, 2 * B), idescY1 = tc_idesc_tf32_k(BM, B);
      uint32_t fresh_y = 1;
      int ny = 0, cur_s = -1, nslab = 0;
      bool ok = true;
      UTC_TRACE_DECL;
      const long long utc_start = clock64();
      // Y += Wnew(i) OmegaT^T
      auto gemm2 = [&](int i) {
        const int st = i % NO;
        UTC_T(1, if (!mbar_wait(&ofull[st], (i / NO) & 1, ctrl)) { ok = false; return; })
        UTC_T(2, if (!mbar_wait(&w_ready, i & 1, ctrl)) { ok = false; return; })
        UTC_T(1, if (fresh_y && ny > 0 && !mbar_wait(&y_empty, (ny - 1) & 1, ctrl)) { ok = false; return; })
        tc_fence_after();
        const uint32_t sO = smem_u32(ringO + st * O_BYTES);
#ifdef RRF_TSQR_TRACE
        const long long utc_g2 = clock64();
#endif
#pragma unroll
        for (int ks = 0; ks < BN / 8; ++ks) {
          const uint64_t oh = tc_desc_k(sO + (ks / 4) * 2 * O_BOX + (ks % 4) * 32);   // hi rows, lo rows right behind
          const uint32_t ah = tmem + TW + ks * 8, al = ah + BN;
          tc_mma_tf32_ts(tmem + TY, ah, oh, idescY2, fresh_y ^ 1u);
          tc_mma_tf32_ts(tmem + TY, al, oh, idescY1, 1u);
          fresh_y = 0;
        }
        tc_commit(&w_empty);
        tc_commit(&oempty[st]);
#ifdef RRF_TSQR_TRACE
        utc_acc[3] += clock64() - utc_g2;      // issue of the second product
#endif
        bool last;
        if (drain_after(i, &last)) {
          tc_commit(&y_full);
          fresh_y = 1;
          ++ny;
        }
      };
      for (int i = 0; i < ntile && ok; ++i) {
        const int st = i % NZ;
        const int L = L0 + i, s = L / NC;
        bool last;
        // a tile after which Y is drained (and a slab change, which always follows one) must not wait behind
        // the next tile's first product: the epilogue warps stand at that drain
        const bool early = do_sample && i > 0 && drain_after(i - 1, &last);
        if (early) gemm2(i - 1);
        if (!ok) break;
        UTC_T(4, if (!mbar_wait(&zfull[st], (i / NZ) & 1, ctrl)) break;)
        if (s != cur_s) {
          UTC_T(4, if (!mbar_wait(&v_ready, nslab & 1, ctrl)) break;)
          ++nslab;
          cur_s = s;
        }
        UTC_T(6, if (i >= 1 && !mbar_wait(&d_empty, (i - 1) & 1, ctrl)) break;)
        tc_fence_after();
        const uint32_t sZ = smem_u32(ringZ + st * Z_BYTES);
#ifdef RRF_TSQR_TRACE
        const long long utc_g1 = clock64();
#endif
#pragma unroll
        for (int ks = 0; ks < B / 8; ++ks) {
          const uint64_t zh = tc_desc_k(sZ + (ks / 4) * 2 * Z_BOX + (ks % 4) * 32);   // hi rows, lo rows right behind
          const uint32_t ah = tmem + TV + ks * 8, al = ah + B;
          tc_mma_tf32_ts(tmem + TD, ah, zh, idescP2, ks > 0 ? 1u : 0u);
          tc_mma_tf32_ts(tmem + TD, al, zh, idescP1, 1u);
        }
        tc_commit(&d_full);
        tc_commit(&zempty[st]);
#ifdef RRF_TSQR_TRACE
        utc_acc[5] += clock64() - utc_g1;      // issue of the first product
#endif
        if (do_sample && i > 0 && !early) gemm2(i - 1);
      }
      if (ok && do_sample && ntile > 0) gemm2(ntile - 1);
#ifdef RRF_TSQR_TRACE
      utc_acc[0] = clock64() - utc_start;
      utc_acc[7] = ntile;
#endif
      UTC_DUMP(16)
    }
  } else {
    // ---------------------------------------------------------------- epilogue warps
    constexpr int HB = B / 2;                  // this warp's columns of V and of Y
    const int quad = warp & 3, half = warp >> 2;
    const int r = quad * 32 + lane;            // row inside the slab = tensor-memory lane
    const uint32_t tlane = tmem + ((uint32_t)(quad * 32) << 16);
    float accY[HB];
#pragma unroll
    for (int j = 0; j < HB; ++j) accY[j] = 0.f;
    int cur_s = -1, ny = 0;
    UTC_TRACE_DECL;
    const long long utc_start = clock64();
    bool is_top = false;
    for (int i = 0; i < ntile; ++i) {
      const int st = i % NW;
      const int L = L0 + i, s = L / NC, c = L - s * NC;
      if (i > 0 && lane == 0) {
        // the TMA store of the previous tile has read its part of the W ring by now (it was issued a whole
        // tile ago); only then does that slot go back to the producer
        bulk_wait_read();
        mbar_arrive(&wempty[(i - 1) % NW]);
      }
      if (s != cur_s) {
        // V[slab] -> tensor memory, split (every product of the previous slab that reads it is complete: the
        // accumulator of its last tile has been drained)
        const int lr = s * BM + r;
        const float* vrow = V + (size_t)(r0 + lr) * ldv + cv0 + half * HB;
#pragma unroll
        for (int g = 0; g < HB / 16; ++g) {
          float hi[16], lo[16];
#pragma unroll
          for (int e4 = 0; e4 < 4; ++e4) {
            float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
            if (lr < rows) x = *reinterpret_cast<const float4*>(vrow + g * 16 + e4 * 4);
            const float xs[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              hi[e4 * 4 + e] = tf32_rn(xs[e]);
              lo[e4 * 4 + e] = tf32_rn(xs[e] - hi[e4 * 4 + e]);
            }
          }
          tmem_st16(tlane + TV + half * HB + g * 16, hi);
          tmem_st16(tlane + TV + B + half * HB + g * 16, lo);
        }
        tmem_st_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&v_ready);
        cur_s = s;
        is_top = lr < top_rows;        // top_rows is a multiple of 32: the same for the whole warp
      }
      UTC_T(1, if (!mbar_wait(&wfull[st], (i / NW) & 1, ctrl)) break;)
      UTC_T(2, if (!mbar_wait(&d_full, i & 1, ctrl)) break;)
#ifdef RRF_TSQR_TRACE
      const long long utc_e0 = clock64();
#endif
      tc_fence_after();
      float y[32];
      {
        float pa[16], pb[16];
        {
          float qa[16], qb[16];                 // the hi x lo part of P
          tmem_ld16x4(tlane + TD + half * 32, tlane + TD + half * 32 + 16, tlane + TD + BN + half * 32,
                      tlane + TD + BN + half * 32 + 16, pa, pb, qa, qb);
#pragma unroll
          for (int e = 0; e < 16; ++e) {
            pa[e] += qa[e];
            pb[e] += qb[e];
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&d_empty);
        const uint32_t sW = smem_u32(ringW + st * W_BYTES + half * W_BOX + r * 128);
#pragma unroll
        for (int c16 = 0; c16 < 8; ++c16) {
          const float4 w = lds128(sW + (((uint32_t)c16 ^ (uint32_t)(r & 7)) << 4));
          const float* pp = c16 < 4 ? pa + c16 * 4 : pb + (c16 - 4) * 4;
          y[c16 * 4 + 0] = w.x - pp[0];
          y[c16 * 4 + 1] = w.y - pp[1];
          y[c16 * 4 + 2] = w.z - pp[2];
          y[c16 * 4 + 3] = w.w - pp[3];
        }
      }
      // ---- Wnew goes back to where the W tile stood in shared memory (same swizzled places, so each thread
      // overwrites exactly what it has read) and TMA stores this warp's 32 x 32 box in whole 128-byte lines;
      // rows past the matrix and columns past its width are zero here and are not written.  Norms on the side:
      // four single-precision partial sums of eight squares each, added in double precision.
      {
        const uint32_t sW = smem_u32(ringW + st * W_BYTES + half * W_BOX + r * 128);
        float q4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int c16 = 0; c16 < 8; ++c16) {
          sts128(sW + (((uint32_t)c16 ^ (uint32_t)(r & 7)) << 4),
                 make_float4(y[c16 * 4], y[c16 * 4 + 1], y[c16 * 4 + 2], y[c16 * 4 + 3]));
#pragma unroll
          for (int e = 0; e < 4; ++e) q4[c16 & 3] = fmaf(y[c16 * 4 + e], y[c16 * 4 + e], q4[c16 & 3]);
        }
        proxy_fence_async_smem();
        __syncwarp();
        if (lane == 0) {
          const int lr0 = s * BM + quad * 32;
          if (lr0 < rows) {
            const uint32_t box = smem_u32(ringW + st * W_BYTES + half * W_BOX + quad * 32 * 128);
            if (lr0 < top_rows) tma_store_2d(&tmTs, box, c * BN + half * 32, lr0);
            else tma_store_2d(&tmCs, box, c * BN + half * 32, r0 + lr0);
          }
          bulk_commit();
        }
        const double q = ((double)q4[0] + (double)q4[1]) + ((double)q4[2] + (double)q4[3]);
        s_top += is_top ? q : 0.0;
        s_trail += is_top ? 0.0 : q;
      }
      if (do_sample) {
        // ---- Wnew -> tensor memory, split, as the left operand of the sample product
#ifdef RRF_TSQR_TRACE
        utc_acc[5] += clock64() - utc_e0;      // P, W, store, norms
#endif
        UTC_T(3, if (i > 0 && !mbar_wait(&w_empty, (i - 1) & 1, ctrl)) break;)
#ifdef RRF_TSQR_TRACE
        const long long utc_e1 = clock64();
#endif
        tc_fence_after();
#pragma unroll
        for (int g = 0; g < 2; ++g) {
          float hi[16], lo[16];
#pragma unroll
          for (int e = 0; e < 16; ++e) {
            hi[e] = tf32_rn(y[g * 16 + e]);
            lo[e] = tf32_rn(y[g * 16 + e] - hi[e]);
          }
          tmem_st16(tlane + TW + half * 32 + g * 16, hi);
          tmem_st16(tlane + TW + BN + half * 32 + g * 16, lo);
        }
        tmem_st_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&w_ready);
#ifdef RRF_TSQR_TRACE
        utc_acc[6] += clock64() - utc_e1;      // split + store to tensor memory
#endif
        bool last;
        if (drain_after(i, &last)) {
          UTC_T(4, if (!mbar_wait(&y_full, ny & 1, ctrl)) break;)
          ++ny;
          tc_fence_after();
#pragma unroll
          for (int g = 0; g < HB / 16; ++g) {
            float v[16], w2[16];
            tmem_ld16(tlane + TY + half * HB + g * 16, v);
            tmem_ld16(tlane + TY + B + half * HB + g * 16, w2);      // the hi x lo part
#pragma unroll
            for (int e = 0; e < 16; ++e) accY[g * 16 + e] += v[e] + w2[e];
          }
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&y_empty);
          if (last) {
            float* out = Ypart + (size_t)(p + s) * (size_t)(BM * B) + (size_t)r * B + half * HB;
#pragma unroll
            for (int k = 0; k < HB / 4; ++k) {
              *reinterpret_cast<float4*>(out + 4 * k) = make_float4(accY[4 * k], accY[4 * k + 1], accY[4 * k + 2], accY[4 * k + 3]);
              accY[4 * k] = accY[4 * k + 1] = accY[4 * k + 2] = accY[4 * k + 3] = 0.f;
            }
          }
        }
      }
    }
    if (lane == 0) bulk_wait_all();      // this warp's stores are complete before the CTA may exit
#ifdef RRF_TSQR_TRACE
    utc_acc[0] = clock64() - utc_start;
    if (warp == 0) { UTC_DUMP(0) }
#endif
  }
  // per-CTA norm partials (all warps join; producer and issuer contribute zeros), then the common exit
  const double bt = block_sum(s_top, red);
  const double br = block_sum(s_trail, red + 32);
  if (tid == 0 && norm_part != nullptr) {
    norm_part[2 * p] = bt;
    norm_part[2 * p + 1] = br;
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, Cfg::COLS);
}

}  // namespace rrf
