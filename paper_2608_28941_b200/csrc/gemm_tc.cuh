// Single-precision Z = V_i^T W[r0:, :] (Algorithm 2 line 8, first product) on the fifth-generation tensor
// cores: tcgen05.mma kind::tf32, operands in shared memory, accumulator in tensor memory.
//
// Same tiling, same stream-K ranges and the same partial-result slots as vtw_sk_kernel, so the
// consumer of the partials does not know which of the two ran.  What differs is the engine:
//
//   * The instruction computes D[128 x B] (+)= A[128 x 8] * B[8 x B] with A = (W tile)^T and B = V tile.
//     Both tiles arrive by TMA with a 128-byte line holding one contraction index and 32 consecutive
//     columns, which is the instruction's transposed ("MN-major") operand form; for 32-bit operands
//     that form needs the swizzle with 32-byte atoms, so these tensor maps differ from the mma.sync
//     kernel's in the swizzle mode (and in the box height).  No transposition anywhere.
//   * fp32 accuracy comes from the same 3xTF32 split as the mma.sync path, x = hi + lo with
//     hi = tf32(x), lo = tf32(x - hi), D += A_lo B_hi + A_hi B_lo + A_hi B_hi.  The split is an
//     element-wise pass by eight warps from the TMA ring into a second ring of (hi, lo) planes at
//     the same byte offsets within a box, so the swizzle never has to be decoded.
//   * The tensor core's own accumulation does not round to nearest.  `chunk` bounds how many
//     64-row tiles are summed inside tensor memory before those warps add the accumulator into
//     registers with ordinary round-to-nearest adds (0: a whole accumulator stays in tensor memory).
//
// Warp roles: 0-7 split operands and drain the accumulator (warp w owns tensor-memory lanes
// 32 (w % 4) ..., i.e. those columns of the tile, and half w / 4 of the B rows of Z), 8 issues TMA
// loads, 9 issues the MMAs.
// Every wait is bounded; on a time-out all roles fall through to the common exit, where tensor
// memory is released.
#pragma once

#include "gemm_sk.cuh"

namespace rrf {

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void proxy_fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// whole warp; writes the base address of `ncols` tensor-memory columns (a power of two >= 32) to *slot
__device__ __forceinline__ void tmem_alloc(uint32_t* slot, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot)), "r"(ncols)
               : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t base, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(base), "r"(ncols) : "memory");
}
// mbarrier arrival once every MMA this thread has issued so far is complete
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}
// Shared-memory operand descriptor for a 32-bit operand whose rows are contraction indices ("MN-major"):
// 128-byte lines of 32 elements along M or N, consecutive lines are consecutive contraction indices,
// and the 32-byte quarter of a line is XORed with the line index modulo 4.  This is the one layout in
// which the tensor core accepts a transposed TF32 operand (with the ordinary 16-byte-chunk swizzle it
// returns zeros), and TMA writes it with CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B.
// `addr` is the first of the eight lines of one K step, `lbo` the byte distance between groups of
// 32 elements along M or N; groups of four lines follow each other at 512 bytes.
__device__ __forceinline__ uint64_t tc_desc(uint32_t addr, uint32_t lbo) {
  return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)((lbo >> 4) & 0x3FFFu) << 16) |
         ((uint64_t)(512u >> 4) << 32) | (1ull << 46) | (1ull << 61);
}
// fp32 accumulator, TF32 operands, both MN-major, D is M x N
__host__ __device__ constexpr uint32_t tc_idesc_tf32(int M, int N) {
  return (1u << 4) | (2u << 7) | (2u << 10) | (1u << 15) | (1u << 16) | ((uint32_t)(N >> 3) << 17) |
         ((uint32_t)(M >> 4) << 24);
}
__device__ __forceinline__ void tc_mma_tf32(uint32_t d_tmem, uint64_t a, uint64_t b, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a), "l"(b), "r"(idesc), "r"(accumulate)
      : "memory");
}
// 16 consecutive columns of this thread's tensor-memory lane.  The load is asynchronous: its registers are
// defined only after tcgen05.wait::ld, so both instructions sit in one asm statement and nothing - not even a
// register copy - can be scheduled between them.
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16]) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];\n\t"
      "tcgen05.wait::ld.sync.aligned;"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// four such loads in flight together, one wait
__device__ __forceinline__ void tmem_ld16x4(uint32_t t0, uint32_t t1, uint32_t t2, uint32_t t3, float (&a)[16],
                                            float (&b)[16], float (&c)[16], float (&d)[16]) {
  uint32_t r[64];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%64];\n\t"
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%65];\n\t"
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%32,%33,%34,%35,%36,%37,%38,%39,%40,%41,%42,%43,%44,%45,%46,%47}, [%66];\n\t"
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%48,%49,%50,%51,%52,%53,%54,%55,%56,%57,%58,%59,%60,%61,%62,%63}, [%67];\n\t"
      "tcgen05.wait::ld.sync.aligned;"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31]), "=r"(r[32]),
        "=r"(r[33]), "=r"(r[34]), "=r"(r[35]), "=r"(r[36]), "=r"(r[37]), "=r"(r[38]), "=r"(r[39]), "=r"(r[40]),
        "=r"(r[41]), "=r"(r[42]), "=r"(r[43]), "=r"(r[44]), "=r"(r[45]), "=r"(r[46]), "=r"(r[47]), "=r"(r[48]),
        "=r"(r[49]), "=r"(r[50]), "=r"(r[51]), "=r"(r[52]), "=r"(r[53]), "=r"(r[54]), "=r"(r[55]), "=r"(r[56]),
        "=r"(r[57]), "=r"(r[58]), "=r"(r[59]), "=r"(r[60]), "=r"(r[61]), "=r"(r[62]), "=r"(r[63])
      : "r"(t0), "r"(t1), "r"(t2), "r"(t3)
      : "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    a[i] = __uint_as_float(r[i]);
    b[i] = __uint_as_float(r[16 + i]);
    c[i] = __uint_as_float(r[32 + i]);
    d[i] = __uint_as_float(r[48 + i]);
  }
}

// x rounded to TF32 (nearest, ties away from zero - what cvt.rna.tf32.f32 returns) with two integer
// instructions, which issue at the full rate where the conversion instruction does not.  A NaN may come out as a
// signed zero; the kernels below use the planes only as tensor-core operands and keep x itself for everything else.
__device__ __forceinline__ float tf32_rn(float x) { return __uint_as_float((__float_as_uint(x) + 0x1000u) & 0xFFFFE000u); }

#ifdef RRF_TSQR_TRACE
__device__ unsigned long long g_vtc_trace[16];
#define VTC_DECL long long vtc_acc[8] = {0, 0, 0, 0, 0, 0, 0, 0}; const bool vtc_on = blockIdx.x == 5 && (threadIdx.x & 31) == 0
#define VTC_T(slot, ...) { const long long vtc_t0 = clock64(); __VA_ARGS__; vtc_acc[slot] += clock64() - vtc_t0; }
#define VTC_DUMP(base) if (vtc_on) { for (int q_ = 0; q_ < 8; ++q_) g_vtc_trace[(base) + q_] = (unsigned long long)vtc_acc[q_]; }
#else
#define VTC_DECL
#define VTC_T(slot, ...) { __VA_ARGS__; }
#define VTC_DUMP(base)
#endif

constexpr int kTcBN = 128;     // columns of W per accumulator = rows of D = tensor-memory lanes
constexpr int kTcSub = 32;     // rows (contraction indices) per ring stage; a 64-row tile is two stages
constexpr int kTcConv = 8;     // warps that split operands and drain the accumulator
constexpr int kTcThreads = (kTcConv + 2) * 32;

__device__ __forceinline__ float4 lds128(uint32_t a) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(a));
  return v;
}
__device__ __forceinline__ void sts128(uint32_t a, const float4& v) {
  asm volatile("st.shared.v4.f32 [%0], {%1,%2,%3,%4};" ::"r"(a), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
}

// One stage of the operand ring, in boxes of 32 lines x 128 bytes:
//   [V_hi (NBV boxes)] [V_lo (NBV)] [W_hi (NBC)] [W_lo (NBC)]
// V_lo follows V_hi at the box stride so that one descriptor covers [V_hi | V_lo] as an operand with
// 2B columns: per K step  D[:, 0:2B] += W_hi^T [V_hi | V_lo]  and  D[:, 0:B] += W_lo^T V_hi  - two
// instructions instead of three, and 14 KB instead of 18 KB read from shared memory (B = 64), which
// is what bounds the tensor core here.  Columns j and B + j of the accumulator are added when it is drained.
template <int B, int RS, int OS>
struct TcCfg {
  static constexpr int NBV = B / 32, NBC = kTcBN / 32;
  static constexpr int BOX = kTcSub * 128;
  static constexpr int RAW = (NBV + NBC) * BOX;       // one stage of the TMA ring
  static constexpr int OPS = 2 * RAW;                 // one stage of the operand ring
  static constexpr int SMEM = RS * RAW + OS * OPS + 1024;
  static constexpr int COLS = 2 * B;                  // tensor-memory columns of the accumulator
};

template <int B, int RS, int OS>
__global__ void __launch_bounds__(kTcThreads, 1)
    vtw_tc_kernel(const __grid_constant__ CUtensorMap tmV,  // V [m][ldv], box [32][32]
                  const __grid_constant__ CUtensorMap tmC,  // C [m][ncols], box [32][32]
                  float* __restrict__ Zpart, int r0, int cv0, int KT, int total, int tpc, int chunk, Ctrl* ctrl) {
  if (*reinterpret_cast<volatile int*>(&ctrl->done)) return;
  using Cfg = TcCfg<B, RS, OS>;
  constexpr int NBV = Cfg::NBV, NBC = Cfg::NBC, BOX = Cfg::BOX, RAW = Cfg::RAW, OPS = Cfg::OPS, COLS = Cfg::COLS;
  static_assert(B == 32 || B == 64 || B == 128, "tensor-memory columns: a power of two, at least 32");
  static_assert(BOX / 16 == kTcConv * 32, "one 16-byte chunk of a box per converter thread");

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
  if (warp == 0) tmem_alloc(&tmem_slot, COLS);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(&tmem_slot);

  // After the second stage of tile i the accumulator is drained if the tile is the last one of its column tile
  // (or of this CTA's range), or if it closes a chunk.  Writer and reader of the accumulator both use this rule.
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
      constexpr uint32_t idesc2 = tc_idesc_tf32(kTcBN, 2 * B), idesc1 = tc_idesc_tf32(kTcBN, B);
      uint32_t fresh = 1;        // the next product overwrites the accumulator
      int ndrain = 0;
      VTC_DECL;
      const long long vtc_s = clock64();
      for (int q = 0; q < nsub; ++q) {
        const int o = q % OS;
        VTC_T(1, if (!mbar_wait(&op_full[o], (q / OS) & 1, ctrl)) break;)
        VTC_T(2, if (fresh && ndrain > 0 && !mbar_wait(&acc_empty, (ndrain - 1) & 1, ctrl)) break;)
        tc_fence_after();
        const uint32_t vH = smem_u32(ops + o * OPS), wH = vH + 2 * NBV * BOX, wL = wH + NBC * BOX;
#pragma unroll
        for (int ks = 0; ks < kTcSub / 8; ++ks) {
          tc_mma_tf32(tmem, tc_desc(wH + ks * 1024, BOX), tc_desc(vH + ks * 1024, BOX), idesc2, fresh ^ 1u);
          tc_mma_tf32(tmem, tc_desc(wL + ks * 1024, BOX), tc_desc(vH + ks * 1024, BOX), idesc1, 1u);
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
#ifdef RRF_TSQR_TRACE
      vtc_acc[0] = clock64() - vtc_s;
      vtc_acc[7] = nsub;
#endif
      VTC_DUMP(8)
    }
  } else {
    // ---------------------------------------------------------------- operand split + accumulator drain
    // warp w drains lanes 32 (w % 4) ... of tensor memory (the hardware's rule) and half w / 4 of the B columns
    constexpr int HB = B / 2;
    const int quad = warp & 3, half = warp >> 2;
    float acc[HB];
#pragma unroll
    for (int j = 0; j < HB; ++j) acc[j] = 0.f;
    int ndrain = 0;
    const uint32_t raw0 = smem_u32(smem) + tid * 16, op0 = smem_u32(ops) + tid * 16;
    VTC_DECL;
    const long long vtc_s = clock64();
    for (int q = 0; q < nsub; ++q) {
      const int s = q % RS, o = q % OS;
      VTC_T(1, if (!mbar_wait(&raw_full[s], (q / RS) & 1, ctrl)) break;)
      VTC_T(2, if (q >= OS && !mbar_wait(&op_empty[o], ((q / OS) - 1) & 1, ctrl)) break;)
#ifdef RRF_TSQR_TRACE
      const long long vtc_c0 = clock64();
#endif
      const uint32_t src = raw0 + s * RAW, dst = op0 + o * OPS;
      float4 x[NBV + NBC];
#pragma unroll
      for (int bx = 0; bx < NBV + NBC; ++bx) x[bx] = lds128(src + bx * BOX);     // box bx, this thread's chunk
#pragma unroll
      for (int bx = 0; bx < NBV + NBC; ++bx) {
        float4 h, l;
        h.x = tf32_rn(x[bx].x);
        h.y = tf32_rn(x[bx].y);
        h.z = tf32_rn(x[bx].z);
        h.w = tf32_rn(x[bx].w);
        l.x = tf32_rn(x[bx].x - h.x);
        l.y = tf32_rn(x[bx].y - h.y);
        l.z = tf32_rn(x[bx].z - h.z);
        l.w = tf32_rn(x[bx].w - h.w);
        const int hb = bx < NBV ? bx : 2 * NBV + (bx - NBV);          // box of the hi plane in the operand stage
        const int lb = bx < NBV ? bx + NBV : 2 * NBV + NBC + (bx - NBV);
        sts128(dst + hb * BOX, h);
        sts128(dst + lb * BOX, l);
      }
      proxy_fence_async_smem();      // the planes are read by the tensor core through the async proxy
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(&op_full[o]);
        mbar_arrive(&raw_empty[s]);
      }
#ifdef RRF_TSQR_TRACE
      vtc_acc[4] += clock64() - vtc_c0;      // split of one stage
#endif
      bool last;
      if ((q & 1) && drain_after(q >> 1, &last)) {
        VTC_T(3, if (!mbar_wait(&acc_full, ndrain & 1, ctrl)) break;)
        ++ndrain;
#ifdef RRF_TSQR_TRACE
        const long long vtc_d0 = clock64();
#endif
        tc_fence_after();
        const uint32_t taddr = tmem + ((uint32_t)(quad * 32) << 16) + half * HB;
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
#ifdef RRF_TSQR_TRACE
        vtc_acc[5] += clock64() - vtc_d0;    // drain
#endif
      }
    }
#ifdef RRF_TSQR_TRACE
    vtc_acc[0] = clock64() - vtc_s;
    if (warp == 0) { VTC_DUMP(0) }
#endif
  }
  // common exit: nothing is in flight once the last accumulator has been drained (or a wait gave up)
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, COLS);
}

}  // namespace rrf
