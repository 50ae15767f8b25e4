// Shared device helpers: control block, bounded waits, TMA / mbarrier wrappers,
// the 128-byte-swizzle address map and the m16n8k8 tensor-core wrappers.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/rrf.h"

namespace rrf {

// Device-resident loop state of Algorithm 2 (lines 1, 4, 5, 9, 10).  Written by the
// init and stop kernels; every other kernel of a block step only reads `done`.
struct Ctrl {
  int done;        // 1 once the while-condition of Algorithm 2 line 5 (or the rank cap) is false
  int status;      // rrf_status_t, sticky for errors
  int steps;       // block steps completed (the paper's i)
  int k;           // steps * b
  unsigned bar;    // arrival counter of the panel kernel's grid barrier
  int pad[3];
  double normA2;   // ||A||_F^2
  double sigma2;   // squared absolute tolerance
  double E_sub;    // Algorithm 2 line 9
  double E_dir;    // ||W[r0+b:, :]||_F^2
  double E_prev;   // stopping quantity after the previous pass, and the ratio of the two before that:
  double r_prev;   // the history the sampling predictor extrapolates (negative: no ratio yet)
  int fused_samples;   // passes whose update also sampled a later panel
  int extra_samples;   // panels sampled by the separate kernel because the predictor had skipped them
  int n_est;           // sampled stopping rules: panels whose estimate was evaluated
  int pad2;
  double E_est;        // sampled stopping rules: the last estimate
};
static_assert(sizeof(Ctrl) <= 256, "the control block has 256 bytes of workspace");

// ~1 s at 2 GHz: every spin in this library gives up after this many SM clocks.
constexpr long long kWaitLimitClocks = 2000000000LL;

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// ---------------------------------------------------------------- mbarrier / TMA

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok;
}
// Bounded wait.  Returns false (and records RRF_ERR_TIMEOUT) when the phase never completes.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, Ctrl* ctrl) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    if (clock64() - t0 > kWaitLimitClocks) {
      atomicExch(&ctrl->status, (int)RRF_ERR_TIMEOUT);
      atomicExch(&ctrl->done, 1);          // kernels already enqueued behind this one return at once
      return false;
    }
  }
  return true;
}
// 2-D tiled TMA load: box at element coordinates (x = innermost, y) -> shared memory.
// x * sizeof(element) must be a multiple of 16 bytes.
__device__ __forceinline__ void tma_load_2d(void* smem_dst, const CUtensorMap* map, int x, int y,
                                            uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(smem_u32(bar))
      : "memory");
}

// Byte offset inside a 1024-byte-aligned shared-memory tile written by a TMA box with
// CU_TENSOR_MAP_SWIZZLE_128B: 16-byte chunk index (address bits 4..6) is XORed with the
// 128-byte line index (bits 7..9).
__device__ __forceinline__ uint32_t swz128(uint32_t off) { return off ^ (((off >> 7) & 7u) << 4); }

// ---------------------------------------------------------------- tensor-core wrappers
// One logical m16n8k8 product C += A * B on the fragment layout shared by the f64 and
// tf32 shapes (g = lane / 4, t = lane % 4):
//   a0:(g, t) a1:(g+8, t) a2:(g, t+4) a3:(g+8, t+4);  b0:(k=t, n=g) b1:(k=t+4, n=g);
//   c0:(g, 2t) c1:(g, 2t+1) c2:(g+8, 2t) c3:(g+8, 2t+1).

__device__ __forceinline__ void mma16x8x8(double (&c)[4], const double (&a)[4], const double (&b)[2]) {
  asm volatile(
      "mma.sync.aligned.m16n8k8.row.col.f64.f64.f64.f64 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+d"(c[0]), "+d"(c[1]), "+d"(c[2]), "+d"(c[3])
      : "d"(a[0]), "d"(a[1]), "d"(a[2]), "d"(a[3]), "d"(b[0]), "d"(b[1]));
}

__device__ __forceinline__ uint32_t to_tf32(float x) {
  uint32_t r;
  asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
  return r;
}
__device__ __forceinline__ void mma_tf32(float (&c)[4], const uint32_t (&a)[4], const uint32_t (&b)[2]) {
  asm volatile(
      "mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}
// fp32 product by the 3xTF32 split: x = hi + lo with hi = tf32(x), lo = tf32(x - hi);
// D = A_lo*B_hi + A_hi*B_lo + A_hi*B_hi (small terms first; A_lo*B_lo is below fp32 round-off),
// then C += D with an ordinary round-to-nearest add: the tensor core's own accumulation does not
// round to nearest, so only the eight products of one k-step are summed inside it.
__device__ __forceinline__ void mma16x8x8(float (&c)[4], const float (&a)[4], const float (&b)[2]) {
  uint32_t ah[4], al[4], bh[2], bl[2];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    ah[i] = to_tf32(a[i]);
    al[i] = to_tf32(a[i] - __uint_as_float(ah[i]));
  }
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    bh[i] = to_tf32(b[i]);
    bl[i] = to_tf32(b[i] - __uint_as_float(bh[i]));
  }
  float d[4] = {0.f, 0.f, 0.f, 0.f};
  mma_tf32(d, al, bh);
  mma_tf32(d, ah, bl);
  mma_tf32(d, ah, bh);
#pragma unroll
  for (int i = 0; i < 4; ++i) c[i] += d[i];
}

// Operands prepared once and used by several products.  In double precision an operand is the value; in single
// precision it is the value split into two TF32 numbers, so that a fragment that feeds several m16n8k8 products
// is split once and not once per product.
template <typename T>
struct Op;
template <>
struct Op<double> {
  double v;
};
template <>
struct Op<float> {
  uint32_t hi, lo;
};
__device__ __forceinline__ Op<double> prep(double x) { return Op<double>{x}; }
__device__ __forceinline__ Op<float> prep(float x) {
  Op<float> o;
  o.hi = to_tf32(x);
  o.lo = to_tf32(x - __uint_as_float(o.hi));
  return o;
}
__device__ __forceinline__ void mma_op(double (&c)[4], const Op<double>& a0, const Op<double>& a1, const Op<double>& a2,
                                       const Op<double>& a3, const Op<double>& b0, const Op<double>& b1) {
  const double a[4] = {a0.v, a1.v, a2.v, a3.v}, b[2] = {b0.v, b1.v};
  mma16x8x8(c, a, b);
}
// D = A_lo*B_hi + A_hi*B_lo + A_hi*B_hi inside the tensor core, then C += D rounded to nearest (see above)
__device__ __forceinline__ void mma_op(float (&c)[4], const Op<float>& a0, const Op<float>& a1, const Op<float>& a2,
                                       const Op<float>& a3, const Op<float>& b0, const Op<float>& b1) {
  const uint32_t ah[4] = {a0.hi, a1.hi, a2.hi, a3.hi}, al[4] = {a0.lo, a1.lo, a2.lo, a3.lo};
  const uint32_t bh[2] = {b0.hi, b1.hi}, bl[2] = {b0.lo, b1.lo};
  float d[4] = {0.f, 0.f, 0.f, 0.f};
  mma_tf32(d, al, bh);
  mma_tf32(d, ah, bl);
  mma_tf32(d, ah, bh);
#pragma unroll
  for (int i = 0; i < 4; ++i) c[i] += d[i];
}

// ---------------------------------------------------------------- small utilities

template <typename T>
struct VecLoad16;  // one 16-byte shared-memory load
template <>
struct VecLoad16<double> {
  static constexpr int N = 2;
  __device__ static __forceinline__ void ld(const unsigned char* p, double (&v)[2]) {
    const double2 x = *reinterpret_cast<const double2*>(p);
    v[0] = x.x;
    v[1] = x.y;
  }
};
template <>
struct VecLoad16<float> {
  static constexpr int N = 4;
  __device__ static __forceinline__ void ld(const unsigned char* p, float (&v)[4]) {
    const float4 x = *reinterpret_cast<const float4*>(p);
    v[0] = x.x;
    v[1] = x.y;
    v[2] = x.z;
    v[3] = x.w;
  }
};

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Fixed-order block reduction of one double per thread (blockDim.x a multiple of 32, <= 1024).
// `scratch` holds at least 32 doubles.  The result is valid in thread 0.
__device__ __forceinline__ double block_sum(double v, double* scratch) {
  v = warp_sum(v);
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  __syncthreads();
  if (lane == 0) scratch[wid] = v;
  __syncthreads();
  double r = 0.0;
  if (wid == 0) {
    const int nw = (blockDim.x + 31) >> 5;
    r = lane < nw ? scratch[lane] : 0.0;
    r = warp_sum(r);
  }
  return r;
}

}  // namespace rrf
