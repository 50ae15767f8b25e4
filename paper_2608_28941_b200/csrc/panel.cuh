// Panel Householder QR (Algorithm 2 line 7, geqrt semantics) on the GPU, plus the small
// kernels around it: compact-WY T factor, Z <- op(T) Z, norms, stop rule, Gaussian fill.
#pragma once

#include "common.cuh"

namespace rrf {

constexpr int kPanelThreads = 512;
constexpr int kPanelMaxG = 160;   // most CTAs a panel grid may have (one per SM)
// doubles of shared memory the panel kernel needs besides the slab: w[b], p[2][b], pivot_row[b], scalars
__host__ __device__ constexpr int panel_extra_doubles(int b) { return 4 * b + 4; }

// Grid-wide barrier over a monotonically increasing arrival counter.  Needs all CTAs
// co-resident (cooperative launch).  Bounded: gives up after kWaitLimitClocks.
__device__ __forceinline__ bool grid_barrier(unsigned* ctr, unsigned target, Ctrl* ctrl,
                                             long long limit = kWaitLimitClocks) {
  __shared__ int ok_s;
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    atomicAdd(ctr, 1u);
    int ok = 1;
    const long long t0 = clock64();
    while (true) {
      unsigned v;
      asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(ctr) : "memory");
      if (v >= target) break;
      if (clock64() - t0 > limit) {
        atomicExch(&ctrl->status, (int)RRF_ERR_TIMEOUT);
        atomicExch(&ctrl->done, 1);        // kernels already enqueued behind this one return at once
        ok = 0;
        break;
      }
    }
    ok_s = ok;
  }
  __syncthreads();
  return ok_s != 0;
}

// ---------------------------------------------------------------- thread-block cluster exchange
// A panel that fits the shared memory of at most 16 CTAs is factored by ONE cluster: the per-column sums
// travel through distributed shared memory (every CTA writes its partials straight into every peer's
// shared memory) and the barrier is an mbarrier per CTA on which every peer arrives - about 0.7 to 1 us per
// column against the 2.4 us of an all-to-all exchange through L2.
constexpr int kClusterMax = 16;
#ifdef RRF_TSQR_TRACE
__device__ unsigned long long g_pcl_trace[16];
#define PCL_STAMP(k) if (j == 8 && blockIdx.x == 0 && threadIdx.x == 0) g_pcl_trace[k] = (unsigned long long)clock64()
#else
#define PCL_STAMP(k)
#endif
constexpr int kRegRows = 256;       // rows of a slab in the register-resident column loop
// px [2][kClusterMax][2b], prx [2][b], ycol/vcol [kRegRows] each, prow [b], send buffers [2][2b]
__host__ __device__ constexpr int panel_cluster_doubles(int b) {
  return 2 * kClusterMax * 2 * b + 2 * b + 2 * kRegRows + b + 4 * b;
}
// One bulk copy from this CTA's shared memory into a peer's, which also counts its bytes on the peer's mbarrier:
// data and signal in one message.
__device__ __forceinline__ void cl_bulk_send(uint32_t dst_cluster, uint32_t src_cta, uint32_t bytes, uint32_t bar_cluster) {
  asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst_cluster), "r"(src_cta), "r"(bytes), "r"(bar_cluster)
               : "memory");
}

__device__ __forceinline__ void proxy_fence_smem_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ uint32_t cl_map(uint32_t addr, uint32_t rank) {   // the same address in CTA `rank` of the cluster
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cl_st(uint32_t addr, double v) {
  asm volatile("st.shared::cluster.f64 [%0], %1;" ::"r"(addr), "d"(v) : "memory");
}
__device__ __forceinline__ void cl_st(uint32_t addr, int v) {
  asm volatile("st.shared::cluster.b32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ void cl_arrive(uint32_t bar_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar_addr) : "memory");
}
__device__ __forceinline__ uint32_t cl_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok;
}
// the hardware barrier of the cluster (unbounded: used once, before any data-dependent exit)
__device__ __forceinline__ void cl_hw_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Barrier over the G CTAs of the cluster: every CTA arrives on every peer's mbarrier and waits, bounded, on its
// own.  Everything this CTA stored before it - into peers' shared memory, or (with `global_too`) into global
// memory - is visible to the peers behind it.  `nx` counts the barriers passed (the phase parity).
__device__ __forceinline__ bool cluster_barrier(uint64_t* cbar, unsigned& nx, int G, bool global_too, Ctrl* ctrl) {
  __shared__ int cl_ok_s;
  __syncthreads();
  if ((int)threadIdx.x < G) {
    if (global_too) __threadfence();
    cl_arrive(cl_map(smem_u32(cbar), threadIdx.x));
  }
  if (threadIdx.x == 0) {
    int ok = 1;
    if (!cl_try_wait(cbar, nx & 1u)) {
      const long long t0 = clock64();
      while (!cl_try_wait(cbar, nx & 1u)) {
        if (clock64() - t0 > kWaitLimitClocks) {
          atomicExch(&ctrl->status, (int)RRF_ERR_TIMEOUT);
          atomicExch(&ctrl->done, 1);
          ok = 0;
          break;
        }
      }
    }
    cl_ok_s = ok;
  }
  ++nx;
  __syncthreads();
  return cl_ok_s != 0;
}

// Sums four per-lane values over the warp with 6 adds and 6 shuffles instead of 20: after the
// exchanges with lanes ^16 and ^8 every lane carries one of the four sums (number 2*bit4 + bit3 of
// its lane index), which three more butterfly steps complete.  Fixed order, so reproducible.
__device__ __forceinline__ double warp_sum4(const double (&v)[4], int lane) {
  const bool hi = lane & 16;
  double a0 = hi ? v[2] : v[0], a1 = hi ? v[3] : v[1];
  const double s0 = hi ? v[0] : v[2], s1 = hi ? v[1] : v[3];
  a0 += __shfl_xor_sync(0xffffffffu, s0, 16);
  a1 += __shfl_xor_sync(0xffffffffu, s1, 16);
  const bool mid = lane & 8;
  double k = mid ? a1 : a0;
  const double snd = mid ? a0 : a1;
  k += __shfl_xor_sync(0xffffffffu, snd, 8);
  k += __shfl_xor_sync(0xffffffffu, k, 4);
  k += __shfl_xor_sync(0xffffffffu, k, 2);
  k += __shfl_xor_sync(0xffffffffu, k, 1);
  return k;
}

// Self test of the bounded wait: one CTA arrives at a barrier that expects two.
__global__ void __launch_bounds__(32) timeout_selftest_kernel(unsigned* ctr, Ctrl* ctrl, long long limit) {
  grid_barrier(ctr, 2u, ctrl, limit);
}

// ------------------------------------------------------------------------------------------
// Householder QR of a rows x b panel.  Each CTA keeps a slab of R consecutive rows in shared
// memory (column-major, double precision, pitch Rp odd) for the whole factorisation.  Column j
// costs one pass over the slab and ONE grid barrier: the pass applies the pending reflector
// H_{j-1} and accumulates p[c] = sum_{row > j} Y[row, j] * X[row, c] for every column c, where
// X[:, c] is the finished vector v_c for c < j and the current Y[:, c] for c >= j.  After the
// barrier every CTA sums the per-CTA partials in CTA order and derives, with alpha = Y[j, j]:
//   beta = -sign(alpha) sqrt(alpha^2 + p[j]),  tau = (beta - alpha)/beta,  v = Y[j+1:, j] * (1/(alpha - beta))
//   w[c] = v^T Y[:, c]   = Y[j, c] + p[c]/(alpha - beta)           (c > j: needed by H_j)
//   g[c] = v_c^T v_j     = v_c[j] + p[c]/(alpha - beta)           (c < j: row j of V^T V, for T)
// so norms, reflector application and the Gram matrix for T share one reduction.
// ------------------------------------------------------------------------------------------
// Where the panel's entries come from: either `nseg` partial panels stacked with a fixed
// stride (rows x ldy each), or the slot layout written by upd_sk_kernel (gemm_sk.cuh).
struct PanelSource {
  int slots;               // 0: stacked segments, 1: stream-K slots
  int nseg;                // stacked: number of partial panels
  long long seg_stride;    // stacked: elements between partial panels
  int ldy;                 // stacked: leading dimension
  int row_off;             // panel row 0 is row `row_off` of the producer's row numbering
  int bm, nc, tpc, wn;     // slots: slab height, tiles per slab, tiles per CTA, warp columns
  int t1, p1, tpc2;        // slots: tiles from t1 on belong to CTAs p1, p1 + 1, ... at tpc2 tiles each (t1 <= 0: none)
};
// CTA (= slot) that computed tile L of a pass
__device__ __forceinline__ int slot_cta(const PanelSource& src, int L) {
  return (src.t1 > 0 && L >= src.t1) ? src.p1 + (L - src.t1) / src.tpc2 : L / src.tpc;
}

// Look-ahead schedule (Section "Implementation", the two-queue variant): the panel was sampled from
// the matrix BEFORE the previous block's reflectors were applied, P = W_old * Omega, so the kernel
// first applies them to the panel itself, Y = (P - Vp (Tp^T (Vp^T P)))[b:, :], where Vp is the previous
// (rows + b) x b block of Householder vectors and Tp its triangular factor.
struct PanelFix {
  int enabled;
  const void* Vp;          // previous V block, element type T, row 0 = b rows above the panel's row 0
  long long ldvp;
  const void* Tp;          // previous T block (b x b, upper triangular), element type T
  long long ldtp;
  double* Gpart;           // [gridDim.x][b*b] per-CTA partial Vp^T P
  double* M;               // [b*b] Tp^T (Vp^T P)
};
constexpr int kFixChunk = 32;   // rows of Vp staged in shared memory at a time
// doubles of shared memory the fix-up needs on top of panel_extra_doubles: the staged rows of Vp
// (pitch b + 8 or b + 4) and a b x (b + 8) matrix (Tp, then M)
__host__ __device__ constexpr int panel_fix_doubles(int b) { return kFixChunk * (b + 8) + b * (b + 8); }

template <typename T>
__device__ __forceinline__ double panel_entry(const T* __restrict__ Y, const PanelSource& src, int r, int c, int b) {
  double s = 0.0;
  if (!src.slots) {
    const T* p = Y + (size_t)(r + src.row_off) * src.ldy + c;
    s = (double)p[0];                     // not 0.0 + p[0]: a lone -0.0 keeps its sign (it decides a reflector's)
    for (int sg = 1; sg < src.nseg; ++sg) s += (double)p[(size_t)sg * src.seg_stride];
  } else {
    const int lr = r + src.row_off;
    const int sl = lr / src.bm, rl = lr - sl * src.bm;
    const int p_lo = slot_cta(src, sl * src.nc), p_hi = slot_cta(src, (sl + 1) * src.nc - 1);
    for (int p = p_lo; p <= p_hi; ++p)
      for (int w = 0; w < src.wn; ++w)
        s += (double)Y[((size_t)(p + sl) * src.wn + w) * (size_t)(src.bm * b) + (size_t)rl * b + c];
  }
  return s;
}

// The same sums for a whole slab, S[c][r] (pitch Rp) = entry (gr0 + r - row0, c), with the loads of eight entries
// in flight per thread: the terms of one entry are a dependent chain of global loads (up to a dozen partial
// panels), and a CTA that holds a tall slab has dozens of entries per thread.  Same order of additions as
// panel_entry, so the same bits.
template <typename T>
__device__ __forceinline__ void panel_load_slab(const T* __restrict__ Y, const PanelSource& src, double* __restrict__ S, int Rp,
                                                int nloc, int b, int lb, int gr0, int row0, int tid, int nthr) {
  constexpr int E = 8;
  const int total = nloc * b;
  const size_t tstride = src.slots ? (size_t)src.bm * b : (size_t)src.seg_stride;
  for (int base = tid; base < total; base += E * nthr) {
    const T* ptr[E];
    int cnt[E];
    double v[E];
    int maxcnt = 0;
#pragma unroll
    for (int e = 0; e < E; ++e) {
      const int idx = base + e * nthr;
      const int r = idx >> lb, c = idx & (b - 1);
      cnt[e] = 0;
      ptr[e] = Y;
      if (idx < total) {
        const int lr = gr0 + r - row0 + src.row_off;
        if (src.slots) {
          const int sl = lr / src.bm, rl = lr - sl * src.bm;
          const int p_lo = slot_cta(src, sl * src.nc), p_hi = slot_cta(src, (sl + 1) * src.nc - 1);
          cnt[e] = (p_hi - p_lo + 1) * src.wn;
          ptr[e] = Y + (size_t)(p_lo + sl) * src.wn * tstride + (size_t)rl * b + c;
        } else {
          cnt[e] = src.nseg;
          ptr[e] = Y + (size_t)lr * src.ldy + c;
        }
      }
      maxcnt = max(maxcnt, cnt[e]);
    }
#pragma unroll
    for (int e = 0; e < E; ++e) {
      const double first = cnt[e] > 0 ? (double)ptr[e][0] : 0.0;
      v[e] = src.slots ? 0.0 + first : first;      // as panel_entry: a lone -0.0 of a stacked panel keeps its sign
    }
    for (int t = 1; t < maxcnt; ++t) {
#pragma unroll
      for (int e = 0; e < E; ++e)
        if (t < cnt[e]) v[e] += (double)ptr[e][(size_t)t * tstride];
    }
#pragma unroll
    for (int e = 0; e < E; ++e) {
      const int idx = base + e * nthr;
      if (idx < total) S[(size_t)(idx & (b - 1)) * Rp + (idx >> lb)] = v[e];
    }
  }
}

// Compact-WY factor T from the Gram rows and tau, by recursive doubling (see tfactor_kernel below).
// The block-level body: every thread of one CTA calls it; `tsm` holds b*(b+1) + (b/2)*(b/2+1) doubles.
template <typename T>
__device__ __forceinline__ void tfactor_block(const double* __restrict__ gram, const double* __restrict__ tau, int b,
                                              T* __restrict__ Tout, long long ldt, double* tsm) {
  const int pitch = b + 1, mp = b / 2 + 1;
  double* Ts = tsm;                        // [b][pitch]: T above and on the diagonal, Gram rows below
  double* Ms = Ts + (size_t)b * pitch;     // [b/2][mp]: (V1^T V2) T22 of every pair of the current round
  const int tid = threadIdx.x;
  const int nthr = blockDim.x;
  // stage the Gram rows (strictly lower triangle) and tau: eight independent loads in flight per thread
  for (int base = 0; base < b * b; base += nthr * 8) {
    double v[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const int idx = base + e * nthr + tid;
      const int r = idx / b, c = idx - r * b;
      v[e] = (idx < b * b && c < r) ? __ldcg(gram + idx) : 0.0;
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const int idx = base + e * nthr + tid;
      const int r = idx / b, c = idx - r * b;
      if (idx < b * b) Ts[r * pitch + c] = v[e];
    }
  }
  __syncthreads();
  if (tid < b) Ts[tid * pitch + tid] = __ldcg(tau + tid);
  __syncthreads();
  for (int s = 1; s < b; s <<= 1) {
    const int per_level = b * s / 2;       // (b / 2s) pairs x s x s entries
    const int ls = 31 - __clz(s);          // s is a power of two
    for (int idx = tid; idx < per_level; idx += nthr) {
      const int q = idx >> (2 * ls), rc = idx & (s * s - 1), r = rc >> ls, c = rc & (s - 1);
      const int o = 2 * s * q;
      // M[r][c] = sum_{k <= c} (v_{o+r}^T v_{o+s+k}) T22[k][c]; two independent partial sums
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
      // T12[r][c] = -sum_{k >= r} T11[r][k] M[k][c]
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
  for (int idx = tid; idx < b * b; idx += nthr) {
    const int r = idx / b, c = idx - r * b;
    Tout[(size_t)r * ldt + c] = c >= r ? (T)Ts[r * pitch + c] : T(0);
  }
}


// The 16 warps of a CTA form RH row groups of 16/RH warps; a lane looks after QMAX rows of its
// group (kept in registers during a pass), so a slab holds up to 32 * QMAX * RH rows.  With PAD the
// slab is allocated at that full height and zero filled below its last row, which removes every
// per-element bounds test from the pass; PAD = false keeps the tests (for the one shape whose slab only
// fits unpadded).
// CL: the grid is one thread-block cluster of at most kClusterMax CTAs; sums and pivot rows are exchanged through
// distributed shared memory and the barriers are cluster_barrier (P, piv and the barrier counter are not used).
// REG (with CL, b <= 64, slabs of at most 256 rows): during the column loop the slab lives in REGISTERS - lane l of
// warp w keeps rows l, l + 32, ..., l + 224 of columns 4w ... 4w + 3 - so a column costs each thread 32 fused
// multiply-adds and a warp reduction instead of a pass over the slab in shared memory (which is what makes a slab
// of 256 rows, i.e. a 4096-row panel on 16 CTAs, worth its while).  Column j and the finished v_{j-1} go round
// through two 256-element arrays in shared memory.
template <typename T, int QMAX, int RH, bool PAD = true, bool CL = false, bool REG = false>
__global__ void __launch_bounds__(kPanelThreads)
    panel_kernel(const T* __restrict__ Y, PanelSource src_fused, PanelSource src_alt, const int* __restrict__ fused_flag,
                 int rows, int b, int R, int Rp,
                 T* __restrict__ V, long long ldv,   // rows x b block of the V array
                 double* __restrict__ P,             // [2][b][Gp] per-CTA partial dots, Gp = gridDim.x rounded up to 32
                 double* __restrict__ piv,           // [2][b] broadcast pivot row
                 double* __restrict__ gram,          // [b][b] strictly-lower part: v_c^T v_j (c < j)
                 double* __restrict__ tau_out,       // [b]
                 unsigned* bar, Ctrl* ctrl, const int* done_flag, PanelFix fix,
                 unsigned bar_base,                 // value of the barrier counter when this launch starts
                 T* __restrict__ Tout, long long ldt,     // non-NULL: CTA 0 also builds the T factor at the end
                 double* __restrict__ csq) {              // non-NULL: [b][Gp] per-CTA sums of squares of the panel's columns
  __shared__ uint64_t cbar;      // cluster mode: this CTA's barrier, on which every CTA of the cluster arrives
  __shared__ uint64_t xbar[2];   // ... and the two on which the per-column messages of the peers are counted
  __shared__ int go_s;
  unsigned nx = 0;               // cluster barriers passed
  if (CL) {
    // The decision to run must be the same in every CTA of the cluster (a CTA that left would never arrive at
    // its peers' barriers): rank 0 reads the flags and tells everyone, under the hardware barrier of the cluster.
    if (threadIdx.x == 0) {
      mbar_init(&cbar, gridDim.x);
      mbar_init(&xbar[0], 1);
      mbar_init(&xbar[1], 1);
      mbar_fence_init();
    }
    cl_hw_sync();                // every CTA of the cluster runs and has its barrier initialised
    if (blockIdx.x == 0 && threadIdx.x < gridDim.x) {
      const int go = !(*reinterpret_cast<const volatile int*>(done_flag) ||
                       *reinterpret_cast<const volatile int*>(&ctrl->status) < 0);
      cl_st(cl_map(smem_u32(&go_s), threadIdx.x), go);
    }
    cl_hw_sync();
    if (!go_s) return;
  } else {
    if (*reinterpret_cast<const volatile int*>(done_flag) || *reinterpret_cast<const volatile int*>(&ctrl->status) < 0) return;
  }
  // the panel's entries were sampled by the fused update, or - where the predictor had skipped that - by
  // the separate sample kernel, in its layout
  const bool use_alt = fused_flag != nullptr && *fused_flag == 0;
  const PanelSource src = use_alt ? src_alt : src_fused;   // a copy in registers, not a pointer into the parameters
  extern __shared__ double psm[];
  double* S = psm;                        // [b][Rp]
  double* w_s = S + (size_t)b * Rp;       // [b]
  double* p_s = w_s + b;                  // [2][b]: per row group, then (first b) the grid-wide sums
  double* pr_s = p_s + 2 * b;             // [b]
  double* sc_s = pr_s + b;                // [4]: tau_j, 1/(alpha - beta)
  // cluster mode: partial sums [2][kClusterMax][b] and pivot rows [2][b] written by the peers, behind everything else
  double* px_s = sc_s + 4 + (fix.enabled ? panel_fix_doubles(b) : 0);
  double* prx_s = px_s + 2 * kClusterMax * 2 * b;
  double* ycol_s = prx_s + 2 * b;         // [kRegRows] column j below its pivot (register-resident loop)
  double* vcol_s = ycol_s + kRegRows;     // [kRegRows] v_{j-1}
  double* prow_s = vcol_s + kRegRows;     // [b] this CTA's entries of the pivot row
  double* snd_s = prow_s + b;             // [2][2b] what this CTA sends per column: its partial sums, its pivot-row entries

  constexpr int NT = kPanelThreads, NW = NT / 32;
  constexpr int NWC = NW / RH;            // warps that share the columns within one row group
  constexpr int CG = 4;                   // columns a warp handles at a time (independent chains)
  constexpr int RS = 32 * QMAX * RH;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int rg = warp / NWC, wc = warp - rg * NWC;
  const int G = gridDim.x, cta = blockIdx.x;
  const int Gp = (G + 31) & ~31;
  // Slab rows are numbered from the first row this kernel touches: with the fix-up that is b rows
  // above the panel (the rows of P that only enter Vp^T P), so the panel starts at slab row `row0`.
  const int row0 = fix.enabled ? b : 0;
  const int ext = rows + row0;
  const int gr0 = cta * R;
  const int nloc = max(0, min(R, ext - gr0));
  const int lb = 31 - __clz(b);           // b is a power of two
  unsigned nbar = 0;                      // grid barriers passed so far

  // load the slab: sum the partial panels in their fixed order
  panel_load_slab<T>(Y, src, S, Rp, nloc, b, lb, gr0, row0, tid, NT);
  if (PAD) {
    const int npad = RS - nloc;
    for (int idx = tid; idx < npad * b; idx += NT) {
      const int c = idx / npad, r = nloc + (idx - c * npad);
      S[(size_t)c * Rp + r] = 0.0;
    }
  }
  __syncthreads();

  if (fix.enabled) {
    // ---- S <- P - Vp (Tp^T (Vp^T P)) on the tensor cores (FP64 m16n8k8)
    const int g = lane >> 2, t = lane & 3;
    double* Vst = sc_s + 4;                              // [kFixChunk][b + 8] or [kFixChunk][b + 4]
    double* Mst = Vst + (size_t)kFixChunk * (b + 8);     // [b][b + 8]: Tp (pitch b + 1), then M
    const T* Vp = reinterpret_cast<const T*>(fix.Vp);
    const T* Tp = reinterpret_cast<const T*>(fix.Tp);
    const int nch = (nloc + kFixChunk - 1) / kFixChunk;
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
    // Tp into shared memory (pitch b + 1), zero below the diagonal
    for (int idx = tid; idx < b * b; idx += NT) {
      const int l = idx >> lb, k = idx & (b - 1);
      Mst[l * (b + 1) + k] = l <= k ? (double)Tp[(size_t)l * fix.ldtp + k] : 0.0;
    }
    // Phase 1: Gpart[cta] = Vp[slab]^T S.  Warp (mt, np) owns G[16 mt .., 16 np ..] (two n-tiles).
    {
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
    if (CL) {
      if (!cluster_barrier(&cbar, nx, G, true, ctrl)) return;
    } else if (!grid_barrier(bar, bar_base + (++nbar) * (unsigned)G, ctrl)) return;
    // Phase 2: CTA c owns columns c, c + G, ... of G = sum of the partials (in CTA order) and of
    // M = Tp^T G, column by column: M[k][c2] = sum_{l <= k} Tp[l][k] G[l][c2].
    {
      const int ncol = cta < b ? (b - cta + G - 1) / G : 0;
      double* Gs = Vst;                                  // up to kFixChunk columns of G at a time
      for (int q0 = 0; q0 < ncol; q0 += kFixChunk) {
        const int nq = min(kFixChunk, ncol - q0);
        __syncthreads();
        for (int idx = tid; idx < nq * b; idx += NT) {
          const int q = idx >> lb, l = idx & (b - 1), c2 = cta + (q0 + q) * G;
          const double* gp = fix.Gpart + (size_t)l * b + c2;
          double sum = 0.0;
          int x = 0;
          for (; x + 8 <= G; x += 8) {
            double v[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) v[e] = __ldcg(gp + (size_t)(x + e) * b * b);
#pragma unroll
            for (int e = 0; e < 8; ++e) sum += v[e];
          }
          for (; x < G; ++x) sum += __ldcg(gp + (size_t)x * b * b);
          Gs[q * b + l] = sum;
        }
        __syncthreads();
        for (int idx = tid; idx < nq * b; idx += NT) {
          const int q = idx >> lb, k = idx & (b - 1), c2 = cta + (q0 + q) * G;
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
    if (CL) {
      if (!cluster_barrier(&cbar, nx, G, true, ctrl)) return;
    } else if (!grid_barrier(bar, bar_base + (++nbar) * (unsigned)G, ctrl)) return;
    // Phase 3: S -= Vp[slab] M.  A task is a 16-row x 8-column tile of a chunk.
    {
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
    }
    __syncthreads();
  }

  // Sums of squares of the columns of the panel as sampled (after the fix-up): the sampled stopping rules
  // estimate the residual from them (est_kernel).  One warp per column, fixed order.
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

  double tau_prev = 0.0;
  if constexpr (CL && REG) {
    static_assert(QMAX == 8 && RH == 1 && PAD, "the register tile is 8 rows x 4 columns per thread");
    const bool has = warp < (b >> 2);                  // warps that hold columns
    const int c0 = warp * 4;
    double x[8][4];
#pragma unroll
    for (int q = 0; q < 8; ++q)
#pragma unroll
      for (int u = 0; u < 4; ++u) x[q][u] = has ? S[(size_t)(c0 + u) * Rp + lane + 32 * q] : 0.0;
    for (int j = 0; j < b; ++j) {
      const int pr = row0 + j;
      const int ow = j >> 2, uj = j & 3;               // warp and tile column that hold column j
      PCL_STAMP(0);
      // pending reflector H_{j-1} on this thread's columns j and later (v_{j-1} is zero above its pivot)
      if (has && j > 0 && tau_prev != 0.0 && c0 + 3 >= j) {
        double v[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) v[q] = vcol_s[lane + 32 * q];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          if (c0 + u >= j) {
            const double f = tau_prev * w_s[c0 + u];
#pragma unroll
            for (int q = 0; q < 8; ++q) x[q][u] -= f * v[q];
          }
        }
      }
      // column j below its pivot, and this CTA's entries of the pivot row, for everyone
      if (warp == ow) {
#pragma unroll
        for (int q = 0; q < 8; ++q) {
          const int r = lane + 32 * q;
          double yv = 0.0;
#pragma unroll
          for (int u = 0; u < 4; ++u) yv = (u == uj) ? x[q][u] : yv;
          ycol_s[r] = (gr0 + r > pr) ? yv : 0.0;
        }
      }
      if (has && pr >= gr0 && pr < gr0 + nloc && ((pr - gr0) & 31) == lane) {
        const int qp = (pr - gr0) >> 5;
#pragma unroll
        for (int q = 0; q < 8; ++q)
          if (q == qp) {
#pragma unroll
            for (int u = 0; u < 4; ++u) prow_s[c0 + u] = x[q][u];
          }
      }
      __syncthreads();
      PCL_STAMP(1);
      if (has) {
        double y[8], acc[4] = {0.0, 0.0, 0.0, 0.0};
#pragma unroll
        for (int q = 0; q < 8; ++q) y[q] = ycol_s[lane + 32 * q];
#pragma unroll
        for (int q = 0; q < 8; ++q)
#pragma unroll
          for (int u = 0; u < 4; ++u) acc[u] += y[q] * x[q][u];
        const double tot = warp_sum4(acc, lane);
        const int u = ((lane >> 4) << 1) | ((lane >> 3) & 1);
        if ((lane & 7) == 0) p_s[c0 + u] = tot;
      }
      __syncthreads();
      PCL_STAMP(2);
      {
        // One message per peer: this CTA's b partial sums and its entries of the pivot row (zeros unless it holds
        // that row), 16 b bytes, copied into the peer's shared memory by cp.async.bulk, which also counts the bytes
        // on the peer's barrier.  Two buffers and two barriers alternate: a peer is at most one column ahead.
        const int pb = j & 1;
        double* snd = snd_s + pb * 2 * b;
        const bool mine = pr >= gr0 && pr < gr0 + nloc;
        if (tid < b) {
          snd[tid] = p_s[tid];
          snd[b + tid] = mine ? prow_s[tid] : 0.0;
        }
        proxy_fence_smem_async();
        __syncthreads();
        const uint32_t bytes = 2u * (uint32_t)b * 8u;
        if (tid == 0) mbar_expect_tx(&xbar[pb], (uint32_t)G * bytes);
        if (tid < G)
          cl_bulk_send(cl_map(smem_u32(px_s + ((size_t)pb * kClusterMax + cta) * 2 * b), tid), smem_u32(snd), bytes,
                       cl_map(smem_u32(&xbar[pb]), tid));
        PCL_STAMP(3);
        if (tid == 0) {
          int ok = 1;
          const uint32_t par = (uint32_t)(j >> 1) & 1u;
          if (!cl_try_wait(&xbar[pb], par)) {
            const long long t0 = clock64();
            while (!cl_try_wait(&xbar[pb], par)) {
              if (clock64() - t0 > kWaitLimitClocks) {
                atomicExch(&ctrl->status, (int)RRF_ERR_TIMEOUT);
                atomicExch(&ctrl->done, 1);
                ok = 0;
                break;
              }
            }
          }
          go_s = ok;
        }
        __syncthreads();
        if (!go_s) return;
        PCL_STAMP(4);
        if (tid < b) {
          // four interleaved partial sums (CTAs q = 0, 4, 8, 12; 1, 5, ...; ...), then their sum: a fixed order
          double v4[4] = {0.0, 0.0, 0.0, 0.0};
          for (int q = 0; q < G; q += 4) {
#pragma unroll
            for (int e = 0; e < 4; ++e)
              if (q + e < G) v4[e] += px_s[((size_t)pb * kClusterMax + q + e) * 2 * b + tid];
          }
          p_s[tid] = (v4[0] + v4[1]) + (v4[2] + v4[3]);
          pr_s[tid] = px_s[((size_t)pb * kClusterMax + pr / R) * 2 * b + b + tid];   // from the CTA that holds row pr
        }
        __syncthreads();
      }
      PCL_STAMP(5);
      if (warp == 0) {
        const double alpha = pr_s[j], s2 = p_s[j];
        double tau = 0.0, rdenom = 0.0;
        if (s2 != 0.0) {
          const double beta = -copysign(sqrt(alpha * alpha + s2), alpha);
          tau = (beta - alpha) / beta;
          rdenom = 1.0 / (alpha - beta);
        }
        if (lane == 0) {
          sc_s[0] = tau;
          sc_s[1] = rdenom;
          if (cta == 0) tau_out[j] = tau;
        }
      }
      __syncthreads();
      PCL_STAMP(6);
      const double tau = sc_s[0], rdenom = sc_s[1];     // rdenom == 0 marks H_j = I
      if (tid < b && tid != j) {
        const double wv = pr_s[tid] + p_s[tid] * rdenom;
        w_s[tid] = wv;
        if (cta == 0 && tid < j) gram[(size_t)j * b + tid] = wv;
      }
      // column j becomes v_j (unit lower trapezoidal, explicit ones and zeros), and goes round as v_{j-1}
      if (warp == ow) {
#pragma unroll
        for (int q = 0; q < 8; ++q) {
          const int r = lane + 32 * q, grow = gr0 + r;
          double xv = 0.0;
#pragma unroll
          for (int u = 0; u < 4; ++u) xv = (u == uj) ? x[q][u] : xv;
          const double vv = grow > pr ? xv * rdenom : ((grow == pr && r < nloc) ? 1.0 : 0.0);
#pragma unroll
          for (int u = 0; u < 4; ++u) x[q][u] = (u == uj) ? vv : x[q][u];
          vcol_s[r] = vv;
        }
      }
      tau_prev = tau;
      __syncthreads();
      PCL_STAMP(7);
    }
    if (has) {
#pragma unroll
      for (int q = 0; q < 8; ++q)
#pragma unroll
        for (int u = 0; u < 4; ++u) S[(size_t)(c0 + u) * Rp + lane + 32 * q] = x[q][u];
    }
    __syncthreads();
  } else
  for (int j = 0; j < b; ++j) {
    const int pr = row0 + j;                           // slab-numbering row of the pivot
    double* Sj = S + (size_t)j * Rp;
    const double* Sjm1 = S + (size_t)(j > 0 ? j - 1 : 0) * Rp;
    // finish column j: pending reflector H_{j-1}
    if (j > 0 && tau_prev != 0.0) {
      const double f = tau_prev * w_s[j];
      for (int r = tid; r < nloc; r += NT)
        if (gr0 + r >= pr) Sj[r] -= f * Sjm1[r];
    }
    __syncthreads();
    // one pass: update trailing columns and take all dot products with column j.  Each lane keeps
    // its rows of column j and of v_{j-1} in registers, masked once per column: rows at or above the
    // pivot do not count in the dot products, and rows the pending reflector must not change see
    // v_{j-1} = 0, so the inner loop needs no tests.  CG columns are in flight per warp.
    {
      double yj[QMAX], vp[QMAX];
      const int rbase = rg * (32 * QMAX) + lane;
#pragma unroll
      for (int q = 0; q < QMAX; ++q) {
        const int r = rbase + 32 * q;
        const bool in = PAD || r < nloc;
        const int grow = gr0 + r;
        yj[q] = (in && grow > pr) ? Sj[r] : 0.0;
        vp[q] = (in && grow >= pr) ? Sjm1[r] : 0.0;
      }
      const bool pending = (j > 0) && (tau_prev != 0.0);
      for (int c0 = wc; c0 < b; c0 += NWC * CG) {
        double x[CG][QMAX], acc[CG];
#pragma unroll
        for (int u = 0; u < CG; ++u) {
          const int c = c0 + u * NWC;
          const double* Sc = S + (size_t)(c < b ? c : 0) * Rp + rbase;
#pragma unroll
          for (int q = 0; q < QMAX; ++q) x[u][q] = (PAD || rbase + 32 * q < nloc) ? Sc[32 * q] : 0.0;
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
              if (PAD || rbase + 32 * q < nloc) Sc[32 * q] = xv;
              a += yj[q] * xv;
            }
          } else {
#pragma unroll
            for (int q = 0; q < QMAX; ++q) a += yj[q] * x[u][q];
          }
          acc[u] = c < b ? a : 0.0;
        }
        {
          const double tot = warp_sum4(acc, lane);
          const int u = ((lane >> 4) << 1) | ((lane >> 3) & 1);
          if ((lane & 7) == 0 && c0 + u * NWC < b) p_s[rg * b + c0 + u * NWC] = tot;
        }
      }
    }
    __syncthreads();
    if (CL) {
      // this CTA's b partial sums, and from the CTA that holds it the pivot row, into every peer's shared memory
      // (two buffers: a peer may be one column ahead, never two)
      const int pb = j & 1;
      for (int idx = tid; idx < G * b; idx += NT) {
        const int q = idx >> lb, c = idx & (b - 1);
        double v = p_s[c];
#pragma unroll
        for (int h = 1; h < RH; ++h) v += p_s[h * b + c];
        cl_st(cl_map(smem_u32(px_s + ((size_t)pb * kClusterMax + cta) * 2 * b + c), q), v);
      }
      if (pr >= gr0 && pr < gr0 + nloc)
        for (int idx = tid; idx < G * b; idx += NT) {
          const int q = idx >> lb, c = idx & (b - 1);
          cl_st(cl_map(smem_u32(prx_s + pb * b + c), q), S[(size_t)c * Rp + (pr - gr0)]);
        }
      if (!cluster_barrier(&cbar, nx, G, false, ctrl)) return;
      if (tid < b) {
        double v = 0.0;
        for (int q = 0; q < G; ++q) v += px_s[((size_t)pb * kClusterMax + q) * 2 * b + tid];     // CTA order: reproducible
        p_s[tid] = v;
        pr_s[tid] = prx_s[pb * b + tid];
      }
      __syncthreads();
    } else {
    double* Pj = P + (size_t)(j & 1) * b * Gp;
    for (int c = tid; c < b; c += NT) {
      double v = p_s[c];
#pragma unroll
      for (int h = 1; h < RH; ++h) v += p_s[h * b + c];
      Pj[(size_t)c * Gp + cta] = v;
    }
    if (pr >= gr0 && pr < gr0 + nloc)
      for (int c = tid; c < b; c += NT) piv[(j & 1) * b + c] = S[(size_t)c * Rp + (pr - gr0)];
    if (!grid_barrier(bar, bar_base + (++nbar) * (unsigned)G, ctrl)) return;

    // every CTA: sum of the per-CTA partials in a fixed order (lane x takes CTAs x, x+32, ...;
    // then the fixed shuffle tree), one warp per column, CG columns of loads in flight at once
    {
      const double prv = tid < b ? __ldcg(piv + (j & 1) * b + tid) : 0.0;
      for (int c0 = warp; c0 < b; c0 += NW * CG) {
        double v[CG][kPanelMaxG / 32];
#pragma unroll
        for (int u = 0; u < CG; ++u) {
          const int c = c0 + u * NW;
#pragma unroll
          for (int q = 0; q < kPanelMaxG / 32; ++q) {
            const int xx = lane + 32 * q;
            v[u][q] = (c < b && xx < G) ? __ldcg(Pj + (size_t)c * Gp + xx) : 0.0;
          }
        }
        double sacc[CG];
#pragma unroll
        for (int u = 0; u < CG; ++u) {
          sacc[u] = 0.0;
#pragma unroll
          for (int q = 0; q < kPanelMaxG / 32; ++q) sacc[u] += v[u][q];
        }
        {
          const double tot = warp_sum4(sacc, lane);
          const int u = ((lane >> 4) << 1) | ((lane >> 3) & 1);
          if ((lane & 7) == 0 && c0 + u * NW < b) p_s[c0 + u * NW] = tot;
        }
      }
      if (tid < b) pr_s[tid] = prv;
      __syncthreads();
    }
    }
    // The reflector's scalars are computed once (square root and divisions are long FP64 sequences
    // and the SM has few FP64 lanes) and shared: tau, 1/(alpha - beta), and whether there is
    // anything to annihilate.
    if (warp == 0) {
      const double alpha = pr_s[j], s2 = p_s[j];
      double tau = 0.0, rdenom = 0.0;
      if (s2 != 0.0) {
        const double beta = -copysign(sqrt(alpha * alpha + s2), alpha);
        tau = (beta - alpha) / beta;
        rdenom = 1.0 / (alpha - beta);
      }
      if (lane == 0) {
        sc_s[0] = tau;
        sc_s[1] = rdenom;
        if (cta == 0) tau_out[j] = tau;
      }
    }
    __syncthreads();
    const double tau = sc_s[0], rdenom = sc_s[1];     // rdenom == 0 marks H_j = I
    if (tid < b && tid != j) {
      const double wv = pr_s[tid] + p_s[tid] * rdenom;
      w_s[tid] = wv;
      if (cta == 0 && tid < j) gram[(size_t)j * b + tid] = wv;
    }
    // column j becomes v_j (unit lower trapezoidal, explicit ones and zeros)
    for (int r = tid; r < nloc; r += NT) {
      const int grow = gr0 + r;
      Sj[r] = grow > pr ? Sj[r] * rdenom : (grow == pr ? 1.0 : 0.0);
    }
    tau_prev = tau;
    __syncthreads();
  }

  for (int idx = tid; idx < nloc * b; idx += NT) {
    const int r = idx >> lb, c = idx & (b - 1);
    if (gr0 + r >= row0) V[(size_t)(gr0 + r - row0) * ldv + c] = (T)S[(size_t)c * Rp + r];
  }
  // CTA 0 wrote the Gram rows and tau itself: it can go on to the T factor without another launch
  if (Tout != nullptr && cta == 0) {
    __syncthreads();
    tfactor_block<T>(gram, tau_out, b, Tout, ldt, psm);
  }
}

// ------------------------------------------------------------------------------------------
// Compact-WY factor from the Gram rows (Eq. "Q_i = I_m - V_i T_i V_i^T").  The column recurrence
// T[0:j, j] = -tau_j T[0:j, 0:j] (V[:, 0:j]^T v_j) is applied a block at a time: if T11 and T22 are
// the factors of two adjacent groups of s reflectors, the factor of the 2s reflectors is
//   [ T11   -T11 (V1^T V2) T22 ]
//   [  0            T22        ]
// so log2(b) rounds of independent s x s products build T from its diagonal tau.  One CTA; T and the
// Gram rows share one shared-memory array (upper / strictly lower triangle).
// ------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256)
    tfactor_kernel(const double* __restrict__ gram, const double* __restrict__ tau, int b,
                   T* __restrict__ Tout, long long ldt, const int* done_flag, unsigned* bar_reset) {
  if (*reinterpret_cast<const volatile int*>(done_flag)) return;
  if (threadIdx.x == 0 && bar_reset != nullptr) *bar_reset = 0;   // the panel before this kernel is finished with it
  extern __shared__ double tsm_k[];
  tfactor_block<T>(gram, tau, b, Tout, ldt, tsm_k);
}

// ------------------------------------------------------------------------------------------
// Zt[col][0:B] = (op(T) * sum of the partial slots of Z[:, col])   with op(T) = T^T (apply Q^T) or
// T (apply Q).  Zpart is in the slot layout of vtw_sk_kernel: column tile ct (bn columns) is the sum
// of slots p + ct for the CTAs p whose tile range [p*tpc, (p+1)*tpc) meets [ct*kt, (ct+1)*kt),
// summed in CTA order.  Each CTA owns kTzCols columns: it stages op(T) (as the A operand, K = row)
// and the summed columns in shared memory with a pitch of 4 mod 16 elements, which makes the scalar
// fragment loads conflict free, and multiplies on the tensor cores.  The output is the transposed
// (K-contiguous) operand of upd_sk_kernel.
// ------------------------------------------------------------------------------------------
constexpr int kTzCols = 32;
constexpr int kTzThreads = 512;
template <typename T, int B>
__global__ void __launch_bounds__(kTzThreads)
    tz_kernel(const T* __restrict__ Zpart, int bn, int nct, int kt, int tpc, const T* __restrict__ Tm, long long ldt,
              int transpose_t, T* __restrict__ Zt, const int* done_flag) {
  if (*reinterpret_cast<const volatile int*>(done_flag)) return;
  constexpr int PA = B + 4, PB = kTzCols + 4;
  constexpr int NWARP = kTzThreads / 32;
  constexpr int MTILES = B / 16, NTILES = kTzCols / 8;
  extern __shared__ unsigned char zsm_raw[];
  T* As = reinterpret_cast<T*>(zsm_raw);          // [B][PA]: As[l][j] = op(T)[j][l]
  T* Bs = As + (size_t)B * PA;                    // [B][PB]: summed Z[l][col]
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int col0 = blockIdx.x * kTzCols;
  {
    constexpr int EA = (B * B + kTzThreads - 1) / kTzThreads;
    T v[EA];
#pragma unroll
    for (int e = 0; e < EA; ++e) {
      const int idx = tid + e * kTzThreads, l = idx / B, j = idx - l * B;
      v[e] = T(0);
      if (idx < B * B) {
        if (transpose_t) { if (l <= j) v[e] = Tm[(size_t)l * ldt + j]; }     // (T^T)[j][l] = T[l][j], upper triangular
        else             { if (j <= l) v[e] = Tm[(size_t)j * ldt + l]; }     // T[j][l]
      }
    }
#pragma unroll
    for (int e = 0; e < EA; ++e) {
      const int idx = tid + e * kTzThreads, l = idx / B, j = idx - l * B;
      if (idx < B * B) As[l * PA + j] = v[e];
    }
  }
  const int ct = col0 / bn, cin = col0 - ct * bn;   // kTzCols divides bn; tiles past the last hold no data
  const int p_lo = (ct * kt) / tpc, p_hi = ((ct + 1) * kt - 1) / tpc;
  {
    // every thread owns EPT entries; the loads of up to eight slots are in flight together and are
    // then added in slot (= CTA) order
    constexpr int EPT = (B * kTzCols + kTzThreads - 1) / kTzThreads;
    constexpr int SB = EPT >= 8 ? 4 : 8;            // slots per batch, bounded by registers
    double sum[EPT];
#pragma unroll
    for (int e = 0; e < EPT; ++e) sum[e] = 0.0;
    if (ct < nct) {
      for (int p0 = p_lo; p0 <= p_hi; p0 += SB) {
        T v[SB][EPT];
#pragma unroll
        for (int u = 0; u < SB; ++u) {
          const T* slot = Zpart + (size_t)(p0 + u + ct) * (size_t)(B * bn) + cin;
#pragma unroll
          for (int e = 0; e < EPT; ++e) {
            const int idx = tid + e * kTzThreads, l = idx / kTzCols, cl = idx - l * kTzCols;
            v[u][e] = (p0 + u <= p_hi && idx < B * kTzCols) ? __ldcg(slot + (size_t)l * bn + cl) : T(0);
          }
        }
#pragma unroll
        for (int u = 0; u < SB; ++u)
#pragma unroll
          for (int e = 0; e < EPT; ++e) sum[e] += (double)v[u][e];
      }
    }
#pragma unroll
    for (int e = 0; e < EPT; ++e) {
      const int idx = tid + e * kTzThreads, l = idx / kTzCols, cl = idx - l * kTzCols;
      if (idx < B * kTzCols) Bs[l * PB + cl] = (T)sum[e];
    }
  }
  __syncthreads();
  for (int tile = warp; tile < MTILES * NTILES; tile += NWARP) {
    const int j0 = (tile / NTILES) * 16, n0 = (tile % NTILES) * 8;
    T acc[4] = {T(0), T(0), T(0), T(0)};
#pragma unroll 4
    for (int ks = 0; ks < B / 8; ++ks) {
      const int k = ks * 8 + t;
      const T af[4] = {As[k * PA + j0 + g], As[k * PA + j0 + g + 8], As[(k + 4) * PA + j0 + g],
                       As[(k + 4) * PA + j0 + g + 8]};
      const T bf[2] = {Bs[k * PB + n0 + g], Bs[(k + 4) * PB + n0 + g]};
      mma16x8x8(acc, af, bf);
    }
    const int j = j0 + g, col = col0 + n0 + 2 * t;
    Zt[(size_t)col * B + j] = acc[0];
    Zt[(size_t)(col + 1) * B + j] = acc[1];
    Zt[(size_t)col * B + j + 8] = acc[2];
    Zt[(size_t)(col + 1) * B + j + 8] = acc[3];
  }
}

// ------------------------------------------------------------------------------------------
// Algorithm 2 lines 2-4: ||A||_F^2 from the first sample kernel's per-CTA partial sums (fixed order), the
// squared tolerance, and the loop state.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
    init_ctrl_kernel(const double* __restrict__ part, int npart, double tol, int relative, int fixed_rank,
                     int b, int max_rank, Ctrl* ctrl, int* __restrict__ done_after, int* __restrict__ samp, int nsteps,
                     int predict) {
  __shared__ double red[32];
  double s = 0.0;
  for (int i = threadIdx.x; i < npart; i += 256) s += part[i];
  const double tot = block_sum(s, red);
  if (threadIdx.x == 0) {
    ctrl->normA2 = tot;
    ctrl->sigma2 = relative ? tol * tol * tot : tol * tol;
    ctrl->E_sub = tot;
    ctrl->E_dir = tot;
    ctrl->E_prev = tot;
    ctrl->r_prev = -1.0;
    ctrl->fused_samples = 0;
    ctrl->extra_samples = 0;
    ctrl->n_est = 0;
    ctrl->E_est = 0.0;
    ctrl->steps = 0;
    ctrl->k = 0;
    ctrl->bar = 0;
    int status = RRF_OK, done = 0;
    if (!(tot == tot) || tot > 1.7e308) {
      status = RRF_ERR_NONFINITE;
      done = 1;
    } else if (!fixed_rank && !(tot > ctrl->sigma2)) {
      done = 1;
    } else if (b > max_rank) {
      done = 1;
      status = RRF_MAX_RANK_REACHED;
    }
    ctrl->status = status;
    ctrl->done = done;
    // done_after[q] = value of `done` when block step q is about to start; steps that never run keep 1
    if (done_after != nullptr) {
      done_after[0] = done;
      for (int q = 1; q <= nsteps; ++q) done_after[q] = 1;
    }
    // samp[q] != 0: the update of pass q also samples a later panel; the stop rule of pass q-1 decides it
    if (samp != nullptr)
      for (int q = 0; q <= nsteps; ++q) samp[q] = predict == 2 ? 0 : 1;
  }
}

// Algorithm 2 lines 9-10 and the test of line 5 for the next pass, on the device.
__global__ void __launch_bounds__(256)
    stop_kernel(const double* __restrict__ norm_part, int npart, int b, int max_rank, int estimator,
                int fixed_rank, double* __restrict__ tr_sub, double* __restrict__ tr_dir, Ctrl* ctrl,
                int* __restrict__ done_after, int reset_bar, int* __restrict__ samp, int predict) {
  if (*reinterpret_cast<volatile int*>(&ctrl->done)) return;
  __shared__ double red[64];
  double st = 0.0, sr = 0.0;
  for (int i = threadIdx.x; i < npart; i += 256) {
    st += norm_part[2 * i];
    sr += norm_part[2 * i + 1];
  }
  const double top = block_sum(st, red);
  const double trail = block_sum(sr, red + 32);
  if (threadIdx.x == 0) {
    const double e_sub = ctrl->E_sub - top;
    ctrl->E_sub = e_sub;
    ctrl->E_dir = trail;
    const int i = ctrl->steps;
    tr_sub[i] = e_sub;
    tr_dir[i] = trail;
    ctrl->steps = i + 1;
    ctrl->k = (i + 1) * b;
    if (reset_bar) ctrl->bar = 0;
    const double E = estimator == 0 ? trail : e_sub;
    // the sampled rules (estimator >= 2) decide in est_kernel; here only the rank cap ends the loop
    const bool below = estimator < 2 && !(E > ctrl->sigma2);
    const bool met = !fixed_rank && below;
    const bool cap = (i + 2) * b > max_rank;
    if (ctrl->status == RRF_OK && !below && cap) ctrl->status = RRF_MAX_RANK_REACHED;
    if (met || cap) ctrl->done = 1;
    if (done_after != nullptr) done_after[i + 1] = (met || cap) ? 1 : 0;
    // Sampling predictor.  The update of pass i+1 also samples a later panel, which is wasted work if
    // pass i+1 turns out to be the last.  Extrapolate the stopping quantity one pass ahead (last reduction
    // ratio, moved on by its last change) and let that update skip the sampling when the two last ratios
    // agree to 30 % and the prediction is below the tolerance.  If the loop goes on after all, the
    // skipped panel is sampled by a kernel of its own.  predict: 0 = by this rule, 1 = always sample,
    // 2 = never sample.
    if (samp != nullptr) {
      const double Ep = ctrl->E_prev;
      double r = (Ep > 0.0) ? E / Ep : 1.0;
      r = r < 0.0 ? 0.0 : (r > 1.0 ? 1.0 : r);
      const double rp = ctrl->r_prev;
      const double dr = (rp >= 0.0 && r > rp) ? r - rp : 0.0;
      const double rr = r + dr > 1.0 ? 1.0 : r + dr;
      const double e = E * rr;
      const bool steady = rp >= 0.0 && fabs(r - rp) <= 0.3 * fmax(r, rp);
      int want = fixed_rank || !steady || e > 0.9 * ctrl->sigma2;
      if (predict == 1) want = 1;
      if (predict == 2) want = 0;
      samp[i + 1] = want;
      ctrl->E_prev = E;
      ctrl->r_prev = r;
    }
  }
}

// ------------------------------------------------------------------------------------------
// Sampled stopping rules (the paper's outlook: criteria based on the spectral norm of the remaining part, and
// a criterion for the variant that never updates A).  Panel i, Y_i = W Omega_i with Omega_i standard Gaussian,
// probes the residual W left by the first i blocks:
//   estimator 2:  E = ||Y_i||_F^2 / b            (E[E] = ||W||_F^2)
//   estimator 3:  E = (200/pi) max_j ||y_j||^2   (||W||_2^2 <= E with probability 1 - 10^-b; Halko et al., Lemma 4.1)
// from the per-CTA column sums of squares the panel kernel left in csq.  If E <= sigma^2 the loop ends with
// k = i b (panel i is discarded).  advance != 0 (no update kernels in the loop): this kernel also counts the
// block and applies the rank cap.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(128)
    est_kernel(const double* __restrict__ csq, int G, int Gp, int b, int max_rank, int estimator, int fixed_rank,
               int advance, int step, double* __restrict__ tr_est, Ctrl* ctrl) {
  if (*reinterpret_cast<volatile int*>(&ctrl->done)) return;
  __shared__ double col[128];
  const int c = threadIdx.x;
  double s = 0.0;
  if (c < b)
    for (int x = 0; x < G; ++x) s += __ldcg(csq + (size_t)c * Gp + x);
  col[c] = c < b ? s : 0.0;
  __syncthreads();
  if (c == 0) {
    double E = 0.0;
    if (estimator == 2) {
      for (int j = 0; j < b; ++j) E += col[j];
      E /= (double)b;
    } else {
      for (int j = 0; j < b; ++j) E = fmax(E, col[j]);
      E *= 63.66197723675813;                     // 200 / pi
    }
    tr_est[step] = E;
    ctrl->E_est = E;
    ctrl->n_est = step + 1;
    if (!fixed_rank && !(E > ctrl->sigma2)) {
      ctrl->done = 1;
    } else if (advance) {
      ctrl->steps = step + 1;
      ctrl->k = (step + 1) * b;
      if ((step + 2) * b > max_rank) {
        ctrl->done = 1;
        if (ctrl->status == RRF_OK) ctrl->status = RRF_MAX_RANK_REACHED;
      }
    }
  }
}

// Squared Frobenius norm of a rows x cols matrix, in two fixed-order stages (accumulated in double): every CTA
// sums a contiguous range of rows, CTA 0's successor kernel adds the partials in CTA order.
template <typename T>
__global__ void __launch_bounds__(256)
    frob2_part_kernel(const T* __restrict__ C, long long ldc, long long rows, long long cols, double* __restrict__ part) {
  __shared__ double red[32];
  const long long per = (rows + gridDim.x - 1) / gridDim.x;
  const long long r_lo = per * blockIdx.x, r_hi = min(rows, r_lo + per);
  double s = 0.0;
  for (long long r = r_lo; r < r_hi; ++r)
    for (long long c = threadIdx.x; c < cols; c += 256) {
      const double v = (double)C[r * ldc + c];
      s += v * v;
    }
  const double tot = block_sum(s, red);
  if (threadIdx.x == 0) part[blockIdx.x] = tot;
}
__global__ void __launch_bounds__(256) frob2_final_kernel(const double* __restrict__ part, int n, double* __restrict__ out) {
  __shared__ double red[32];
  double s = 0.0;
  for (int i = threadIdx.x; i < n; i += 256) s += part[i];
  const double tot = block_sum(s, red);
  if (threadIdx.x == 0) *out = tot;
}

// dst (cols x rows, leading dimension ldd) = src^T for a rows x cols matrix src (leading dimension lds), both stored
// row by row: square tiles of 256 bytes a side (32 doubles, 64 floats) pass through shared memory so that reads and
// writes are both along rows.  This is all the column-major entry points need: a column-major matrix is its
// transpose stored row by row.
template <typename T>
__global__ void __launch_bounds__(256)
    transpose_kernel(const T* __restrict__ src, long long lds, long long rows, long long cols, T* __restrict__ dst,
                     long long ldd) {
  constexpr int D = 256 / (int)sizeof(T), RS = 256 / D;      // tile side; tile rows covered by one sweep of the block
  __shared__ T tile[D][D + 1];
  const long long tiles_c = (cols + D - 1) / D, tiles = tiles_c * ((rows + D - 1) / D);
  const int tx = threadIdx.x % D, ty = threadIdx.x / D;
  for (long long t = blockIdx.x; t < tiles; t += gridDim.x) {
    const long long r0 = (t / tiles_c) * D, c0 = (t % tiles_c) * D;
    for (int i = ty; i < D; i += RS)
      if (r0 + i < rows && c0 + tx < cols) tile[i][tx] = src[(r0 + i) * lds + c0 + tx];
    __syncthreads();
    for (int i = ty; i < D; i += RS)
      if (c0 + i < cols && r0 + tx < rows) dst[(c0 + i) * ldd + r0 + tx] = tile[tx][i];
    __syncthreads();
  }
}

// dst (rows x b, dense) = sum of the nseg stacked partial panels the sample kernel wrote, in their fixed order
template <typename T>
__global__ void __launch_bounds__(256)
    panel_sum_kernel(const T* __restrict__ Ypart, int nseg, long long seg_stride, long long rows, int b,
                     T* __restrict__ dst, const Ctrl* ctrl) {
  if (*reinterpret_cast<const volatile int*>(&ctrl->done)) return;
  const long long total = rows * b;
  for (long long idx = (long long)blockIdx.x * 256 + threadIdx.x; idx < total; idx += (long long)gridDim.x * 256) {
    double s = (double)Ypart[idx];
    for (int sg = 1; sg < nseg; ++sg) s += (double)Ypart[idx + (long long)sg * seg_stride];
    dst[idx] = (T)s;
  }
}

// ------------------------------------------------------------------------------------------
// Algorithm 2 line 6: standard Gaussians from a counter-based generator (Philox-4x32, 10
// rounds, Salmon et al. 2011; Box-Muller in double).  Counter = (pair index, 0, vector index,
// 0), key = seed: one call yields elements (j, 2q) and (j, 2q+1) of OmegaT.
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ void philox4x32_10(uint32_t (&c)[4], uint32_t k0, uint32_t k1) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint64_t p0 = (uint64_t)0xD2511F53u * c[0];
    const uint64_t p1 = (uint64_t)0xCD9E8D57u * c[2];
    const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c[1] ^ k0;
    const uint32_t n1 = (uint32_t)p1;
    const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c[3] ^ k1;
    const uint32_t n3 = (uint32_t)p0;
    c[0] = n0; c[1] = n1; c[2] = n2; c[3] = n3;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
}

template <typename T>
__global__ void __launch_bounds__(256)
    omega_kernel(T* __restrict__ O, long long ldo, long long n, int nvec, int first_vec, uint64_t seed) {
  const long long npairs = (n + 1) / 2;
  const long long total = npairs * nvec;
  for (long long idx = (long long)blockIdx.x * 256 + threadIdx.x; idx < total; idx += (long long)gridDim.x * 256) {
    const long long jv = idx / npairs, q = idx - jv * npairs;
    const uint64_t vec = (uint64_t)(first_vec + jv);
    uint32_t c[4] = {(uint32_t)q, (uint32_t)((uint64_t)q >> 32), (uint32_t)vec, (uint32_t)(vec >> 32)};
    philox4x32_10(c, (uint32_t)seed, (uint32_t)(seed >> 32));
    const uint64_t a = ((uint64_t)c[1] << 32) | c[0], bb = ((uint64_t)c[3] << 32) | c[2];
    const double u1 = ((double)(a >> 12) + 0.5) * (1.0 / 4503599627370496.0);   // (0, 1), exact
    const double u2 = ((double)(bb >> 12) + 0.5) * (1.0 / 4503599627370496.0);
    const double rad = sqrt(-2.0 * log(u1));
    double sn, cs;
    sincospi(2.0 * u2, &sn, &cs);
    T* row = O + jv * ldo;
    row[2 * q] = (T)(rad * cs);
    if (2 * q + 1 < n) row[2 * q + 1] = (T)(rad * sn);
  }
}

// Register-resident arithmetic loop used to measure the attainable rate of one pipe:
// kind 0 = f64 mma m16n8k8, 1 = f64 FMA, 2 = f32 FMA, 3 = tf32 mma m16n8k8.
__global__ void __launch_bounds__(256) peak_kernel(double* __restrict__ sink, int iters, int kind) {
  double out = 0.0;
  if (kind == 0) {
    double c[8][4];
    for (int i = 0; i < 8; ++i)
      for (int j = 0; j < 4; ++j) c[i][j] = 0.0;
    const double a[4] = {threadIdx.x * 1e-9 + 1.0, 2.0, 3.0, 4.0}, b[2] = {threadIdx.x * 1e-9 - 1.0, 0.5};
    for (int it = 0; it < iters; ++it) {
#pragma unroll
      for (int i = 0; i < 8; ++i) mma16x8x8(c[i], a, b);
    }
    for (int i = 0; i < 8; ++i)
      for (int j = 0; j < 4; ++j) out += c[i][j];
  } else if (kind == 3) {
    float c[8][4];
    for (int i = 0; i < 8; ++i)
      for (int j = 0; j < 4; ++j) c[i][j] = 0.f;
    const uint32_t a[4] = {threadIdx.x, 1u, 2u, 3u}, b[2] = {threadIdx.x, 5u};
    for (int it = 0; it < iters; ++it) {
#pragma unroll
      for (int i = 0; i < 8; ++i) mma_tf32(c[i], a, b);
    }
    for (int i = 0; i < 8; ++i)
      for (int j = 0; j < 4; ++j) out += c[i][j];
  } else if (kind == 1) {
    double c[16];
    for (int i = 0; i < 16; ++i) c[i] = i;
    const double a = threadIdx.x * 1e-9 + 1.0, b = 1e-9;
    for (int it = 0; it < iters; ++it) {
#pragma unroll
      for (int i = 0; i < 16; ++i) c[i] = fma(c[i], a, b);
    }
    for (int i = 0; i < 16; ++i) out += c[i];
  } else {
    float c[16];
    for (int i = 0; i < 16; ++i) c[i] = (float)i;
    const float a = threadIdx.x * 1e-9f + 1.0f, b = 1e-9f;
    for (int it = 0; it < iters; ++it) {
#pragma unroll
      for (int i = 0; i < 16; ++i) c[i] = fmaf(c[i], a, b);
    }
    for (int i = 0; i < 16; ++i) out += c[i];
  }
  sink[(size_t)blockIdx.x * blockDim.x + threadIdx.x] = out;
}

template <typename T>
__global__ void __launch_bounds__(256) eye_kernel(T* __restrict__ Q, long long ldq, long long m, int k) {
  const long long total = m * k;
  for (long long idx = (long long)blockIdx.x * 256 + threadIdx.x; idx < total; idx += (long long)gridDim.x * 256) {
    const long long r = idx / k, c = idx - r * k;
    Q[r * ldq + c] = r == c ? T(1) : T(0);
  }
}

// dst (rows_total x ncols) <- first rows_copy rows of src, zeros below
template <typename T>
__global__ void __launch_bounds__(256)
    copy_rows_kernel(T* __restrict__ dst, long long ldd, const T* __restrict__ src, long long lds, long long rows_copy,
                     long long rows_total, long long ncols) {
  const long long total = rows_total * ncols;
  for (long long idx = (long long)blockIdx.x * 256 + threadIdx.x; idx < total; idx += (long long)gridDim.x * 256) {
    const long long r = idx / ncols, c = idx - r * ncols;
    dst[r * ldd + c] = r < rows_copy ? src[r * lds + c] : T(0);
  }
}

}  // namespace rrf
