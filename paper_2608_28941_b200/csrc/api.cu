// C ABI of the range finder: argument checks, workspace carving, tensor maps and the
// enqueue of Algorithm 2's block loop.  See include/rrf.h for the contract of every call.
#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cmath>
#include <cstring>
#include <mutex>
#include <new>
#include <type_traits>
#include <vector>

#include "gemm_sk.cuh"
#include "gemm_tc.cuh"
#include "gemm_tc_upd.cuh"
#include "gemm_tc_vtw.cuh"
#include "panel_blk.cuh"

// NVTX ranges around the phases of rrf_run (host-side enqueue order), compiled in with -DRRF_NVTX only
// (python -m paper_2608_28941_b200.build --nvtx); one range per kernel group, named "<phase> <block step>".
#ifdef RRF_NVTX
#include <nvtx3/nvToolsExt.h>
static const char* const kNvtxPhase[] = {"init", "sample", "panel", "tfactor", "vtw", "tz", "update", "stop", "end"};
#define RRF_NVTX_MARK(open, phase, step)                                   \
  do {                                                                     \
    if (open) nvtxRangePop();                                              \
    char nm_[48];                                                          \
    std::snprintf(nm_, sizeof nm_, "rrf %s %d", kNvtxPhase[phase], step);  \
    nvtxRangePushA(nm_);                                                   \
    open = true;                                                           \
  } while (0)
#define RRF_NVTX_CLOSE(open) \
  do {                       \
    if (open) nvtxRangePop(); \
    open = false;            \
  } while (0)
#else
#define RRF_NVTX_MARK(open, phase, step) (void)(open)
#define RRF_NVTX_CLOSE(open) (void)(open)
#endif

namespace rrf {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

constexpr int kMaxSmem = 232448;   // 227 KB opt-in dynamic shared memory per CTA on sm_100
constexpr int kMaxSms = kPanelMaxG;       // workspace sizes are bounds for devices with up to this many SMs

}  // namespace rrf

struct rrf_ctx {
  int device;
  int sms;
  int smem_optin;
  rrf::EncodeTiledFn encode;
  rrf::Ctrl* d_ctrl;     // status words for the calls that do not run Algorithm 2's loop
  int last_cuda;
  int panel_smem_max;    // dynamic shared memory the panel kernel may use (opt-in limit minus its static part)
  int tsqr_smem_max;     // the same for the tree panel kernel
  int blk_smem_max;      // the same for the blocked panel kernel
  int profiling;
  cudaStream_t aux;                      // side stream: the T factor is built while V^T W runs
  std::vector<cudaEvent_t> sync_events;  // fork/join events between the caller's stream and `aux`
  std::vector<cudaEvent_t> events;
  rrf_profile_t profile;
  // rrf_run as a CUDA graph: captured on the second call with the same arguments, replayed after that
  cudaStream_t cap;                      // stream the capture runs on (the caller's may be the legacy stream)
  cudaGraph_t graph;
  cudaGraphExec_t gexec;
  std::vector<unsigned char> gkey;       // arguments the instantiated graph was captured for
  std::vector<unsigned char> gcand;      // arguments of the last directly enqueued call
  std::vector<std::pair<int, int>> gmarks;
  int graph_off;                         // set when a capture failed: enqueue directly from then on
  int cand_steps;                        // block steps the last directly enqueued call ran, -1 if it did not end by its own rule
  int gsteps;                            // block steps the instantiated graph holds (it may hold fewer than max_rank / b)
  int cluster_ok;                        // a 16-CTA cluster of the panel kernel can be resident on this device
  int f32_engine;                        // single-precision V^T W: 0 = mma.sync 3xTF32, 1 = tcgen05 3xTF32
  int tc_chunk;                          // tcgen05: 64-row tiles summed in tensor memory between round-to-nearest adds
};

namespace rrf {

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
static inline int ceil_div(long long a, long long b) { return (int)((a + b - 1) / b); }

// ------------------------------------------------------------------ tile configuration
constexpr int kSampleBM = 128, kSampleStages = 2;
constexpr int kVtwBK = 64;

struct SamplePlan { int nslabs, nseg, kt_per_seg, ctas; };
constexpr int kSampleMaxSeg = 12;
// K segments are chosen to fill whole waves of one CTA per SM with equal K ranges
static SamplePlan plan_sample(int sms, long long rows, long long n, int esize, int kbs) {
  SamplePlan p;
  const int KE = 128 / esize;
  p.nslabs = ceil_div(rows, kSampleBM);
  const int KT = ceil_div(n, KE * kbs);
  int best = 1;
  double best_eff = 0.0;
  for (int nseg = 1; nseg <= std::min(KT, kSampleMaxSeg); ++nseg) {
    const int ctas = p.nslabs * nseg, waves = ceil_div(ctas, sms), per = ceil_div(KT, nseg);
    const double eff = (double)ctas / ((double)waves * sms) * (double)KT / ((double)per * nseg);
    if (eff > best_eff + 1e-9) {
      best_eff = eff;
      best = nseg;
    }
  }
  p.kt_per_seg = ceil_div(KT, best);
  p.nseg = ceil_div(KT, p.kt_per_seg);
  p.ctas = sms;   // one CTA per SM walks the items
  return p;
}

// stream-K plan of Z = V^T C: tiles (column tile, K chunk), one CTA per SM
struct VtwPlan { int bn, nct, KT, total, tpc, P, npad, slots, tc, chunk; };
static VtwPlan plan_vtw(int sms, long long rows, long long ncols, int bn) {
  VtwPlan p;
  p.bn = bn;
  p.nct = ceil_div(ncols, bn);
  p.npad = ceil_div(ncols, 128) * 128;   // Zt rows: a multiple of every tile width in use
  p.KT = ceil_div(rows, kVtwBK);
  p.total = p.nct * p.KT;
  p.tpc = ceil_div(p.total, sms);
  p.P = ceil_div(p.total, p.tpc);
  p.slots = p.P + p.nct;
  p.tc = 0;
  p.chunk = 0;
  return p;
}
// stream-K plan of the fused update: tiles (row slab, column tile)
// what the tcgen05 version of the fused update needs beyond the common arguments
struct UpdTc {
  const rrf_ctx* h;       // for the tensor maps built per launch
  const void* V;          // reflectors (read directly, not through a tensor map)
  long long ldv;
  const void* Zt;         // [npad][b], written by the T Z kernel
  int npad;
  const void* Om;         // OmegaT as the run sees it
  long long ldom;
  void* zsplit;           // [2][npad][b]: TF32 planes of Zt
  void* osplit;           // [2][b][ldo2]: TF32 planes of the rows of OmegaT being sampled with
  long long ldo2;
  int chunk;
  CUtensorMap tmZs, tmOs;
};
// p0, Lb: this launch's CTAs are numbers p0 ... of the pass and start at tile Lb (a pass split over two launches)
struct UpdPlan { int NS, NC, total, tpc, P, slots; const UpdTc* tc; int p0, Lb; };
static UpdPlan plan_upd(int sms, long long rows, long long ncols, int bm, int bn, int wn) {
  UpdPlan p;
  p.NS = ceil_div(rows, bm);
  p.NC = ceil_div(ncols, bn);
  p.total = p.NS * p.NC;
  p.tpc = ceil_div(p.total, sms);
  p.P = ceil_div(p.total, p.tpc);
  p.slots = (p.P + p.NS) * wn;
  p.tc = nullptr;
  p.p0 = 0;
  p.Lb = 0;
  return p;
}
// The panel kernel's variants: rows a lane keeps in registers, row groups, and whether the slab is
// allocated at its full height (32 * rows per lane * groups, zero filled) or exactly (the fallback for
// the one shape that only fits unpadded).
constexpr int kPanelVariants = 6;
static const int kVariantRows[kPanelVariants] = {64, 128, 224, 320, 512, 224};
static const bool kVariantPad[kPanelVariants] = {true, true, true, true, true, false};
template <typename T>
static const void* panel_variant(int q) {
  switch (q) {
    case 0: return (const void*)panel_kernel<T, 2, 1>;
    case 1: return (const void*)panel_kernel<T, 4, 1>;
    case 2: return (const void*)panel_kernel<T, 7, 1>;
    case 3: return (const void*)panel_kernel<T, 5, 2>;
    case 4: return (const void*)panel_kernel<T, 8, 2>;
    default: return (const void*)panel_kernel<T, 7, 1, false>;
  }
}
template <typename T>
static const void* panel_variant_cl(int q) {     // the same shapes as one thread-block cluster (padded ones only)
  switch (q) {
    case 0: return (const void*)panel_kernel<T, 2, 1, true, true>;
    case 1: return (const void*)panel_kernel<T, 4, 1, true, true>;
    case 2: return (const void*)panel_kernel<T, 7, 1, true, true>;
    case 3: return (const void*)panel_kernel<T, 5, 2, true, true>;
    case 4: return (const void*)panel_kernel<T, 8, 2, true, true>;
    default: return (const void*)panel_kernel<T, 8, 1, true, true, true>;   // slab in registers during the column loop
  }
}
constexpr int kPanelVariantsCl = 6;
constexpr int kPanelVariantReg = 5;
constexpr int kClusterMaxRows = 128;
struct PanelPlan { int G, R, Rp, variant; size_t smem; bool cl; };
// ctas == 0: the panel is spread over every SM (short slabs, short passes).  ctas > 0: the panel is
// confined to that many CTAs so that the other SMs stay free for the GEMM kernels of the look-ahead
// schedule; `fix` adds the b rows above the panel and the shared memory of the late reflector
// application.
// The panel as ONE thread-block cluster (sums through distributed shared memory): possible when at most
// kClusterMax slabs hold it.  The grid is a power of two so that every cluster size is one the hardware takes;
// CTAs past the last row hold no rows and only take part in the exchanges.
static bool plan_panel_cl(const rrf_ctx* h, long long rows, int b, PanelPlan* p, bool fix) {
  if (!h->cluster_ok || (fix && b > 64)) return false;
  const long long ext = rows + (fix ? b : 0);
  const int R = std::max(64, ceil_div(ext, kClusterMax));
  // With slabs taller than this the longer pass over a slab costs more than the cheaper exchange saves
  // (measured: 4096 x 64 takes 279 us as one cluster of 16 against 260 us on 148 CTAs; 1024 x 16 falls from 64 to 54)
  // With the register-resident column loop (b <= 64) a 4096 x 64 panel takes 232 us on its own, but inside a run, where
  // 16 CTAs also sum the partial panels and store V, the 4096-row passes of config 4 take 284 us against 261 us.
  const bool reg = b <= 64 && R <= kRegRows;
  if (!reg && R > kClusterMaxRows) return false;
  int G = 1;
  while (G < ceil_div(ext, R)) G *= 2;
  if (G > kClusterMax) return false;
  const size_t extra = (size_t)panel_extra_doubles(b) + (fix ? panel_fix_doubles(b) : 0) + panel_cluster_doubles(b);
  if (reg) {
    p->R = R;
    p->G = G;
    p->Rp = kRegRows + 1;
    p->variant = kPanelVariantReg;
    p->cl = true;
    p->smem = ((size_t)b * p->Rp + extra) * sizeof(double);
    return p->smem <= (size_t)h->panel_smem_max;
  }
  for (int q = 0; q < kPanelVariantReg; ++q) {
    if (R > kVariantRows[q]) continue;
    p->R = R;
    p->G = G;
    p->Rp = kVariantRows[q] + 1;
    p->variant = q;
    p->cl = true;
    p->smem = ((size_t)b * p->Rp + extra) * sizeof(double);
    if (p->smem <= (size_t)h->panel_smem_max) return true;
  }
  return false;
}
static bool plan_panel(const rrf_ctx* h, long long rows, int b, PanelPlan* p, int ctas = 0, bool fix = false) {
  p->cl = false;
  if (fix && b > 64) return false;
  const long long ext = rows + (fix ? b : 0);
  // tall slabs keep the grid, and with it the all-to-all read of the partial sums, small
  const int R = std::max(64, ceil_div(ext, ctas > 0 ? ctas : h->sms));
  p->R = R;
  p->G = ceil_div(ext, R);
  if (p->G > h->sms) return false;
  const size_t extra = (size_t)panel_extra_doubles(b) + (fix ? panel_fix_doubles(b) : 0);
  for (int q = 0; q < kPanelVariants; ++q) {
    if (R > kVariantRows[q]) continue;
    if (kVariantPad[q]) {
      p->Rp = kVariantRows[q] + 1;          // odd pitch: the transposing load/store phases stay conflict free
    } else {
      if (fix) continue;
      p->Rp = ((size_t)b * (R | 1) + extra) * sizeof(double) <= (size_t)h->panel_smem_max ? (R | 1) : R;
    }
    p->variant = q;
    p->smem = ((size_t)b * p->Rp + extra) * sizeof(double);
    if (p->smem <= (size_t)h->panel_smem_max) return true;
  }
  return false;
}
constexpr int kTsqrMaxB = 64;      // widest panel the tree kernel factors (wider ones take the per-column kernel)
// Plan of the tree panel kernel: leaf slab height (one of the factorisation's tilings), fan-in, levels.
struct TreePlan { TsqrPlan t; int ctas, Rp, nbar; size_t smem; double est_us; };
static size_t tsqr_smem_bytes(int b, int slab_rows) {
  return ((size_t)b * (slab_rows + 1) + panel_fix_doubles(b) + tsqr_small_doubles(b)) * sizeof(double);
}
// rough time of one CTA-local factorisation of `rows` x b (microseconds): b dependent columns
static double tsqr_level_us(int rows, int b) { return b * (1100.0 + 0.09 * rows * b) / 1965.0 + 6.0; }
// max_ctas == 0: any number up to the SM count.  Returns false if no tiling fits.
static bool plan_tree(const rrf_ctx* h, long long rows, int b, int max_ctas, bool fix, TreePlan* out) {
  if (b > kTsqrMaxB) return false;
  const long long ext = rows + (fix ? b : 0);
  const int limit = max_ctas > 0 ? std::min(max_ctas, h->sms) : h->sms;
  int vmax = -1;                                     // tallest tiling that fits in shared memory
  for (int v = 0; v < 5; ++v)
    if (tsqr_smem_bytes(b, tsqr_variant_rows(v)) <= (size_t)h->tsqr_smem_max) vmax = v;
  if (vmax < 0) return false;
  const int f = tsqr_variant_rows(vmax) / b;
  bool found = false;
  for (int v = 0; v <= vmax; ++v) {
    const int R = tsqr_variant_rows(v);
    if (R < (fix ? 2 * b : b)) continue;
    TreePlan p{};
    p.t.R = R;
    p.t.f = f;
    p.t.cnt[0] = ceil_div(ext, R);
    p.t.var[0] = v;
    p.t.off[0] = 0;
    int l = 0, top = v;
    double est = tsqr_level_us(R, b);
    bool ok = true;
    while (p.t.cnt[l] > 1) {
      if (f < 2 || l + 1 >= 6) { ok = false; break; }
      p.t.cnt[l + 1] = ceil_div(p.t.cnt[l], f);
      p.t.off[l + 1] = p.t.off[l] + p.t.cnt[l];
      const int need = std::min(f, p.t.cnt[l]) * b;
      int nv = 0;
      while (tsqr_variant_rows(nv) < need) ++nv;
      p.t.var[l + 1] = nv;
      top = std::max(top, nv);
      est += tsqr_level_us(tsqr_variant_rows(nv), b) + 8.0;   // + the way down and two barriers
      ++l;
    }
    if (!ok) continue;
    p.t.nlev = l + 1;
    p.ctas = p.t.off[l] + p.t.cnt[l];
    if (p.ctas > limit) continue;
    p.Rp = tsqr_variant_rows(top) + 1;
    p.smem = tsqr_smem_bytes(b, tsqr_variant_rows(top));
    p.nbar = 2 * p.t.nlev - 1 + (fix ? 2 : 0);
    p.est_us = est + 0.25 * b + 10.0 + (fix ? 25.0 : 0.0);     // + elimination, final product, fix-up
    if (!found || p.est_us < out->est_us) {
      *out = p;
      found = true;
    }
  }
  return found;
}
// Plan of the blocked panel kernel (panel_blk.cuh): slab height per CTA and which of its small matrices fit in
// shared memory beside the slab.
struct BlkPlan { int G, R, RS, Rp, ksplit, c_in_smem, gslab; size_t smem; };
// `global_slab`: keep the slabs in global memory (no height limit; the panel can be confined to very few SMs)
static bool plan_blk(const rrf_ctx* h, long long rows, int b, BlkPlan* p, int ctas = 0, bool fix = false,
                     bool global_slab = false) {
  if (fix && b > 64) return false;
  p->gslab = 0;
  if (global_slab) {
    const long long ext = rows + (fix ? b : 0);
    const size_t fixd = fix ? (size_t)panel_fix_doubles(b) : 0;
    p->R = std::max(64, ceil_div(ext, ctas > 0 ? ctas : h->sms));
    p->G = ceil_div(ext, p->R);
    p->RS = (p->R + 15) / 16 * 16;
    p->Rp = p->RS + 1;
    p->ksplit = std::max(1, 16 / (b / 16));
    p->c_in_smem = 1;
    p->gslab = 1;
    p->smem = (std::max(fixd, p->ksplit > 1 ? (size_t)kBlkDw : 0) + (size_t)kMB * (b + 8) + 16 + 8 + 8 + 8 + 64 + 64 + 8 + 8) * sizeof(double);
    return p->G <= h->sms;
  }
  const long long ext = rows + (fix ? b : 0);
  const size_t small = 16 + 8 + 8 + 8 + 64 + 64 + 8 + 8;
  const size_t fixd = fix ? (size_t)panel_fix_doubles(b) : 0;
  int R = std::max(64, ceil_div(ext, ctas > 0 ? ctas : h->sms));
  if (ctas == 0) {
    // Every column costs one exchange among all CTAs, whose latency grows with their number, while the pass
    // over a slab is cheap: prefer few tall slabs (up to 320 rows) where shared memory allows.
    const size_t room = (size_t)h->blk_smem_max / sizeof(double) - std::max(fixd, (size_t)kBlkDw) - (size_t)kMB * (b + 8) - small;
    const int tall = std::min(320, (int)(room / b - 1) / 16 * 16);
    if (tall > R) R = tall;
  }
  p->R = R;
  p->G = ceil_div(ext, R);
  if (p->G > h->sms) return false;
  p->RS = (R + 15) / 16 * 16;
  // roomy: odd pitch, D partials of the K-split warps and C staged in shared memory
  p->ksplit = std::max(1, 16 / (b / 16));
  p->c_in_smem = 1;
  p->Rp = p->RS + 1;
  p->smem = ((size_t)b * p->Rp + std::max(fixd, p->ksplit > 1 ? (size_t)kBlkDw : 0) + (size_t)kMB * (b + 8) + small) * sizeof(double);
  if (p->smem <= (size_t)h->blk_smem_max) return true;
  // tight: nothing but the slab (and the fix-up staging)
  p->ksplit = 1;
  p->c_in_smem = 0;
  p->Rp = p->RS;
  p->smem = ((size_t)b * p->Rp + fixd + small) * sizeof(double);
  return p->smem <= (size_t)h->blk_smem_max;
}
// Fewest CTAs whose shared memory holds a rows x b panel with the fix-up staging; 0 if none.
static int panel_min_ctas(const rrf_ctx* h, long long rows, int b) {
  if (b > 64) return 0;
  const size_t extra = (size_t)panel_extra_doubles(b) + panel_fix_doubles(b);
  int best = 0;
  for (int q = 0; q < kPanelVariants; ++q)
    if (kVariantPad[q] && ((size_t)b * (kVariantRows[q] + 1) + extra) * sizeof(double) <= (size_t)h->panel_smem_max)
      best = std::max(best, kVariantRows[q]);
  return best > 0 ? ceil_div(rows + b, best) : 0;
}
static size_t direct_scratch_bytes(int sms, int b) {
  // P[2][b][Gp] + piv[2][b] + gram[b][b] + tau[b] (+ barrier word, padded)
  const int gp = (sms + 31) / 32 * 32;
  return align_up(((size_t)2 * gp * b + 2 * (size_t)b + (size_t)b * b + b) * sizeof(double) + 256, 256);
}
static size_t tsqr_scratch_bytes(int sms, int b) {
  // Rbuf, Xbuf, Kbuf [CTA][b*b] + Ubuf [2][b*b]
  return b <= kTsqrMaxB ? align_up(((size_t)3 * sms + 2) * b * b * sizeof(double), 256) : 0;
}
// blocked panel kernel: exchange lines, per-CTA partials, reduced block, and three tag arrays (zeroed before use)
// zeroed before use: the flagged words of the exchanges, Lw [2][16][Gp][2], Pw [8 b][Gp][2], Rw [16 b][2]
static size_t blk_tag_bytes(int sms, int b) {
  const size_t gp = (size_t)(sms + 31) / 32 * 32;
  return align_up(((size_t)2 * 16 * gp * 2 + (size_t)kMB * b * gp * 2 + (size_t)16 * b * 2) * sizeof(unsigned long long), 256);
}
static size_t blk_slab_bytes(int sms, int b, long long rows) {   // slabs in global memory: [G][b][Rp], Rp <= R + 17
  return align_up((size_t)b * (size_t)(2 * (rows + b) + 17LL * sms) * sizeof(double), 256);   // G R < 2 (rows + b)
}
static size_t blk_scratch_bytes(int sms, int b, long long rows) {
  return blk_tag_bytes(sms, b) + align_up((size_t)sms * kMB * b * sizeof(double), 256) + blk_slab_bytes(sms, b, rows);
}
static size_t panel_scratch_bytes(int sms, int b, long long rows) {
  return direct_scratch_bytes(sms, b) + tsqr_scratch_bytes(sms, b) + blk_scratch_bytes(sms, b, rows);
}
constexpr int kLookMaxCtas = 48;   // most CTAs a confined panel may take
// Rough cost model of one pass, in microseconds, used only to choose the schedule (fitted to event
// timings on a B200; the look-ahead is right or wrong by its measured time, not by this model).
struct PassModel {
  int sms;
  double rows, n;
  int b;
  bool f64;
  bool tc;      // single precision on tcgen05
  bool cl;      // the confined panel runs as one thread-block cluster with its slab in registers
  // flop per microsecond the two GEMM kernels sustain on the whole device
  double vtw() const { return 2.0 * rows * n * b / (f64 ? 33e6 : (tc ? 75e6 : 45e6)) + 10.0; }
  double upd() const { return 4.0 * rows * n * b / (f64 ? 27e6 : (tc ? 100e6 : 32e6)) + 15.0; }
  // fix-up + panel + T factor on `ctas` SMs, with the launch and event hand-overs of the side stream
  double panel_chain(int ctas) const {
    const double R = std::max(64.0, (rows + b) / ctas);
    if (cl)     // one cluster, slab in registers: 4096 x 64 takes 232 us, 4096 x 32 107 us, 1024 x 16 55 us on their own
      return (b * (3700.0 + 42.0 * b) + 40000.0 + 0.07 * R * b * b) / 1965.0 + 20.0;
    const double cycles = b * (7000.0 + 0.14 * R * b) + 20000.0 + 0.07 * R * b * b;
    return cycles / 1965.0 + 0.3 * b + (f64 ? 45.0 : 85.0);
  }
  // the stream-K GEMMs lose a little more than the SMs they give up (tile quantisation)
  double scale(int ctas) const { return std::pow((double)sms / (sms - ctas), 1.15); }
  double step_ungated(int ctas) const { return std::max(panel_chain(ctas), (vtw() + upd()) * scale(ctas)); }
  double step_gated(int ctas) const { return vtw() + std::max(panel_chain(ctas), upd() * scale(ctas)); }
  double step_serial() const { return vtw() + upd() + b * 4.2 + 25.0; }
};
static size_t look_scratch_bytes(int b) {   // Gpart[kLookMaxCtas][b*b] + M[b*b]
  return align_up((size_t)(kLookMaxCtas + 1) * b * b * sizeof(double), 256);
}
struct PanelScratch { double *P, *piv, *gram, *tau; unsigned* bar; TsqrScratch ts; BlkScratch bk; unsigned* blk_tags; size_t blk_tag_bytes; double* gslab; };
// `sms`: the SM count the buffers were sized for (the handle's bound kMaxSms for caller workspaces)
static PanelScratch carve_panel(unsigned char* base, int sms, int b, bool with_tree = true) {
  PanelScratch s;
  s.P = reinterpret_cast<double*>(base);
  s.piv = s.P + (size_t)2 * ((sms + 31) / 32 * 32) * b;
  s.gram = s.piv + 2 * (size_t)b;
  s.tau = s.gram + (size_t)b * b;
  s.bar = reinterpret_cast<unsigned*>(s.tau + b);
  s.ts = TsqrScratch{nullptr, nullptr, nullptr, nullptr};
  s.bk = BlkScratch{nullptr, nullptr, nullptr, nullptr};
  s.blk_tags = nullptr;
  s.blk_tag_bytes = 0;
  s.gslab = nullptr;
  if (with_tree && b <= kTsqrMaxB) {
    double* t = reinterpret_cast<double*>(base + direct_scratch_bytes(sms, b));
    const size_t blk = (size_t)sms * b * b;
    s.ts = TsqrScratch{t, t + blk, t + 2 * blk, t + 3 * blk};
  }
  if (with_tree) {
    unsigned char* q = base + direct_scratch_bytes(sms, b) + tsqr_scratch_bytes(sms, b);
    const size_t gp = (size_t)(sms + 31) / 32 * 32;
    s.blk_tags = reinterpret_cast<unsigned*>(q);
    s.blk_tag_bytes = blk_tag_bytes(sms, b);
    s.bk.Lw = reinterpret_cast<unsigned long long*>(q);
    s.bk.Pw = s.bk.Lw + (size_t)2 * 16 * gp * 2;
    s.bk.Rw = s.bk.Pw + (size_t)kMB * b * gp * 2;
    s.bk.Cg = reinterpret_cast<double*>(q + blk_tag_bytes(sms, b));
    s.gslab = reinterpret_cast<double*>(q + blk_tag_bytes(sms, b) + align_up((size_t)sms * kMB * b * sizeof(double), 256));
  }
  return s;
}

// ------------------------------------------------------------------ tensor maps
static bool make_map(const rrf_ctx* h, CUtensorMap* map, int dtype, const void* base, unsigned long long rows,
                     unsigned long long cols, unsigned long long ld, unsigned box_rows, bool atom32 = false) {
  const int esize = dtype == RRF_F64 ? 8 : 4;
  cuuint64_t gdim[2] = {cols, rows};
  cuuint64_t gstr[1] = {ld * (unsigned long long)esize};
  cuuint32_t box[2] = {(cuuint32_t)(128 / esize), box_rows};
  cuuint32_t estr[2] = {1, 1};
  const CUresult r = h->encode(map, dtype == RRF_F64 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT64 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32,
                               2, const_cast<void*>(base), gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                               atom32 ? CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B : CU_TENSOR_MAP_SWIZZLE_128B,
                               CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
static bool ld_ok(long long ld, long long mincols, int esize) { return ld >= mincols && (ld * esize) % 16 == 0; }
static bool b_ok(int dtype, int b) {
  if (dtype == RRF_F64) return b == 16 || b == 32 || b == 64 || b == 128;
  if (dtype == RRF_F32) return b == 32 || b == 64 || b == 128;
  return false;
}

// ------------------------------------------------------------------ typed launchers
template <typename T, int B>
struct Ops {
  static constexpr int KE = 128 / (int)sizeof(T);
  // sample (first block only)
  static constexpr int S_WM = (B == 16) ? 8 : 4, S_WN = (B == 16) ? 1 : 2;
  static constexpr int S_KBS = (B >= 128) ? 2 : 4;   // 128-byte K boxes per pipeline stage
  static constexpr int S_SMEM = kSampleStages * S_KBS * (kSampleBM + B) * 128 + 1024;
  // vtw: M = B, 8 consumer warps + 1 producer warp
  static constexpr int V_BN = (B * (int)sizeof(T) >= 1024) ? 64 : 128;
  static constexpr int V_WM = (B == 16) ? 1 : (B == 128 ? 4 : 2), V_WN = 8 / V_WM;
  static constexpr int V_STAGE = kVtwBK * (B + V_BN) * (int)sizeof(T);
  static constexpr int V_STAGES = (3 * V_STAGE + 1024 > 200 * 1024) ? 2 : (4 * V_STAGE + 1024 > 200 * 1024 ? 3 : 4);
  static constexpr int V_SMEM = V_STAGES * V_STAGE + 1024;
  static constexpr int TC_B = (B == 16) ? 32 : B;
  // vtw on tcgen05 (single precision only), W tile in tensor memory: stages of the TMA ring and of V's plane ring
  static constexpr int TC_RS = (B >= 128) ? 5 : 6, TC_OS = 2;
  static_assert(TcCfg<TC_B, TC_RS, TC_OS>::SMEM + 1024 <= kMaxSmem, "shared memory");
  // fused update: slab height 128 (64 for the widest block), two 128-byte column groups per tile
  static constexpr int U_BM = (B >= 128) ? 64 : 128;
  static constexpr int U_BNB = (sizeof(T) == 8 && B == 32) ? 4 : 2;
  static constexpr int U_WM = U_BM / 16, U_WN = 8 / U_WM;
  static constexpr int U_BN = U_BNB * KE;
  static constexpr int U_KB = B / KE;
  static constexpr int U_VBYTES = U_KB * U_BM * 128;
  static constexpr int U_STAGE = U_BNB * U_BM * 128 + U_KB * U_BN * 128 + U_BNB * B * 128;
  static constexpr int U_STAGES = (U_VBYTES + 3 * U_STAGE + 1024 <= 226 * 1024) ? 3 : 2;
  static constexpr int U_SMEM = U_VBYTES + U_STAGES * U_STAGE + 1024;
  static constexpr bool U_PW = false;   // the widest fp64 block needs the registers of 8 warps
  // fused update on tcgen05: single precision, 128-row slabs and 64-column tiles (the same as above for b <= 64)
  static constexpr bool kHasUpdTc = std::is_same<T, float>::value && B <= 64 && U_BM == kUtcBM && U_BN == kUtcBN && U_WN == 1;
  static_assert(U_SMEM + 1024 <= kMaxSmem && V_SMEM + 1024 <= kMaxSmem && S_SMEM + 1024 <= kMaxSmem, "shared memory");

  static cudaError_t setup() {
    cudaError_t e;
    e = cudaFuncSetAttribute(sample_kernel<T, B, kSampleBM, S_WM, S_WN, kSampleStages, S_KBS>,
                             cudaFuncAttributeMaxDynamicSharedMemorySize, S_SMEM);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(vtw_sk_kernel<T, B, V_BN, kVtwBK, V_WM, V_WN, V_STAGES>,
                             cudaFuncAttributeMaxDynamicSharedMemorySize, V_SMEM);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(upd_sk_kernel<T, B, U_BM, U_BNB, U_WM, U_WN, U_STAGES, U_PW>,
                             cudaFuncAttributeMaxDynamicSharedMemorySize, U_SMEM);
    if (e != cudaSuccess) return e;
    if constexpr (std::is_same<T, float>::value) {
      e = cudaFuncSetAttribute(vtw_tc_kernel<B, TC_RS, TC_OS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               TcCfg<B, TC_RS, TC_OS>::SMEM);
      if (e != cudaSuccess) return e;
    }
    if constexpr (kHasUpdTc) {
      e = cudaFuncSetAttribute(upd_tc_kernel<B>, cudaFuncAttributeMaxDynamicSharedMemorySize, UtcCfg<B>::SMEM);
      if (e != cudaSuccess) return e;
    }
    e = cudaFuncSetAttribute(tz_kernel<T, B>, cudaFuncAttributeMaxDynamicSharedMemorySize, Z_SMEM);
    return e;
  }
  static void sample(const CUtensorMap& tmW, const CUtensorMap& tmO, void* Ypart, int r0, int rows, int n, int j0,
                     const SamplePlan& p, Ctrl* ctrl, const int* only_if_zero, double* sq_part, cudaStream_t st) {
    sample_kernel<T, B, kSampleBM, S_WM, S_WN, kSampleStages, S_KBS>
        <<<std::min(p.nslabs * p.nseg, p.ctas), S_WM * S_WN * 32, S_SMEM, st>>>(tmW, tmO, (T*)Ypart, r0, rows, n, j0, p.nslabs,
                                                                                  p.nseg, p.kt_per_seg, ctrl, only_if_zero, sq_part);
  }
  static void vtw(const CUtensorMap& tmV, const CUtensorMap& tmC, void* Zpart, int r0, int cv0, const VtwPlan& p,
                  Ctrl* ctrl, cudaStream_t st) {
    if constexpr (std::is_same<T, float>::value) {
      if (p.tc) {     // the maps then have 32-row boxes
        vtw_tc_kernel<B, TC_RS, TC_OS><<<p.P, kTcThreads, TcCfg<B, TC_RS, TC_OS>::SMEM, st>>>(
            tmV, tmC, (float*)Zpart, r0, cv0, p.KT, p.total, p.tpc, p.chunk, ctrl);
        return;
      }
    }
    vtw_sk_kernel<T, B, V_BN, kVtwBK, V_WM, V_WN, V_STAGES>
        <<<p.P, 9 * 32, V_SMEM, st>>>(tmV, tmC, (T*)Zpart, r0, cv0, p.KT, p.total, p.tpc, ctrl);
  }
  static constexpr int Z_SMEM = (B * (B + 4) + B * (kTzCols + 4)) * (int)sizeof(T);
  static void tz(const void* Zpart, const VtwPlan& vp, const void* Tm, long long ldt, int transpose_t, void* Zt,
                 const int* done_flag, cudaStream_t st) {
    tz_kernel<T, B><<<vp.npad / kTzCols, kTzThreads, Z_SMEM, st>>>((const T*)Zpart, vp.bn, vp.nct, vp.KT, vp.tpc, (const T*)Tm,
                                                            ldt, transpose_t, (T*)Zt, done_flag);
  }
  static void update(const CUtensorMap& tmV, const CUtensorMap& tmZ, const CUtensorMap& tmC, const CUtensorMap& tmO,
                     void* C, long long ldc, void* top, long long ldtop, int r0, int rows, int ncols, int cv0,
                     int top_rows, int j0, void* Ypart, double* norm_part, const UpdPlan& p, Ctrl* ctrl,
                     const int* samp_flag, cudaStream_t st) {
    if constexpr (kHasUpdTc) {
      if (p.tc != nullptr) {
        const UpdTc& x = *p.tc;
        split_planes_kernel<<<std::min(1024, ceil_div((long long)x.npad * B, 256)), 256, 0, st>>>(
            (const float*)x.Zt, B, x.npad, B, (float*)x.zsplit, B, &ctrl->done);
        if (j0 >= 0)
          split_planes_kernel<<<std::min(1024, ceil_div((long long)ncols * B, 256)), 256, 0, st>>>(
              (const float*)x.Om + (size_t)j0 * x.ldom, x.ldom, B, ncols, (float*)x.osplit, x.ldo2, &ctrl->done);
        // where the updated tiles go: the working matrix, and the rows of B that this pass completes
        CUtensorMap tmCs, tmTs;
        bool maps_ok = make_map(x.h, &tmCs, RRF_F32, C, (unsigned long long)r0 + rows, ncols, ldc, 32);
        if (maps_ok && top_rows > 0) maps_ok = make_map(x.h, &tmTs, RRF_F32, top, top_rows, ncols, ldtop, 32);
        if (top_rows <= 0) tmTs = tmCs;
        if (!maps_ok) {
          // cannot happen for arguments that passed the entry checks (aligned bases, leading dimensions of whole
          // 16 bytes); if it does, the run ends with an error status instead of an update that never ran
          static const int kErr[2] = {1, (int)RRF_ERR_CUDA};     // Ctrl::done, Ctrl::status
          cudaMemcpyAsync(ctrl, kErr, sizeof(kErr), cudaMemcpyHostToDevice, st);
          return;
        }
        upd_tc_kernel<B><<<p.P, kUtcThreads, UtcCfg<B>::SMEM, st>>>(
            tmC, x.tmZs, x.tmOs, tmCs, tmTs, (const float*)x.V, x.ldv, r0, rows, ncols, cv0, top_rows, j0 >= 0 ? 1 : 0,
            x.npad, (float*)Ypart, norm_part, p.NC, p.total, p.tpc, x.chunk * kUtcYChunkFactor, ctrl);
        return;
      }
    }
    upd_sk_kernel<T, B, U_BM, U_BNB, U_WM, U_WN, U_STAGES, U_PW><<<p.P, (U_PW ? 9 : 8) * 32, U_SMEM, st>>>(
        tmV, tmZ, tmC, tmO, (T*)C, ldc, (T*)top, ldtop, r0, rows, ncols, cv0, top_rows, j0, (T*)Ypart, norm_part, p.NC,
        p.total, p.tpc, ctrl, samp_flag, p.p0, p.Lb);
  }
};

struct OpTable {
  int s_kbs, v_bn, u_bm, u_bn, u_wn, has_upd_tc;
  cudaError_t (*setup)();
  void (*sample)(const CUtensorMap&, const CUtensorMap&, void*, int, int, int, int, const SamplePlan&, Ctrl*,
                 const int*, double*, cudaStream_t);
  void (*vtw)(const CUtensorMap&, const CUtensorMap&, void*, int, int, const VtwPlan&, Ctrl*, cudaStream_t);
  void (*tz)(const void*, const VtwPlan&, const void*, long long, int, void*, const int*, cudaStream_t);
  void (*update)(const CUtensorMap&, const CUtensorMap&, const CUtensorMap&, const CUtensorMap&, void*, long long,
                 void*, long long, int, int, int, int, int, int, void*, double*, const UpdPlan&, Ctrl*, const int*,
                 cudaStream_t);
};
template <typename T, int B>
static OpTable make_ops() {
  return OpTable{Ops<T, B>::S_KBS, Ops<T, B>::V_BN, Ops<T, B>::U_BM, Ops<T, B>::U_BN, Ops<T, B>::U_WN, Ops<T, B>::kHasUpdTc ? 1 : 0, &Ops<T, B>::setup, &Ops<T, B>::sample,
                 &Ops<T, B>::vtw,  &Ops<T, B>::tz, &Ops<T, B>::update};
}
static const OpTable* get_ops(int dtype, int b) {
  static const OpTable d16 = make_ops<double, 16>(), d32 = make_ops<double, 32>(), d64 = make_ops<double, 64>(),
                       d128 = make_ops<double, 128>(), f32 = make_ops<float, 32>(), f64 = make_ops<float, 64>(),
                       f128 = make_ops<float, 128>();
  if (dtype == RRF_F64) {
    switch (b) {
      case 16: return &d16;
      case 32: return &d32;
      case 64: return &d64;
      case 128: return &d128;
    }
  } else if (dtype == RRF_F32) {
    switch (b) {
      case 32: return &f32;
      case 64: return &f64;
      case 128: return &f128;
    }
  }
  return nullptr;
}

// panel QR + T factor, enqueued on `st`
struct NoMark {
  void operator()(int, int) const {}
};
struct PanelOpts {
  PanelSource alt{};               // where the panel is if the fused update skipped sampling it ...
  const int* fused_flag = nullptr; // ... which is the case when this device word is 0 (NULL: always `src`)
  PanelFix fix{};                  // look-ahead fix-up (enabled == 0: none)
  int ctas = 0;                    // 0: one slab per SM; > 0: confine the panel to this many CTAs
  unsigned* bar_reset = nullptr;   // the T-factor kernel zeroes this word (the panel's barrier counter)
  bool merge_t = false;            // CTA 0 of the panel kernel builds T itself: no T-factor launch
  unsigned bar_base = 0;           // value of the barrier counter when this launch starts (it is not reset
                                   // between the launches of the look-ahead schedule)
  unsigned* bar_used = nullptr;    // out: what this launch adds to the counter
  cudaStream_t st_t = nullptr;     // side stream for the T factor, with its fork / join events
  cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
  bool no_cluster = false;         // keep the per-column kernel on a cooperative grid even where one cluster would hold the panel
  bool tree = false;               // b <= 64: use the tree kernel (no grid barrier per column)
  bool blocked = false;            // use the blocked kernel (micro-panels of eight columns, panel_blk.cuh) if it fits
  bool global_slab = false;        // blocked kernel: keep the slabs in global memory
  unsigned seq_base = 0;           // blocked kernel: first tag value of this launch (tags only grow within a run)
  double* csq = nullptr;           // [b][Gp]: the panel kernel leaves the column sums of squares of the panel here
  int* g_out = nullptr;            // out: CTAs of the per-column panel kernel (Gp = g rounded up to 32)
};
template <typename Mark = NoMark>
static rrf_status_t launch_panel(rrf_ctx* h, int dtype, const void* Y, PanelSource src,
                                 long long rows, int b, void* V, long long ldv, void* Tout, long long ldt,
                                 const PanelScratch& ps, Ctrl* ctrl, const int* done_flag, cudaStream_t st,
                                 Mark mark = Mark(), int step = 0, const PanelOpts& o = PanelOpts()) {
  // (a square panel goes to the per-column kernel: its last column has nothing below the pivot, for which the
  // Householder convention is H = I, tau = 0, while the reconstruction from a tree always reflects, tau = 2)
  if (b <= kTsqrMaxB && o.tree && ps.ts.Rbuf != nullptr && rows > b) {
    // tree kernel: factorisation, T factor and all, in one cooperative launch
    TreePlan tp;
    if (!plan_tree(h, rows, b, o.ctas, o.fix.enabled != 0, &tp)) return RRF_ERR_WORKSPACE;
    int rows_i = (int)rows, Rp = tp.Rp;
    PanelFix fix = o.fix;
    PanelSource alt = o.alt;
    const int* fused_flag = o.fused_flag;
    unsigned bar_base = o.bar_base;
    unsigned* bar = ps.bar;
    TsqrPlan plan = tp.t;
    TsqrScratch tsc = ps.ts;
    void* args[] = {&Y, &src, &alt, &fused_flag, &rows_i, &b, &Rp, &V, &ldv, &plan, &tsc,
                    &bar, &ctrl, &done_flag, &fix, &bar_base, &Tout, &ldt};
    if (o.bar_used != nullptr) *o.bar_used = (unsigned)tp.nbar * (unsigned)tp.ctas;
    mark(RRF_PHASE_PANEL, step);
    const void* fn = dtype == RRF_F64 ? (const void*)panel_tsqr_kernel<double> : (const void*)panel_tsqr_kernel<float>;
    const cudaError_t e = cudaLaunchCooperativeKernel(fn, dim3(tp.ctas), dim3(kPanelThreads), args, tp.smem, st);
    if (e != cudaSuccess) {
      h->last_cuda = (int)e;
      return RRF_ERR_CUDA;
    }
    if (o.ev_join != nullptr) cudaEventRecord(o.ev_join, st);   // T is ready when the panel kernel is
    return RRF_OK;
  }
  int rows_i = (int)rows;
  double *P = ps.P, *piv = ps.piv, *gram = ps.gram, *tau = ps.tau;
  unsigned* bar = ps.bar;
  PanelFix fix = o.fix;
  PanelSource alt = o.alt;
  const int* fused_flag = o.fused_flag;
  unsigned bar_base = o.bar_base;
  void* Tmerged = o.merge_t ? Tout : nullptr;
  double* csq = o.csq;
  const size_t tsmem = ((size_t)b * (b + 1) + (size_t)(b / 2) * (b / 2 + 1)) * sizeof(double);
  cudaError_t e;
  BlkPlan bp;
  // a panel too tall for shared memory goes to the blocked kernel with its slabs in global memory
  PanelPlan pp_probe;
  const bool too_tall = ps.bk.Lw != nullptr && !plan_panel(h, rows, b, &pp_probe, o.ctas, o.fix.enabled != 0) &&
                        !(o.fix.enabled && b > 64);
  const bool want_global = o.global_slab || too_tall;
  if ((o.blocked || too_tall) && ps.bk.Lw != nullptr &&
      ((!want_global && plan_blk(h, rows, b, &bp, o.ctas, o.fix.enabled != 0)) ||
       plan_blk(h, rows, b, &bp, o.ctas, o.fix.enabled != 0, true))) {
    // blocked kernel: micro-panels of eight columns, exchanges instead of grid barriers
    int R = bp.R, Rp = bp.Rp, RS = bp.RS, ksplit = bp.ksplit, c_in_smem = bp.c_in_smem;
    BlkScratch bk = ps.bk;
    unsigned seq_base = o.seq_base;
    double* gslab = bp.gslab ? ps.gslab : nullptr;
    void* args[] = {&Y, &src, &alt, &fused_flag, &rows_i, &b, &R, &Rp, &RS, &V, &ldv, &gram, &tau, &bk, &seq_base,
                    &ksplit, &c_in_smem, &bar, &ctrl, &done_flag, &fix, &bar_base, &Tmerged, &ldt, &csq, &gslab};
    size_t smem = bp.smem;
    if (o.merge_t) smem = std::max(smem, tsmem);
    if (o.bar_used != nullptr) *o.bar_used = (unsigned)(o.fix.enabled ? 2 : 0) * (unsigned)bp.G;
    if (o.g_out != nullptr) *o.g_out = bp.G;
    mark(RRF_PHASE_PANEL, step);
    const void* fn = dtype == RRF_F64 ? (const void*)panel_blk_kernel<double> : (const void*)panel_blk_kernel<float>;
    e = cudaLaunchCooperativeKernel(fn, dim3(bp.G), dim3(kPanelThreads), args, smem, st);
  } else {
    PanelPlan pp;
    const bool as_cluster = !o.no_cluster && !o.blocked && plan_panel_cl(h, rows, b, &pp, o.fix.enabled != 0);
    if (!as_cluster && !plan_panel(h, rows, b, &pp, o.ctas, o.fix.enabled != 0)) return RRF_ERR_WORKSPACE;
    int R = pp.R, Rp = pp.Rp;
    void* args[] = {&Y,   &src, &alt, &fused_flag, &rows_i, &b,    &R,    &Rp,        &V,   &ldv,      &P,
                    &piv, &gram, &tau, &bar,       &ctrl,   &done_flag, &fix, &bar_base, &Tmerged, &ldt, &csq};
    if (o.merge_t) pp.smem = std::max(pp.smem, tsmem);
    if (o.bar_used != nullptr) *o.bar_used = as_cluster ? 0u : (unsigned)(b + (o.fix.enabled ? 2 : 0)) * (unsigned)pp.G;
    if (o.g_out != nullptr) *o.g_out = pp.G;
    mark(RRF_PHASE_PANEL, step);
    if (as_cluster) {
      const void* fn = dtype == RRF_F64 ? panel_variant_cl<double>(pp.variant) : panel_variant_cl<float>(pp.variant);
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = dim3(pp.G);
      cfg.blockDim = dim3(kPanelThreads);
      cfg.dynamicSmemBytes = pp.smem;
      cfg.stream = st;
      cudaLaunchAttribute at[1];
      at[0].id = cudaLaunchAttributeClusterDimension;
      at[0].val.clusterDim.x = pp.G;
      at[0].val.clusterDim.y = 1;
      at[0].val.clusterDim.z = 1;
      cfg.attrs = at;
      cfg.numAttrs = 1;
      e = cudaLaunchKernelExC(&cfg, fn, args);
    } else {
      const void* fn = dtype == RRF_F64 ? panel_variant<double>(pp.variant) : panel_variant<float>(pp.variant);
      e = cudaLaunchCooperativeKernel(fn, dim3(pp.G), dim3(kPanelThreads), args, pp.smem, st);
    }
  }
  if (e == cudaSuccess && !o.merge_t) {
    cudaStream_t tt = st;
    if (o.ev_fork != nullptr) {          // fork: the T factor runs on the side stream after the panel
      cudaEventRecord(o.ev_fork, st);
      cudaStreamWaitEvent(o.st_t, o.ev_fork, 0);
      tt = o.st_t;
    } else {
      mark(RRF_PHASE_TFACTOR, step);
    }
    if (dtype == RRF_F64)
      tfactor_kernel<double><<<1, 256, tsmem, tt>>>(gram, tau, b, (double*)Tout, ldt, done_flag, o.bar_reset);
    else
      tfactor_kernel<float><<<1, 256, tsmem, tt>>>(gram, tau, b, (float*)Tout, ldt, done_flag, o.bar_reset);
    e = cudaGetLastError();
    if (o.ev_join != nullptr) cudaEventRecord(o.ev_join, o.st_t);
  }
  if (e != cudaSuccess) {
    h->last_cuda = (int)e;
    return RRF_ERR_CUDA;
  }
  return RRF_OK;
}

// attributes of the panel and T-factor kernels; reports the dynamic shared memory a panel may use
static cudaError_t setup_panel_kernels(int smem_optin, int* panel_smem_max, int* cluster_ok) {
  cudaError_t e;
  const void* pk[2 * kPanelVariants + 2 * kPanelVariantsCl];
  for (int q = 0; q < kPanelVariants; ++q) {
    pk[q] = panel_variant<double>(q);
    pk[kPanelVariants + q] = panel_variant<float>(q);
  }
  for (int q = 0; q < kPanelVariantsCl; ++q) {
    pk[2 * kPanelVariants + q] = panel_variant_cl<double>(q);
    pk[2 * kPanelVariants + kPanelVariantsCl + q] = panel_variant_cl<float>(q);
  }
  size_t stat = 0;
  for (const void* f : pk) {
    cudaFuncAttributes fa;
    e = cudaFuncGetAttributes(&fa, f);
    if (e != cudaSuccess) return e;
    stat = std::max(stat, fa.sharedSizeBytes);
  }
  *panel_smem_max = std::min(smem_optin, kMaxSmem) - (int)stat;
  for (const void* f : pk) {
    e = cudaFuncSetAttribute(f, cudaFuncAttributeMaxDynamicSharedMemorySize, *panel_smem_max);
    if (e != cudaSuccess) return e;
  }
  // clusters of up to kClusterMax CTAs (above the portable 8): allowed per kernel, and checked once for residency
  *cluster_ok = 1;
  for (int q = 0; q < 2 * kPanelVariantsCl; ++q) {
    if (cudaFuncSetAttribute(pk[2 * kPanelVariants + q], cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess) {
      cudaGetLastError();
      *cluster_ok = 0;
    }
  }
  if (*cluster_ok) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(kClusterMax);
    cfg.blockDim = dim3(kPanelThreads);
    cfg.dynamicSmemBytes = *panel_smem_max;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = kClusterMax;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    int nclusters = 0;
    if (cudaOccupancyMaxActiveClusters(&nclusters, pk[2 * kPanelVariants + kPanelVariantsCl - 1], &cfg) != cudaSuccess || nclusters < 1) {
      cudaGetLastError();
      *cluster_ok = 0;
    }
  }
  const int tmax = (128 * 129 + 64 * 65) * 8;
  e = cudaFuncSetAttribute(tfactor_kernel<double>, cudaFuncAttributeMaxDynamicSharedMemorySize, tmax);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(tfactor_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, tmax);
}

static cudaError_t setup_tree_kernels(int smem_optin, int* tsqr_smem_max) {
  const void* fk[2] = {(const void*)panel_tsqr_kernel<double>, (const void*)panel_tsqr_kernel<float>};
  size_t stat = 0;
  for (const void* f : fk) {
    cudaFuncAttributes fa;
    const cudaError_t e = cudaFuncGetAttributes(&fa, f);
    if (e != cudaSuccess) return e;
    stat = std::max(stat, fa.sharedSizeBytes);
  }
  *tsqr_smem_max = std::min(smem_optin, kMaxSmem) - (int)stat;
  for (const void* f : fk) {
    const cudaError_t e = cudaFuncSetAttribute(f, cudaFuncAttributeMaxDynamicSharedMemorySize, *tsqr_smem_max);
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

static cudaError_t setup_blk_kernels(int smem_optin, int* blk_smem_max) {
  const void* fk[2] = {(const void*)panel_blk_kernel<double>, (const void*)panel_blk_kernel<float>};
  size_t stat = 0;
  for (const void* f : fk) {
    cudaFuncAttributes fa;
    const cudaError_t e = cudaFuncGetAttributes(&fa, f);
    if (e != cudaSuccess) return e;
    stat = std::max(stat, fa.sharedSizeBytes);
  }
  *blk_smem_max = std::min(smem_optin, kMaxSmem) - (int)stat;
  for (const void* f : fk) {
    const cudaError_t e = cudaFuncSetAttribute(f, cudaFuncAttributeMaxDynamicSharedMemorySize, *blk_smem_max);
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

static cudaError_t setup_all(int smem_optin, int* panel_smem_max, int* cluster_ok) {
  cudaError_t e;
  for (int b : {16, 32, 64, 128}) {
    e = get_ops(RRF_F64, b)->setup();
    if (e != cudaSuccess) return e;
  }
  for (int b : {32, 64, 128}) {
    e = get_ops(RRF_F32, b)->setup();
    if (e != cudaSuccess) return e;
  }
  return setup_panel_kernels(smem_optin, panel_smem_max, cluster_ok);
}

static size_t tc_zsplit_bytes(int npad, int b) { return align_up((size_t)2 * npad * b * sizeof(float), 256); }
static size_t tc_split_bytes(int npad, int b, long long n) {
  return tc_zsplit_bytes(npad, b) + align_up((size_t)2 * b * align_up((size_t)n, 4) * sizeof(float), 256);
}

// ------------------------------------------------------------------ workspace of rrf_run
struct RunLayout {
  size_t ctrl, traces, done_after, norm_part, init_part, ypart, ypart2, zpart, zt, tcsplit, panel, look, csq, w, omega, total;
  int init_ctas, max_norm_parts;
  long long ldw;
};
constexpr int kInitCtas = 148 * 8;

static bool run_layout(const rrf_params_t* p, bool need_omega, RunLayout* L) {
  const int sms = kMaxSms;
  const int esize = p->dtype == RRF_F64 ? 8 : 4;
  const int b = p->b, steps = p->max_rank / b;
  const OpTable* ops = get_ops(p->dtype, b);
  size_t ymax = 0, zmax = 0;
  int npad = 0;
  for (int i = 0; i < steps; ++i) {
    const long long rows = p->m - (long long)i * b;
    ymax = std::max(ymax, (size_t)kSampleMaxSeg * (size_t)rows * b);   // first block only, any SM count
    const UpdPlan up = plan_upd(sms, rows, p->n, ops->u_bm, ops->u_bn, ops->u_wn);
    ymax = std::max(ymax, (size_t)(sms + up.NS) * ops->u_wn * ops->u_bm * b);   // slots <= (P + NS) * wn, P <= sms
    const VtwPlan vp = plan_vtw(sms, rows, p->n, ops->v_bn);
    zmax = std::max(zmax, (size_t)(sms + vp.nct) * b * ops->v_bn);
    npad = vp.npad;
  }
  size_t off = 0;
  L->ctrl = off; off += 256;
  L->traces = off; off += align_up(((size_t)3 * steps + 1) * sizeof(double), 256);   // E_sub, E_dir, estimates
  L->done_after = off; off += align_up((size_t)(2 * steps + 3) * sizeof(int), 256);   // + the look-ahead barrier word + samp[]
  L->init_ctas = kInitCtas;
  L->init_part = off; off += align_up((size_t)kInitCtas * sizeof(double), 256);
  L->max_norm_parts = sms;
  L->norm_part = off; off += align_up((size_t)2 * sms * sizeof(double), 256);
  L->ypart = off; off += align_up(ymax * esize, 256);
  L->ypart2 = off; off += align_up(ymax * esize, 256);   // the look-ahead schedule keeps two sampled panels
  L->zpart = off; off += align_up(zmax * esize, 256);
  L->zt = off; off += align_up((size_t)npad * b * esize, 256);
  L->tcsplit = off;      // single precision: TF32 planes of Zt and of b rows of OmegaT for the tcgen05 update
  if (ops->has_upd_tc) off += tc_split_bytes(npad, b, p->n);
  L->panel = off; off += panel_scratch_bytes(sms, b, p->m);
  L->look = off; off += look_scratch_bytes(b);
  L->csq = off; off += align_up((size_t)2 * b * ((sms + 31) / 32 * 32) * sizeof(double), 256);   // two panels in flight
  L->w = off;
  L->ldw = (long long)align_up((size_t)p->n, 16);   // rows of the working copy start on 128-byte lines
  if (!(p->flags & RRF_FLAG_INPLACE)) off += align_up((size_t)p->m * (size_t)L->ldw * esize, 256);
  L->omega = off;
  if (need_omega) off += align_up((size_t)p->max_rank * (size_t)p->n * esize, 256);
  L->total = off;
  return true;
}

static rrf_status_t check_params(const rrf_params_t* p) {
  if (p == nullptr) return RRF_ERR_INVALID_ARG;
  if (p->dtype != RRF_F64 && p->dtype != RRF_F32) return RRF_ERR_INVALID_ARG;
  if (!b_ok(p->dtype, p->b)) return RRF_ERR_INVALID_ARG;
  if (p->m < 1 || p->n < 1 || p->m > 0x7fffffffLL || p->n > 0x7fffffffLL) return RRF_ERR_INVALID_ARG;
  if (p->max_rank < p->b || p->max_rank % p->b != 0) return RRF_ERR_INVALID_ARG;
  if (p->max_rank > p->m || p->max_rank > p->n) return RRF_ERR_INVALID_ARG;
  if (!(p->tol >= 0.0)) return RRF_ERR_INVALID_ARG;
  if (p->estimator < 0 || p->estimator > 3) return RRF_ERR_INVALID_ARG;
  if (p->estimator >= 2 && (p->flags & RRF_FLAG_PANEL_TREE)) return RRF_ERR_INVALID_ARG;
  if (p->flags & RRF_FLAG_NO_UPDATE) {
    // without the update there is no residual to measure: only a sampled rule or the rank cap ends the loop
    if (p->estimator < 2 && !(p->flags & RRF_FLAG_FIXED_RANK)) return RRF_ERR_INVALID_ARG;
    if (p->flags & (RRF_FLAG_INPLACE | RRF_FLAG_PANEL_TREE | RRF_FLAG_TWO_QUEUES)) return RRF_ERR_INVALID_ARG;
  }
  if (p->tune_panel_ctas < 0 || p->tune_gate < 0 || p->tune_gate > 2) return RRF_ERR_INVALID_ARG;
  return RRF_OK;
}

}  // namespace rrf

using namespace rrf;

extern "C" {

const char* rrf_status_string(rrf_status_t s) {
  switch (s) {
    case RRF_OK: return "ok";
    case RRF_MAX_RANK_REACHED: return "rank cap reached before the tolerance";
    case RRF_ERR_INVALID_ARG: return "invalid argument";
    case RRF_ERR_WORKSPACE: return "workspace too small or panel too tall";
    case RRF_ERR_CUDA: return "CUDA error";
    case RRF_ERR_TIMEOUT: return "bounded device-side wait gave up";
    case RRF_ERR_NONFINITE: return "input contains NaN or Inf";
  }
  return "unknown status";
}

rrf_status_t rrf_create(rrf_handle_t* out, int device) {
  if (out == nullptr) return RRF_ERR_INVALID_ARG;
  *out = nullptr;
  if (cudaSetDevice(device) != cudaSuccess) return RRF_ERR_CUDA;
  rrf_ctx* h = new (std::nothrow) rrf_ctx();
  if (h == nullptr) return RRF_ERR_CUDA;
  h->device = device;
  h->last_cuda = 0;
  h->profiling = 0;
  h->aux = nullptr;
  h->cap = nullptr;
  h->graph = nullptr;
  h->gexec = nullptr;
  h->graph_off = 0;
  h->cand_steps = -1;
  h->gsteps = 0;
  h->f32_engine = 1;      // single precision runs on tcgen05 unless rrf_set_single_engine says otherwise
  h->tc_chunk = 2;
  std::memset(&h->profile, 0, sizeof(h->profile));
  cudaError_t e = cudaDeviceGetAttribute(&h->sms, cudaDevAttrMultiProcessorCount, device);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&h->smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device);
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (e == cudaSuccess) e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q);
  if (e == cudaSuccess && (fn == nullptr || q != cudaDriverEntryPointSuccess)) e = cudaErrorUnknown;
  if (e == cudaSuccess && h->sms > kMaxSms) e = cudaErrorInvalidConfiguration;
  h->encode = reinterpret_cast<EncodeTiledFn>(fn);
  if (e == cudaSuccess) e = setup_all(h->smem_optin, &h->panel_smem_max, &h->cluster_ok);
  if (e == cudaSuccess) e = setup_tree_kernels(h->smem_optin, &h->tsqr_smem_max);
  if (e == cudaSuccess) e = setup_blk_kernels(h->smem_optin, &h->blk_smem_max);
  // The side stream carries the panel chain of the look-ahead schedule, the critical path wherever that schedule is
  // chosen: its kernels (a whole thread-block cluster where the panel is short) are placed ahead of GEMM CTAs that
  // wait at the same moment.
  int prio_lo = 0, prio_hi = 0;
  if (e == cudaSuccess) e = cudaDeviceGetStreamPriorityRange(&prio_lo, &prio_hi);
  if (e == cudaSuccess) e = cudaStreamCreateWithPriority(&h->aux, cudaStreamNonBlocking, prio_hi);
  if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&h->cap, cudaStreamNonBlocking);
  if (e == cudaSuccess) e = cudaMalloc(&h->d_ctrl, sizeof(Ctrl));
  if (e == cudaSuccess) e = cudaMemset(h->d_ctrl, 0, sizeof(Ctrl));
  if (e != cudaSuccess) {
    delete h;
    return RRF_ERR_CUDA;
  }
  if (h->smem_optin > kMaxSmem) h->smem_optin = kMaxSmem;
  *out = h;
  return RRF_OK;
}

rrf_status_t rrf_destroy(rrf_handle_t h) {
  if (h == nullptr) return RRF_ERR_INVALID_ARG;
  cudaSetDevice(h->device);
  cudaFree(h->d_ctrl);
  for (cudaEvent_t ev : h->events) cudaEventDestroy(ev);
  for (cudaEvent_t ev : h->sync_events) cudaEventDestroy(ev);
  if (h->gexec != nullptr) cudaGraphExecDestroy(h->gexec);
  if (h->graph != nullptr) cudaGraphDestroy(h->graph);
  if (h->aux != nullptr) cudaStreamDestroy(h->aux);
  if (h->cap != nullptr) cudaStreamDestroy(h->cap);
  delete h;
  return RRF_OK;
}

rrf_status_t rrf_last_status(rrf_handle_t h, void* cuda_stream) {
  if (h == nullptr) return RRF_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  Ctrl c;
  if (cudaMemcpyAsync(&c, h->d_ctrl, sizeof(Ctrl), cudaMemcpyDeviceToHost, st) != cudaSuccess) return RRF_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return RRF_ERR_CUDA;
  if (c.status != 0) cudaMemsetAsync(h->d_ctrl, 0, sizeof(Ctrl), st);
  return (rrf_status_t)c.status;
}

rrf_status_t rrf_set_single_engine(rrf_handle_t h, int32_t engine, int32_t chunk_tiles) {
  if (h == nullptr || engine < 0 || engine > 1 || chunk_tiles < 0) return RRF_ERR_INVALID_ARG;
  h->f32_engine = engine;
  h->tc_chunk = chunk_tiles;
  return RRF_OK;
}

rrf_status_t rrf_set_profiling(rrf_handle_t h, int32_t enable) {
  if (h == nullptr) return RRF_ERR_INVALID_ARG;
  h->profiling = enable ? 1 : 0;
  return RRF_OK;
}

rrf_status_t rrf_get_profile(rrf_handle_t h, rrf_profile_t* out) {
  if (h == nullptr || out == nullptr) return RRF_ERR_INVALID_ARG;
  *out = h->profile;
  return RRF_OK;
}

rrf_status_t rrf_measure_peak(rrf_handle_t h, int32_t kind, double ms, double* tflops) {
  if (h == nullptr || tflops == nullptr || kind < 0 || kind > 3 || !(ms > 0.0)) return RRF_ERR_INVALID_ARG;
  if (cudaSetDevice(h->device) != cudaSuccess) return RRF_ERR_CUDA;
  double* sink = nullptr;
  const int blocks = h->sms * 2, threads = 256;
  if (cudaMalloc(&sink, sizeof(double) * blocks * threads) != cudaSuccess) return RRF_ERR_CUDA;
  cudaEvent_t e0, e1;
  cudaEventCreate(&e0);
  cudaEventCreate(&e1);
  // flops of one loop iteration of one warp
  const double per_iter = (kind == 0 || kind == 3) ? 8.0 * 2.0 * 16 * 8 * 8 : 32.0 * 16 * 2.0;
  auto run = [&](int iters) {
    cudaEventRecord(e0);
    peak_kernel<<<blocks, threads>>>(sink, iters, kind);
    cudaEventRecord(e1);
    cudaEventSynchronize(e1);
    float t = 0.f;
    cudaEventElapsedTime(&t, e0, e1);
    return (double)t;
  };
  run(1000);
  const double t1 = run(20000);
  const int iters = (int)std::min(2.0e8, std::max(20000.0, 20000.0 * ms / std::max(t1, 1e-3)));
  const double t = run(iters);
  *tflops = (double)blocks * (threads / 32) * (double)iters * per_iter / (t * 1e-3) / 1e12;
  cudaEventDestroy(e0);
  cudaEventDestroy(e1);
  cudaFree(sink);
  return cudaGetLastError() == cudaSuccess ? RRF_OK : RRF_ERR_CUDA;
}

rrf_status_t rrf_selftest_timeout(rrf_handle_t h, double limit_ms, void* cuda_stream) {
  if (h == nullptr || !(limit_ms > 0.0) || limit_ms > 1000.0) return RRF_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  if (cudaMemsetAsync(&h->d_ctrl->bar, 0, sizeof(unsigned), st) != cudaSuccess) return RRF_ERR_CUDA;
  timeout_selftest_kernel<<<1, 32, 0, st>>>(&h->d_ctrl->bar, h->d_ctrl, (long long)(limit_ms * 2.0e6));
  return cudaGetLastError() == cudaSuccess ? RRF_OK : RRF_ERR_CUDA;
}

rrf_status_t rrf_workspace_bytes(const rrf_params_t* p, size_t* bytes) {
  if (bytes == nullptr) return RRF_ERR_INVALID_ARG;
  const rrf_status_t s = check_params(p);
  if (s != RRF_OK) return s;
  RunLayout L;
  run_layout(p, true, &L);
  *bytes = L.total;
  return RRF_OK;
}

rrf_status_t rrf_fill_omega(rrf_handle_t h, int32_t dtype, uint64_t seed, int64_t n, int32_t nvec, int32_t first_vec,
                            void* dOmegaT, int64_t ldo, void* cuda_stream) {
  if (h == nullptr || dOmegaT == nullptr || n < 1 || nvec < 1 || first_vec < 0 || ldo < n) return RRF_ERR_INVALID_ARG;
  if (dtype != RRF_F64 && dtype != RRF_F32) return RRF_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  const long long total = ((n + 1) / 2) * nvec;
  const int grid = (int)std::min<long long>((total + 255) / 256, (long long)h->sms * 16);
  if (dtype == RRF_F64)
    omega_kernel<double><<<grid, 256, 0, st>>>((double*)dOmegaT, ldo, n, nvec, first_vec, seed);
  else
    omega_kernel<float><<<grid, 256, 0, st>>>((float*)dOmegaT, ldo, n, nvec, first_vec, seed);
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) {
    h->last_cuda = (int)e;
    return RRF_ERR_CUDA;
  }
  return RRF_OK;
}

rrf_status_t rrf_panel_workspace_bytes(int32_t dtype, int64_t rows, int32_t b, size_t* bytes) {
  if (bytes == nullptr || !b_ok(dtype, b) || rows < b) return RRF_ERR_INVALID_ARG;
  *bytes = panel_scratch_bytes(kMaxSms, b, rows);
  return RRF_OK;
}

static rrf_status_t panel_qr_entry(rrf_handle_t h, int32_t dtype, int64_t rows, int32_t b, const void* dY, int64_t ldy,
                                   void* dV, int64_t ldv, void* dT, int64_t ldt, void* d_workspace,
                                   size_t workspace_bytes, void* cuda_stream, bool tree, bool blocked = false) {
  if (h == nullptr || dY == nullptr || dV == nullptr || dT == nullptr || d_workspace == nullptr)
    return RRF_ERR_INVALID_ARG;
  if (!b_ok(dtype, b) || rows < b || rows > 0x7fffffffLL || ldy < b || ldv < b || ldt < b || ldy > 0x7fffffffLL)
    return RRF_ERR_INVALID_ARG;
  if (tree && b > kTsqrMaxB) return RRF_ERR_INVALID_ARG;
  if (workspace_bytes < panel_scratch_bytes(kMaxSms, b, rows)) return RRF_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  PanelScratch ps = carve_panel((unsigned char*)d_workspace, h->sms, b);
  if (cudaMemsetAsync(ps.bar, 0, sizeof(unsigned), st) != cudaSuccess) return RRF_ERR_CUDA;
  if (cudaMemsetAsync(ps.blk_tags, 0, ps.blk_tag_bytes, st) != cudaSuccess) return RRF_ERR_CUDA;
  PanelSource src{};
  src.slots = 0;
  src.nseg = 1;
  src.seg_stride = 0;
  src.ldy = (int)ldy;
  PanelOpts po;
  po.tree = tree;
  po.blocked = blocked;
  return launch_panel(h, dtype, dY, src, rows, b, dV, ldv, dT, ldt, ps, h->d_ctrl, &h->d_ctrl->done, st, NoMark(), 0, po);
}

rrf_status_t rrf_panel_qr(rrf_handle_t h, int32_t dtype, int64_t rows, int32_t b, const void* dY, int64_t ldy,
                          void* dV, int64_t ldv, void* dT, int64_t ldt, void* d_workspace, size_t workspace_bytes,
                          void* cuda_stream) {
  return panel_qr_entry(h, dtype, rows, b, dY, ldy, dV, ldv, dT, ldt, d_workspace, workspace_bytes, cuda_stream, false);
}

rrf_status_t rrf_panel_qr_blocked(rrf_handle_t h, int32_t dtype, int64_t rows, int32_t b, const void* dY, int64_t ldy,
                                 void* dV, int64_t ldv, void* dT, int64_t ldt, void* d_workspace,
                                 size_t workspace_bytes, void* cuda_stream) {
  return panel_qr_entry(h, dtype, rows, b, dY, ldy, dV, ldv, dT, ldt, d_workspace, workspace_bytes, cuda_stream, false, true);
}

rrf_status_t rrf_panel_qr_tree(rrf_handle_t h, int32_t dtype, int64_t rows, int32_t b, const void* dY, int64_t ldy,
                               void* dV, int64_t ldv, void* dT, int64_t ldt, void* d_workspace,
                               size_t workspace_bytes, void* cuda_stream) {
  return panel_qr_entry(h, dtype, rows, b, dY, ldy, dV, ldv, dT, ldt, d_workspace, workspace_bytes, cuda_stream, true);
}

// ---- building blocks of the column-sharded variant: sample one panel, squared Frobenius norm
rrf_status_t rrf_sample_workspace_bytes(int32_t dtype, int64_t rows, int32_t b, size_t* bytes) {
  if (bytes == nullptr || !b_ok(dtype, b) || rows < 1) return RRF_ERR_INVALID_ARG;
  const int esize = dtype == RRF_F64 ? 8 : 4;
  *bytes = align_up((size_t)kSampleMaxSeg * (size_t)rows * b * esize, 256) + 256;
  return RRF_OK;
}

rrf_status_t rrf_sample_panel(rrf_handle_t h, int32_t dtype, int64_t rows, int64_t n, int32_t b, const void* dC,
                              int64_t ldc, const void* dOmegaT, int64_t ldo, void* dY, void* d_workspace,
                              size_t workspace_bytes, void* cuda_stream) {
  if (h == nullptr || dC == nullptr || dOmegaT == nullptr || dY == nullptr || d_workspace == nullptr)
    return RRF_ERR_INVALID_ARG;
  const int esize = dtype == RRF_F64 ? 8 : 4;
  if (!b_ok(dtype, b) || rows < 1 || n < 1 || rows > 0x7fffffffLL || n > 0x7fffffffLL) return RRF_ERR_INVALID_ARG;
  if (!ld_ok(ldc, n, esize) || !ld_ok(ldo, n, esize) || !aligned16(dC) || !aligned16(dOmegaT)) return RRF_ERR_INVALID_ARG;
  size_t need = 0;
  rrf_sample_workspace_bytes(dtype, rows, b, &need);
  if (workspace_bytes < need || (reinterpret_cast<uintptr_t>(d_workspace) & 255u)) return RRF_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  const OpTable* ops = get_ops(dtype, b);
  CUtensorMap tmC, tmO;
  if (!make_map(h, &tmC, dtype, dC, rows, n, ldc, kSampleBM) || !make_map(h, &tmO, dtype, dOmegaT, b, n, ldo, b))
    return RRF_ERR_INVALID_ARG;
  const SamplePlan sp = plan_sample(h->sms, rows, n, esize, ops->s_kbs);
  ops->sample(tmC, tmO, d_workspace, 0, (int)rows, (int)n, 0, sp, h->d_ctrl, nullptr, nullptr, st);
  const int grid = (int)std::min<long long>((rows * b + 255) / 256, (long long)h->sms * 8);
  if (dtype == RRF_F64)
    panel_sum_kernel<double><<<grid, 256, 0, st>>>((const double*)d_workspace, sp.nseg, rows * b, rows, b, (double*)dY, h->d_ctrl);
  else
    panel_sum_kernel<float><<<grid, 256, 0, st>>>((const float*)d_workspace, sp.nseg, rows * b, rows, b, (float*)dY, h->d_ctrl);
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) {
    h->last_cuda = (int)e;
    return RRF_ERR_CUDA;
  }
  return RRF_OK;
}

rrf_status_t rrf_frobenius_sq(rrf_handle_t h, int32_t dtype, int64_t rows, int64_t cols, const void* dC, int64_t ldc,
                       double* d_out, void* d_workspace, size_t workspace_bytes, void* cuda_stream) {
  if (h == nullptr || d_out == nullptr || d_workspace == nullptr || rows < 0 || cols < 1 || ldc < cols) return RRF_ERR_INVALID_ARG;
  if (dtype != RRF_F64 && dtype != RRF_F32) return RRF_ERR_INVALID_ARG;
  if (rows > 0 && dC == nullptr) return RRF_ERR_INVALID_ARG;
  const int grid = h->sms * 4;
  if (workspace_bytes < (size_t)grid * sizeof(double)) return RRF_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  double* part = (double*)d_workspace;
  if (dtype == RRF_F64)
    frob2_part_kernel<double><<<grid, 256, 0, st>>>((const double*)dC, ldc, rows, cols, part);
  else
    frob2_part_kernel<float><<<grid, 256, 0, st>>>((const float*)dC, ldc, rows, cols, part);
  frob2_final_kernel<<<1, 256, 0, st>>>(part, grid, d_out);
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) {
    h->last_cuda = (int)e;
    return RRF_ERR_CUDA;
  }
  return RRF_OK;
}

rrf_status_t rrf_apply_workspace_bytes(int32_t dtype, int64_t m, int64_t ncols, int32_t b, size_t* bytes) {
  if (bytes == nullptr || !b_ok(dtype, b) || m < b || ncols < 1) return RRF_ERR_INVALID_ARG;
  const int esize = dtype == RRF_F64 ? 8 : 4;
  const VtwPlan vp = plan_vtw(kMaxSms, m, ncols, get_ops(dtype, b)->v_bn);
  const size_t zslots = (size_t)(kMaxSms + vp.nct) * b * vp.bn;
  *bytes = align_up((size_t)vp.npad * b * esize, 256) + align_up(zslots * esize, 256);
  if (get_ops(dtype, b)->has_upd_tc) *bytes += tc_zsplit_bytes(vp.npad, b);
  return RRF_OK;
}

}  // extern "C"

namespace rrf {

// C <- Q^T C (forward over the blocks, T^T) or C <- Q C (backward, T).
static rrf_status_t apply_blocks(rrf_handle_t h, int dtype, long long m, int b, int k, const void* dV, long long ldv,
                                 const void* dT, long long ldt, void* dC, long long ldc, long long ncols,
                                 void* d_workspace, size_t workspace_bytes, cudaStream_t st, bool transpose) {
  if (h == nullptr || dV == nullptr || dT == nullptr || dC == nullptr || d_workspace == nullptr)
    return RRF_ERR_INVALID_ARG;
  const int esize = dtype == RRF_F64 ? 8 : 4;
  if (!b_ok(dtype, b) || k < 0 || k % b != 0 || k > m || m > 0x7fffffffLL || ncols < 1 || ncols > 0x7fffffffLL)
    return RRF_ERR_INVALID_ARG;
  if (!ld_ok(ldv, k, esize) || !ld_ok(ldc, ncols, esize) || ldt < k || !aligned16(dV) || !aligned16(dC))
    return RRF_ERR_INVALID_ARG;
  size_t need = 0;
  if (rrf_apply_workspace_bytes(dtype, m, ncols, b, &need) != RRF_OK) return RRF_ERR_INVALID_ARG;
  if (workspace_bytes < need || (reinterpret_cast<uintptr_t>(d_workspace) & 255u)) return RRF_ERR_WORKSPACE;
  if (k == 0) return RRF_OK;
  const OpTable* ops = get_ops(dtype, b);
  const VtwPlan vp0 = plan_vtw(kMaxSms, m, ncols, ops->v_bn);
  unsigned char* ws = (unsigned char*)d_workspace;
  void* Zt = ws;
  void* Zpart = ws + align_up((size_t)vp0.npad * b * esize, 256);
  CUtensorMap tmV_k, tmC_k, tmV_u, tmC_u, tmZ;
  const bool tc = dtype == RRF_F32 && h->f32_engine == 1;
  const unsigned kbox = tc ? kTcSub : kVtwBK;     // rows of a TMA box of the V^T C kernel in use
  if (!make_map(h, &tmV_k, dtype, dV, m, k, ldv, kbox, tc) || !make_map(h, &tmC_k, dtype, dC, m, ncols, ldc, kbox, tc) ||
      !make_map(h, &tmV_u, dtype, dV, m, k, ldv, ops->u_bm) || !make_map(h, &tmC_u, dtype, dC, m, ncols, ldc, ops->u_bm) ||
      !make_map(h, &tmZ, dtype, Zt, vp0.npad, b, b, ops->u_bn))
    return RRF_ERR_INVALID_ARG;
  UpdTc utc{};
  const bool utc_on = tc && ops->has_upd_tc;
  if (utc_on) {
    utc.h = h;
    utc.V = dV;
    utc.ldv = ldv;
    utc.Zt = Zt;
    utc.npad = vp0.npad;
    utc.zsplit = (unsigned char*)Zpart + align_up((size_t)(kMaxSms + vp0.nct) * b * vp0.bn * esize, 256);
    utc.chunk = h->tc_chunk;
    if (!make_map(h, &utc.tmZs, dtype, utc.zsplit, 2ull * vp0.npad, b, b, kUtcBN)) return RRF_ERR_INVALID_ARG;
    utc.tmOs = utc.tmZs;   // not read: nothing is sampled here
  }
  const int nblk = k / b;
  for (int q = 0; q < nblk; ++q) {
    const int l = transpose ? q : nblk - 1 - q;
    const int r0 = l * b, rows = (int)(m - r0);
    VtwPlan vp = plan_vtw(h->sms, rows, ncols, ops->v_bn);
    vp.tc = tc;
    vp.chunk = h->tc_chunk;
    ops->vtw(tmV_k, tmC_k, Zpart, r0, r0, vp, h->d_ctrl, st);
    ops->tz(Zpart, vp, (const char*)dT + (size_t)r0 * esize, ldt, transpose ? 1 : 0, Zt, &h->d_ctrl->done, st);
    UpdPlan up = plan_upd(h->sms, rows, ncols, ops->u_bm, ops->u_bn, ops->u_wn);
    if (utc_on) up.tc = &utc;
    ops->update(tmV_u, tmZ, tmC_u, tmC_u, dC, ldc, dC, ldc, r0, rows, (int)ncols, r0, 0, -1, nullptr, nullptr, up,
                h->d_ctrl, nullptr, st);
  }
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) {
    h->last_cuda = (int)e;
    return RRF_ERR_CUDA;
  }
  return RRF_OK;
}

}  // namespace rrf

extern "C" {

rrf_status_t rrf_apply_qt(rrf_handle_t h, int32_t dtype, int64_t m, int32_t b, int32_t k, const void* dV, int64_t ldv,
                          const void* dT, int64_t ldt, void* dC, int64_t ldc, int64_t ncols, void* d_workspace,
                          size_t workspace_bytes, void* cuda_stream) {
  return apply_blocks(h, dtype, m, b, k, dV, ldv, dT, ldt, dC, ldc, ncols, d_workspace, workspace_bytes,
                      (cudaStream_t)cuda_stream, true);
}

rrf_status_t rrf_apply_q(rrf_handle_t h, int32_t dtype, int64_t m, int32_t b, int32_t k, const void* dV, int64_t ldv,
                         const void* dT, int64_t ldt, void* dC, int64_t ldc, int64_t ncols, void* d_workspace,
                         size_t workspace_bytes, void* cuda_stream) {
  return apply_blocks(h, dtype, m, b, k, dV, ldv, dT, ldt, dC, ldc, ncols, d_workspace, workspace_bytes,
                      (cudaStream_t)cuda_stream, false);
}

rrf_status_t rrf_form_q(rrf_handle_t h, int32_t dtype, int64_t m, int32_t b, int32_t k, const void* dV, int64_t ldv,
                        const void* dT, int64_t ldt, void* dQ, int64_t ldq, void* d_workspace, size_t workspace_bytes,
                        void* cuda_stream) {
  if (h == nullptr || dQ == nullptr || k < 1 || m < k || ldq < k) return RRF_ERR_INVALID_ARG;
  if (dtype != RRF_F64 && dtype != RRF_F32) return RRF_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  const int grid = (int)std::min<long long>(((long long)m * k + 255) / 256, (long long)h->sms * 16);
  if (dtype == RRF_F64)
    eye_kernel<double><<<grid, 256, 0, st>>>((double*)dQ, ldq, m, k);
  else
    eye_kernel<float><<<grid, 256, 0, st>>>((float*)dQ, ldq, m, k);
  return apply_blocks(h, dtype, m, b, k, dV, ldv, dT, ldt, dQ, ldq, k, d_workspace, workspace_bytes, st, false);
}

rrf_status_t rrf_transfer_workspace_bytes(int32_t dtype, int64_t m, int64_t ncols, int32_t b, size_t* bytes) {
  size_t apply = 0;
  const rrf_status_t s = rrf_apply_workspace_bytes(dtype, m, ncols, b, &apply);
  if (s != RRF_OK) return s;
  const int esize = dtype == RRF_F64 ? 8 : 4;
  *bytes = align_up((size_t)m * align_up((size_t)ncols, 16) * esize, 256) + apply;
  return RRF_OK;
}

rrf_status_t rrf_subspace_transfer(rrf_handle_t h, int32_t dtype, int64_t m, int32_t b, int32_t k_old,
                                   const void* dV_old, int64_t ldv_old, const void* dT_old, int64_t ldt_old,
                                   int32_t k_new, const void* dV_new, int64_t ldv_new, const void* dT_new,
                                   int64_t ldt_new, const void* dM, int64_t ldm, int64_t ncols, void* dMout,
                                   int64_t ldmo, void* d_workspace, size_t workspace_bytes, void* cuda_stream) {
  if (h == nullptr || dM == nullptr || dMout == nullptr || d_workspace == nullptr) return RRF_ERR_INVALID_ARG;
  if (!b_ok(dtype, b) || k_old < 1 || k_new < 1 || k_old > m || k_new > m || ncols < 1 || ldm < ncols || ldmo < ncols)
    return RRF_ERR_INVALID_ARG;
  size_t need = 0;
  if (rrf_transfer_workspace_bytes(dtype, m, ncols, b, &need) != RRF_OK) return RRF_ERR_INVALID_ARG;
  if (workspace_bytes < need || (reinterpret_cast<uintptr_t>(d_workspace) & 255u)) return RRF_ERR_WORKSPACE;
  const int esize = dtype == RRF_F64 ? 8 : 4;
  const long long ldc = (long long)align_up((size_t)ncols, 16);
  const size_t cbytes = align_up((size_t)m * ldc * esize, 256);
  unsigned char* ws = (unsigned char*)d_workspace;
  void* Cm = ws;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  const int grid = (int)std::min<long long>(((long long)m * ncols + 255) / 256, (long long)h->sms * 16);
  if (dtype == RRF_F64)
    copy_rows_kernel<double><<<grid, 256, 0, st>>>((double*)Cm, ldc, (const double*)dM, ldm, k_old, m, ncols);
  else
    copy_rows_kernel<float><<<grid, 256, 0, st>>>((float*)Cm, ldc, (const float*)dM, ldm, k_old, m, ncols);
  rrf_status_t s = apply_blocks(h, dtype, m, b, k_old, dV_old, ldv_old, dT_old, ldt_old, Cm, ldc, ncols, ws + cbytes,
                                workspace_bytes - cbytes, st, false);
  if (s != RRF_OK) return s;
  s = apply_blocks(h, dtype, m, b, k_new, dV_new, ldv_new, dT_new, ldt_new, Cm, ldc, ncols, ws + cbytes,
                   workspace_bytes - cbytes, st, true);
  if (s != RRF_OK) return s;
  const int grid2 = (int)std::min<long long>(((long long)k_new * ncols + 255) / 256, (long long)h->sms * 16);
  if (dtype == RRF_F64)
    copy_rows_kernel<double><<<grid2, 256, 0, st>>>((double*)dMout, ldmo, (const double*)Cm, ldc, k_new, k_new, ncols);
  else
    copy_rows_kernel<float><<<grid2, 256, 0, st>>>((float*)dMout, ldmo, (const float*)Cm, ldc, k_new, k_new, ncols);
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) {
    h->last_cuda = (int)e;
    return RRF_ERR_CUDA;
  }
  return RRF_OK;
}

rrf_status_t rrf_run(rrf_handle_t h, const rrf_params_t* p, void* dA, int64_t lda, const void* dOmegaT, int64_t ldo,
                     void* dV, int64_t ldv, void* dT, void* dB, int64_t ldb, void* d_workspace, size_t workspace_bytes,
                     void* cuda_stream, rrf_result_t* out, double* h_E_sub_trace, double* h_E_dir_trace,
                     double* h_E_est_trace) {
  if (out == nullptr) return RRF_ERR_INVALID_ARG;
  std::memset(out, 0, sizeof(*out));
  auto fail = [&](rrf_status_t s) {
    out->status = s;
    return s;
  };
  if (h == nullptr) return fail(RRF_ERR_INVALID_ARG);
  rrf_status_t s = check_params(p);
  if (s != RRF_OK) return fail(s);
  const int esize = p->dtype == RRF_F64 ? 8 : 4;
  const int b = p->b;
  const long long m = p->m, n = p->n;
  const bool unchanged = (p->flags & RRF_FLAG_NO_UPDATE) != 0;     // A is never updated, B is not produced
  if (dA == nullptr || dV == nullptr || dT == nullptr || (dB == nullptr && !unchanged) || d_workspace == nullptr)
    return fail(RRF_ERR_INVALID_ARG);
  if (!ld_ok(lda, n, esize) || !ld_ok(ldv, p->max_rank, esize) || (dB != nullptr && !ld_ok(ldb, n, esize)))
    return fail(RRF_ERR_INVALID_ARG);
  if (dOmegaT != nullptr && (!ld_ok(ldo, n, esize) || !aligned16(dOmegaT))) return fail(RRF_ERR_INVALID_ARG);
  if (!aligned16(dA) || !aligned16(dV) || (dB != nullptr && !aligned16(dB)) || (reinterpret_cast<uintptr_t>(d_workspace) & 255u))
    return fail(RRF_ERR_INVALID_ARG);
  RunLayout L;
  run_layout(p, dOmegaT == nullptr, &L);
  if (workspace_bytes < L.total) return fail(RRF_ERR_WORKSPACE);
  // Schedule.  Two queues (look-ahead) when the tallest panel fits in the shared memory of a small
  // share of the SMs, so that confining the panel there costs the GEMM kernels little; else one queue.
  const int steps_total = p->max_rank / b;
  // the tree panel kernel is opt-in: it is the slower of the two on every size measured so far
  const bool tree = (p->flags & RRF_FLAG_PANEL_TREE) != 0 && b <= kTsqrMaxB;
  const bool blocked = (p->flags & RRF_FLAG_PANEL_BLOCKED) != 0;
  int look_ctas = 0;
  bool look_cl = false;
  PanelPlan pcl_probe, pcl_probe0;
  if (blocked && !tree) {
    // opt-in blocked panel kernel: under look-ahead (only if asked for) the panel is confined to a few SMs, its
    // slabs in global memory when shared memory does not hold them
    if ((p->flags & RRF_FLAG_TWO_QUEUES) && steps_total >= 2 && b <= 64 && !unchanged)
      look_ctas = p->tune_panel_ctas > 0 ? std::min((int)p->tune_panel_ctas, h->sms / 3) : 12;
  } else if (tree) {
    TreePlan tl;
    const int cap = std::min(kLookMaxCtas, h->sms / 3);
    const int lim = p->tune_panel_ctas > 0 ? std::min(cap, (int)p->tune_panel_ctas) : cap;
    if ((p->flags & RRF_FLAG_TWO_QUEUES) && steps_total >= 2 && plan_tree(h, m, b, lim, true, &tl)) look_ctas = tl.ctas;
    if (look_ctas == 0 && !plan_tree(h, m, b, 0, false, &tl)) return fail(RRF_ERR_WORKSPACE);
  } else if (!(p->flags & RRF_FLAG_ONE_QUEUE) && !unchanged && steps_total >= 2 && plan_panel_cl(h, m - b, b, &pcl_probe, true) &&
             plan_panel_cl(h, m, b, &pcl_probe0, false)) {
    // every panel of the chain fits one thread-block cluster (the first as it is, the later ones with the b rows
    // of the fix-up): the chain takes only that many SMs
    const PassModel pm{h->sms, (double)m, (double)n, b, p->dtype == RRF_F64, p->dtype == RRF_F32 && h->f32_engine == 1, true};
    const double t = std::min(pm.step_ungated(kClusterMax), pm.step_gated(kClusterMax));
    if ((p->flags & RRF_FLAG_TWO_QUEUES) || t < pm.step_serial()) {
      // A cluster needs its SMs inside one GPC, and where the GEMM kernels' CTAs land cannot be chosen: with exactly
      // the cluster's SMs kept free the panel often waits for a GEMM kernel to drain.  Where the panel chain is the
      // critical path the GEMM kernels therefore leave 44 SMs free (measured on 4096 x 11008 fp32: 2.61 ms against
      // 2.69 with 16, 2.67 with 20, 2.72 with 32); where the GEMMs are, they get every SM the cluster does not
      // take (4096 x 4096 fp64, b = 32: 2.51 ms with 16 against 2.88 with 44).
      const int gcl = std::max(pcl_probe.G, pcl_probe0.G);
      const bool chain_critical = pm.panel_chain(gcl) > (pm.vtw() + pm.upd()) * pm.scale(gcl);
      const int keep = chain_critical ? std::max(gcl, std::min(44, h->sms / 3)) : gcl;
      look_ctas = p->tune_panel_ctas > 0 ? std::max(gcl, std::min((int)p->tune_panel_ctas, h->sms / 3)) : keep;
      look_cl = true;
    }
  } else if (!(p->flags & RRF_FLAG_ONE_QUEUE) && !unchanged && steps_total >= 2) {
    const int fewest = panel_min_ctas(h, m, b);
    const int cap = std::min(kLookMaxCtas, h->sms / 3);
    if (fewest > 0 && fewest <= cap) {
      const PassModel pm{h->sms, (double)m, (double)n, b, p->dtype == RRF_F64, p->dtype == RRF_F32 && h->f32_engine == 1, false};
      int best = fewest;
      double best_t = std::min(pm.step_ungated(fewest), pm.step_gated(fewest));
      for (int c = fewest + 1; c <= cap; ++c) {
        const double t = std::min(pm.step_ungated(c), pm.step_gated(c));
        if (t < best_t * 0.995) {
          best_t = t;
          best = c;
        }
      }
      if (p->tune_panel_ctas > 0) best = std::min(cap, std::max(fewest, (int)p->tune_panel_ctas));
      PanelPlan ppl;
      const bool wanted = (p->flags & RRF_FLAG_TWO_QUEUES) || best_t < pm.step_serial();
      if (wanted && plan_panel(h, m, b, &ppl, best, true)) look_ctas = best;
    }
  }
  // (a panel too tall for shared memory is factored by the blocked kernel with its slabs in global memory)

  cudaStream_t const user_st = (cudaStream_t)cuda_stream;
  cudaStream_t st = user_st;
  if (cudaSetDevice(h->device) != cudaSuccess) return fail(RRF_ERR_CUDA);
  unsigned char* ws = (unsigned char*)d_workspace;
  Ctrl* ctrl = reinterpret_cast<Ctrl*>(ws + L.ctrl);
  const int steps = p->max_rank / b;
  // Block steps the launch sequence holds.  A graph captured for a call that repeats the previous one holds only as
  // many as that one needed (plus one): the passes after the stop, whose kernels start and return, are then not
  // launched at all.  Should the data have changed so that the loop is still open at the end, the call is run again
  // in full (which is why an in-place run, whose input is gone by then, always holds every pass).
  int steps_run = steps;
  double* tr_sub = reinterpret_cast<double*>(ws + L.traces);
  double* tr_dir = tr_sub + steps;
  double* tr_est = tr_dir + steps;                   // [steps + 1]
  const bool sampled = p->estimator >= 2;
  double* csq0 = reinterpret_cast<double*>(ws + L.csq);
  const int csq_gp = (h->sms + 31) / 32 * 32;
  auto csq_buf = [&](int i) { return csq0 + (size_t)(i & 1) * b * csq_gp; };
  int* done_after = reinterpret_cast<int*>(ws + L.done_after);
  unsigned* look_bar = reinterpret_cast<unsigned*>(done_after + steps + 1);
  int* samp = done_after + steps + 2;   // [steps + 1]: does the update of pass q sample a later panel
  // Sampling predictor (see stop_kernel): worth its one skipped-kernel launch per pass only where a pass is
  // long, i.e. where the sample it can save is worth more than those launches cost.
  int predict = 1;
  const bool predictor_built = b < 128 && p->dtype == RRF_F64;   // see upd_sk_kernel
  if (!predictor_built) {
    predict = 1;
  } else if (p->flags & RRF_FLAG_SAMPLE_NEVER) {
    predict = 2;
  } else if (!(p->flags & RRF_FLAG_SAMPLE_ALWAYS) && !(p->flags & RRF_FLAG_FIXED_RANK)) {
    const PassModel pm{h->sms, (double)m, (double)n, b, p->dtype == RRF_F64, false, false};
    if (pm.vtw() + pm.upd() > 600.0) predict = 0;
  }
  const bool predicting = predict != 1;
  double* look_G = reinterpret_cast<double*>(ws + L.look);
  double* init_part = reinterpret_cast<double*>(ws + L.init_part);
  double* norm_part = reinterpret_cast<double*>(ws + L.norm_part);
  void* Ypart = ws + L.ypart;
  void* Zpart = ws + L.zpart;
  void* Zt = ws + L.zt;
  PanelScratch ps = carve_panel(ws + L.panel, h->sms, b);
  ps.bar = &ctrl->bar;
  const bool inplace = (p->flags & RRF_FLAG_INPLACE) != 0;
  const bool fixed = (p->flags & RRF_FLAG_FIXED_RANK) != 0;
  std::vector<std::pair<int, int>> marks;   // profiling: (phase, block step) of every recorded event
  size_t nev = 0;
  bool capturing = false;
  // Everything rrf_run puts on the device, on stream `st` (and the side stream, forked from and joined
  // back to it): enqueued directly, or recorded into a CUDA graph.
  auto enqueue = [&]() -> rrf_status_t {
  if (look_ctas > 0 && cudaMemsetAsync(look_bar, 0, sizeof(unsigned), st) != cudaSuccess) return RRF_ERR_CUDA;
  if (cudaMemsetAsync(ps.blk_tags, 0, ps.blk_tag_bytes, st) != cudaSuccess) return RRF_ERR_CUDA;   // exchange tags of the blocked panel kernel
  void* W = inplace ? dA : (void*)(ws + L.w);
  const long long ldw = inplace ? lda : L.ldw;
  const void* Om = dOmegaT;
  long long ldom = ldo;
  if (Om == nullptr) {
    Om = ws + L.omega;
    ldom = n;
    s = rrf_fill_omega(h, p->dtype, p->seed, n, p->max_rank, 0, ws + L.omega, n, st);
    if (s != RRF_OK) return s;
  }
  const OpTable* ops = get_ops(p->dtype, b);
  const int npad = plan_vtw(h->sms, m, n, ops->v_bn).npad;
  // Pass 0 reads A itself and writes W (no copy W <- A): the first panels are sampled from A, V_0^T A is taken
  // from A, and the update of pass 0 loads its tiles from A and stores them to W.
  CUtensorMap tmW_s, tmA_s, tmA_k, tmA_u, tmO, tmV_k, tmW_k, tmV_u, tmW_u, tmZ;
  const bool tc = p->dtype == RRF_F32 && h->f32_engine == 1;
  const unsigned kbox = tc ? kTcSub : kVtwBK;     // rows of a TMA box of the V^T W kernel in use
  if (!make_map(h, &tmA_s, p->dtype, dA, m, n, lda, kSampleBM) || !make_map(h, &tmA_k, p->dtype, dA, m, n, lda, kbox, tc) ||
      !make_map(h, &tmA_u, p->dtype, dA, m, n, lda, ops->u_bm) ||
      !make_map(h, &tmW_s, p->dtype, W, m, n, ldw, kSampleBM) ||
      !make_map(h, &tmO, p->dtype, Om, p->max_rank, n, ldom, b) ||
      !make_map(h, &tmV_k, p->dtype, dV, m, p->max_rank, ldv, kbox, tc) ||
      !make_map(h, &tmW_k, p->dtype, W, m, n, ldw, kbox, tc) ||
      !make_map(h, &tmV_u, p->dtype, dV, m, p->max_rank, ldv, ops->u_bm) ||
      !make_map(h, &tmW_u, p->dtype, W, m, n, ldw, ops->u_bm) ||
      !make_map(h, &tmZ, p->dtype, Zt, npad, b, b, ops->u_bn))
    return RRF_ERR_INVALID_ARG;
  UpdTc utc{};
  const bool utc_on = tc && ops->has_upd_tc;
  if (utc_on) {
    utc.h = h;
    utc.V = dV;
    utc.ldv = ldv;
    utc.Zt = Zt;
    utc.npad = npad;
    utc.Om = Om;
    utc.ldom = ldom;
    utc.zsplit = ws + L.tcsplit;
    utc.osplit = ws + L.tcsplit + tc_zsplit_bytes(npad, b);
    utc.ldo2 = (long long)align_up((size_t)n, 4);
    utc.chunk = h->tc_chunk;
    if (!make_map(h, &utc.tmZs, p->dtype, utc.zsplit, 2ull * npad, b, b, kUtcBN) ||
        !make_map(h, &utc.tmOs, p->dtype, utc.osplit, 2ull * b, n, utc.ldo2, b))
      return RRF_ERR_INVALID_ARG;
  }

  // profiling: one event before every kernel, tagged with (phase, block step)
  bool nvtx_open = false;
  auto mark = [&](int phase, int step) {
    RRF_NVTX_MARK(nvtx_open, phase, step);
    if (!h->profiling) return;
    if (nev == h->events.size()) {
      cudaEvent_t ev;
      if (cudaEventCreate(&ev) != cudaSuccess) return;
      h->events.push_back(ev);
    }
    cudaEventRecordWithFlags(h->events[nev++], st, capturing ? cudaEventRecordExternal : cudaEventRecordDefault);
    marks.emplace_back(phase, step);
  };

  // Algorithm 2 lines 1-4.  V <- 0 and the loop state are memsets; ||A||_F^2 is summed by the first sample
  // kernel, which reads all of A anyway, and W <- A never happens as a copy (pass 0 reads A, writes W).
  mark(RRF_PHASE_INIT, -1);
  if (cudaMemsetAsync(ctrl, 0, 256, st) != cudaSuccess) return RRF_ERR_CUDA;   // also: the stop flag of the last run
  if (cudaMemset2DAsync(dV, (size_t)ldv * esize, 0, (size_t)p->max_rank * esize, (size_t)m, st) != cudaSuccess)
    return RRF_ERR_CUDA;

  // fork/join events for the side stream, created once and kept in the handle
  while (h->sync_events.size() < (size_t)4 * steps + 2) {
    cudaEvent_t ev;
    if (cudaEventCreateWithFlags(&ev, cudaEventDisableTiming) != cudaSuccess) return RRF_ERR_CUDA;
    h->sync_events.push_back(ev);
  }

  // Algorithm 2 lines 5-11: every pass is enqueued; passes after the stop return at once.
  auto panel_failed = [&](rrf_status_t ps_status) {
    out->cuda_error = h->last_cuda;
    if (!capturing) {
      cudaStreamSynchronize(st);
      cudaStreamSynchronize(h->aux);
    }
    return ps_status;
  };
  void* const V0 = dV;
  auto Vblk = [&](int r0) { return (void*)((char*)V0 + ((size_t)r0 * ldv + r0) * esize); };
  auto Tblk = [&](int r0) { return (void*)((char*)dT + (size_t)r0 * esize); };
  const SamplePlan sp = plan_sample(h->sms, m, n, esize, ops->s_kbs);
  PanelSource src{};
  src.slots = 0;
  src.nseg = sp.nseg;
  src.seg_stride = m * b;
  src.ldy = b;
  src.row_off = 0;
  mark(RRF_PHASE_SAMPLE, 0);
  ops->sample(tmA_s, tmO, Ypart, 0, (int)m, (int)n, 0, sp, ctrl, nullptr, init_part, st);
  init_ctrl_kernel<<<1, 256, 0, st>>>(init_part, std::min(sp.nslabs * sp.nseg, sp.ctas), p->tol, p->tol_is_relative,
                                      fixed ? 1 : 0, b, p->max_rank, ctrl, done_after, samp, steps, predict);

  if (unchanged) {
    // The variant of the paper's outlook that leaves A unchanged and returns no B: every panel is sampled from
    // A itself, Y_i = A Omega_i, pulled through the reflector blocks found so far (Q_0^T first), and its rows
    // i b.. are factored.  One pass over A per block instead of three; only a sampled rule (or the cap) stops it.
    void* Pbuf = ws + L.w;             // m x b panel, dense (the working copy of A is not needed here)
    const int npad_p = plan_vtw(h->sms, m, b, ops->v_bn).npad;
    CUtensorMap tmP_k, tmP_u, tmZp;
    if (!make_map(h, &tmP_k, p->dtype, Pbuf, m, b, b, kbox, tc) || !make_map(h, &tmP_u, p->dtype, Pbuf, m, b, b, ops->u_bm) ||
        !make_map(h, &tmZp, p->dtype, Zt, npad_p, b, b, ops->u_bn))
      return RRF_ERR_INVALID_ARG;
    unsigned bar_next = 0, bar_used = 0;
    const int sum_grid = (int)std::min<long long>((m * b + 255) / 256, (long long)h->sms * 8);
    for (int i = 0; i < steps_run; ++i) {
      const int r0 = i * b, rows = (int)(m - r0);
      if (i > 0) {
        mark(RRF_PHASE_SAMPLE, i);
        ops->sample(tmA_s, tmO, Ypart, 0, (int)m, (int)n, r0, sp, ctrl, nullptr, nullptr, st);
      }
      if (p->dtype == RRF_F64)
        panel_sum_kernel<double><<<sum_grid, 256, 0, st>>>((const double*)Ypart, sp.nseg, m * b, m, b, (double*)Pbuf, ctrl);
      else
        panel_sum_kernel<float><<<sum_grid, 256, 0, st>>>((const float*)Ypart, sp.nseg, m * b, m, b, (float*)Pbuf, ctrl);
      for (int l = 0; l < i; ++l) {
        const int q0 = l * b, rl = (int)(m - q0);
        VtwPlan vp = plan_vtw(h->sms, rl, b, ops->v_bn);
        vp.tc = tc;
        vp.chunk = h->tc_chunk;
        mark(RRF_PHASE_VTW, i);
        ops->vtw(tmV_k, tmP_k, Zpart, q0, q0, vp, ctrl, st);
        mark(RRF_PHASE_TZ, i);
        ops->tz(Zpart, vp, Tblk(q0), p->max_rank, 1, Zt, &ctrl->done, st);
        const UpdPlan up = plan_upd(h->sms, rl, b, ops->u_bm, ops->u_bn, ops->u_wn);
        mark(RRF_PHASE_UPDATE, i);
        ops->update(tmV_u, tmZp, tmP_u, tmP_u, Pbuf, b, Pbuf, b, q0, rl, b, q0, 0, -1, nullptr, nullptr, up, ctrl, nullptr, st);
      }
      PanelSource sd{};
      sd.nseg = 1;
      sd.ldy = b;
      sd.row_off = r0;
      PanelOpts po;
      po.merge_t = true;
      po.blocked = blocked;
      po.seq_base = 256u * (unsigned)i;
      po.bar_base = bar_next;
      po.bar_used = &bar_used;
      po.csq = csq_buf(i);
      int pg = 0;
      po.g_out = &pg;
      s = launch_panel(h, p->dtype, Pbuf, sd, rows, b, Vblk(r0), ldv, Tblk(r0), p->max_rank, ps, ctrl, &ctrl->done, st,
                       mark, i, po);
      if (s != RRF_OK) return panel_failed(s);
      bar_next += bar_used;
      mark(RRF_PHASE_STOP, i);
      est_kernel<<<1, 128, 0, st>>>(csq_buf(i), pg, (pg + 31) & ~31, b, p->max_rank, sampled ? p->estimator : 2,
                                    fixed ? 1 : 0, 1, i, tr_est, ctrl);
    }
  } else if (look_ctas == 0) {
    // One queue.  The panel of pass 0 is sampled by its own kernel; the panel of pass i+1 comes out
    // of the fused update of pass i.
    PanelSource alt{};             // the upcoming panel as the separate sample kernel would leave it
    const int* fused_flag = nullptr;
    for (int i = 0; i < steps_run; ++i) {
      const int r0 = i * b, rows = (int)(m - r0);
      PanelOpts po;
      po.st_t = h->aux;
      po.ev_fork = h->sync_events[2 * i];
      po.ev_join = h->sync_events[2 * i + 1];
      po.alt = alt;
      po.fused_flag = fused_flag;
      po.tree = tree;
      po.blocked = blocked;
      po.seq_base = 256u * (unsigned)i;
      int pg = 0;
      if (sampled) po.csq = csq_buf(i);
      po.g_out = &pg;
      s = launch_panel(h, p->dtype, Ypart, src, rows, b, Vblk(r0), ldv, Tblk(r0), p->max_rank, ps, ctrl, &ctrl->done,
                       st, mark, i, po);
      if (s != RRF_OK) return panel_failed(s);
      if (sampled)                     // the sampled rule looks at panel i before block i is applied
        est_kernel<<<1, 128, 0, st>>>(csq_buf(i), pg, (pg + 31) & ~31, b, p->max_rank, p->estimator, fixed ? 1 : 0, 0, i,
                                      tr_est, ctrl);
      VtwPlan vp = plan_vtw(h->sms, rows, n, ops->v_bn);
      vp.tc = tc;
      vp.chunk = h->tc_chunk;
      mark(RRF_PHASE_VTW, i);
      ops->vtw(tmV_k, i == 0 ? tmA_k : tmW_k, Zpart, r0, r0, vp, ctrl, st);
      mark(RRF_PHASE_TZ, i);
      cudaStreamWaitEvent(st, h->sync_events[2 * i + 1], 0);   // join: T_i is needed from here on
      ops->tz(Zpart, vp, Tblk(r0), p->max_rank, 1, Zt, &ctrl->done, st);
      UpdPlan up = plan_upd(h->sms, rows, n, ops->u_bm, ops->u_bn, ops->u_wn);
      if (utc_on) up.tc = &utc;
      const int j0 = (i + 1 < steps) ? r0 + b : -1;   // Omega rows of the next pass, if there is one
      mark(RRF_PHASE_UPDATE, i);
      ops->update(tmV_u, tmZ, i == 0 ? tmA_u : tmW_u, tmO, W, ldw, (char*)dB + (size_t)r0 * ldb * esize, ldb, r0, rows, (int)n, r0, b,
                  j0, Ypart, norm_part, up, ctrl, samp + i, st);
      mark(RRF_PHASE_STOP, i);
      stop_kernel<<<1, 256, 0, st>>>(norm_part, up.P, b, p->max_rank, p->estimator, fixed ? 1 : 0, tr_sub, tr_dir, ctrl,
                                     done_after, 1, predicting ? samp : nullptr, predict);
      if (j0 >= 0 && predicting) {
        // the next panel, sampled on its own if the loop goes on and the update had been told to skip it
        const SamplePlan sp2 = plan_sample(h->sms, rows - b, n, esize, ops->s_kbs);
        ops->sample(tmW_s, tmO, Ypart, r0 + b, rows - b, (int)n, j0, sp2, ctrl, samp + i, nullptr, st);
        alt = PanelSource{};
        alt.nseg = sp2.nseg;
        alt.seg_stride = (long long)(rows - b) * b;
        alt.ldy = b;
        fused_flag = samp + i;
      }
      src.slots = 1;
      src.row_off = b;
      src.bm = ops->u_bm;
      src.nc = up.NC;
      src.tpc = up.tpc;
      src.wn = ops->u_wn;
    }
  } else {
    // Two queues (the paper's look-ahead variant, Figure "DAG" (b)).  The fused update of pass i-1
    // samples the panel of pass i+1 from the matrix as it stands after pass i-1; the panel kernel of
    // pass i+1 applies the reflectors of pass i to that panel itself (PanelFix) and factors it on
    // `look_ctas` SMs while the GEMM kernels of pass i run on the other SMs.
    //   side stream : panel_0 | fix + panel_1 | fix + panel_2 | ...
    //   main stream :           V^T W, T Z, update, stop of pass 0 | of pass 1 | ...
    const int gsms = h->sms - look_ctas;
    void* Ybuf[2] = {Ypart, ws + L.ypart2};
    cudaEvent_t evS = h->sync_events[3 * steps], evS2 = h->sync_events[3 * steps + 1];
    auto evP = [&](int i) { return h->sync_events[3 * i]; };
    auto evU = [&](int i) { return h->sync_events[3 * i + 1]; };
    auto evZ = [&](int i) { return h->sync_events[3 * i + 2]; };
    auto evH = [&](int i) { return h->sync_events[3 * steps + 2 + i]; };
    // Where the update alone outlasts the next panel, the panel is held back until V^T W and T Z of
    // the pass are done, and V^T W gets every SM; otherwise the panel chain is the critical path and
    // starts as early as its inputs allow.
    auto gated = [&](int rows_i) {
      if (p->tune_gate != 0) return p->tune_gate == 2;
      if (look_cl) return false;       // a cluster takes so few SMs that holding it back never pays (measured)
      const PassModel pm{h->sms, (double)rows_i, (double)n, b, p->dtype == RRF_F64, tc, look_cl};
      return pm.step_gated(look_ctas) < pm.step_ungated(look_ctas);
    };
    PanelSource src1 = src;           // panel 1: sampled from A by the sample kernel
    src1.row_off = b;
    src1.nseg = plan_sample(gsms, m, n, esize, ops->s_kbs).nseg;
    cudaEventRecord(evS, st);
    cudaStreamWaitEvent(h->aux, evS, 0);
    ps.bar = look_bar;
    // the barrier counter is zeroed once per run and runs on from panel to panel (a panel that does not
    // run because the loop has ended adds nothing, and then no later panel runs either)
    unsigned bar_next = 0, bar_used = 0;
    PanelOpts po;
    po.ctas = look_ctas;
    po.tree = tree;
    po.blocked = blocked;
    po.merge_t = true;
    po.bar_used = &bar_used;
    std::vector<int> panel_g(steps + 1, 0);
    po.g_out = &panel_g[0];
    if (sampled) po.csq = csq_buf(0);
    s = launch_panel(h, p->dtype, Ybuf[0], src, m, b, Vblk(0), ldv, Tblk(0), p->max_rank, ps, ctrl, done_after, h->aux,
                     NoMark(), 0, po);
    if (s != RRF_OK) return panel_failed(s);
    bar_next += bar_used;
    cudaEventRecord(evP(0), h->aux);
    if (steps > 1) {                  // the second panel is sampled while the first is factored
      mark(RRF_PHASE_SAMPLE, 0);
      const SamplePlan sp1 = plan_sample(gsms, m, n, esize, ops->s_kbs);   // beside the first panel
      ops->sample(tmA_s, tmO, Ybuf[1], 0, (int)m, (int)n, b, sp1, ctrl, nullptr, nullptr, st);
      cudaEventRecord(evS2, st);
    }
    UpdPlan up_prev{};
    int pv_t1 = 0, pv_p1 = 0, pv_tpc2 = 0;   // how the update of the previous pass was split over two launches
    PanelSource alt_prev{};        // the panel of pass i+1 as the separate sample kernel would leave it
    for (int i = 0; i < steps_run; ++i) {
      const int r0 = i * b, rows = (int)(m - r0);
      const bool gate = gated(rows);
      auto next_panel = [&]() -> rrf_status_t {
        PanelSource sn = src1;
        if (i == 0) cudaStreamWaitEvent(h->aux, evS2, 0);
        if (i >= 1) {
          cudaStreamWaitEvent(h->aux, evU(i - 1), 0);   // the panel sampled by the update of pass i-1
          sn.slots = 1;
          sn.row_off = 2 * b;
          sn.bm = ops->u_bm;
          sn.nc = up_prev.NC;
          sn.tpc = up_prev.tpc;
          sn.wn = ops->u_wn;
          sn.t1 = pv_t1;
          sn.p1 = pv_p1;
          sn.tpc2 = pv_tpc2;
        }
        PanelOpts pn = po;
        pn.bar_base = bar_next;
        if (i >= 1) {
          pn.alt = alt_prev;
          pn.fused_flag = predicting ? samp + (i - 1) : nullptr;
        }
        pn.fix.enabled = 1;
        pn.fix.Vp = Vblk(r0);
        pn.fix.ldvp = ldv;
        pn.fix.Tp = Tblk(r0);
        pn.fix.ldtp = p->max_rank;
        pn.fix.Gpart = look_G;
        pn.fix.M = look_G + (size_t)kLookMaxCtas * b * b;
        if (gate) cudaStreamWaitEvent(h->aux, evZ(i), 0);
        pn.g_out = &panel_g[i + 1];
        pn.seq_base = 256u * (unsigned)(i + 1);
        if (sampled) pn.csq = csq_buf(i + 1);
        const rrf_status_t ls = launch_panel(h, p->dtype, Ybuf[(i + 1) & 1], sn, rows - b, b, Vblk(r0 + b), ldv,
                                             Tblk(r0 + b), p->max_rank, ps, ctrl, done_after + i, h->aux, NoMark(),
                                             i + 1, pn);
        if (ls == RRF_OK) {
          cudaEventRecord(evP(i + 1), h->aux);
          bar_next += bar_used;
        }
        return ls;
      };
      if (i + 1 < steps_run && !gate) {
        s = next_panel();
        if (s != RRF_OK) return panel_failed(s);
      }
      mark(RRF_PHASE_PANEL, i);                        // time the main stream waits for V_i, T_i
      cudaStreamWaitEvent(st, evP(i), 0);
      if (sampled)                     // the sampled rule looks at panel i before block i is applied
        est_kernel<<<1, 128, 0, st>>>(csq_buf(i), panel_g[i], (panel_g[i] + 31) & ~31, b, p->max_rank, p->estimator,
                                      fixed ? 1 : 0, 0, i, tr_est, ctrl);
      VtwPlan vp = plan_vtw(gate ? h->sms : gsms, rows, n, ops->v_bn);
      vp.tc = tc;
      vp.chunk = h->tc_chunk;
      mark(RRF_PHASE_VTW, i);
      ops->vtw(tmV_k, i == 0 ? tmA_k : tmW_k, Zpart, r0, r0, vp, ctrl, st);
      mark(RRF_PHASE_TZ, i);
      ops->tz(Zpart, vp, Tblk(r0), p->max_rank, 1, Zt, &ctrl->done, st);
      if (i + 1 < steps_run && gate) {
        cudaEventRecord(evZ(i), st);
        s = next_panel();
        if (s != RRF_OK) return panel_failed(s);
      }
      UpdPlan up = plan_upd(gsms, rows, n, ops->u_bm, ops->u_bn, ops->u_wn);
      if (utc_on) up.tc = &utc;
      const int j0 = (i + 2 < steps) ? r0 + 2 * b : -1;   // Omega rows of the pass after the next
      // Gated passes: the panel kernel, started together with the update, is done long before it, and its SMs
      // would idle.  The last tiles of the pass are therefore left to a second launch of the update kernel that
      // follows the panel kernel on ITS stream and so runs on the SMs it leaves: `look_ctas` CTAs with as many
      // tiles as they can do in the time the first launch still needs (by the schedule model, with a wide margin).
      int t1 = 0, tpc2 = 0;
      if (gate && !look_cl && !utc_on && i + 1 < steps_run && !h->profiling) {
        const PassModel pm{h->sms, (double)rows, (double)n, b, p->dtype == RRF_F64, tc, false};
        const double t_upd = pm.upd() * pm.scale(look_ctas), t_pan = pm.panel_chain(look_ctas);
        if (t_pan < 0.9 * t_upd) {
          const double t_all = ((double)gsms * t_upd + (double)look_ctas * t_pan) / h->sms;   // both launches end together
          // 0.35 of what the model allows: measured on 8192 x 8192, b = 64 (8.685 ms without the second launch):
          // 8.654 / 8.607 / 8.653 / 8.94 / 9.28 ms with 0.2 / 0.4 / 0.6 / 0.8 / 1.0 of it
          const double share = 0.35 * (double)look_ctas * (t_all - t_pan) / ((double)gsms * t_upd);
          const int tiles_h = (int)(share * up.total);
          if (tiles_h >= 4 * look_ctas) {
            tpc2 = ceil_div(tiles_h, look_ctas);
            t1 = up.total - tpc2 * look_ctas;
          }
        }
      }
      mark(RRF_PHASE_UPDATE, i);
      if (t1 > 0) {
        UpdPlan um = up, uh = up;
        um.total = t1;
        um.tpc = ceil_div(t1, gsms);
        um.P = ceil_div(t1, um.tpc);
        uh.p0 = um.P;
        uh.Lb = t1;
        uh.tpc = tpc2;
        uh.P = ceil_div(up.total - t1, tpc2);
        ops->update(tmV_u, tmZ, i == 0 ? tmA_u : tmW_u, tmO, W, ldw, (char*)dB + (size_t)r0 * ldb * esize, ldb, r0, rows, (int)n,
                    r0, b, j0, Ybuf[i & 1], norm_part, um, ctrl, samp + i, st);
        // behind the panel kernel of pass i+1 on the side stream (which has waited for T Z of this pass)
        ops->update(tmV_u, tmZ, i == 0 ? tmA_u : tmW_u, tmO, W, ldw, (char*)dB + (size_t)r0 * ldb * esize, ldb, r0, rows, (int)n,
                    r0, b, j0, Ybuf[i & 1], norm_part, uh, ctrl, samp + i, h->aux);
        cudaEventRecord(evH(i), h->aux);
        cudaStreamWaitEvent(st, evH(i), 0);
        up.tpc = um.tpc;          // what the loader of the sampled panel needs to find the partial results
        up.P = um.P + uh.P;
      } else {
        ops->update(tmV_u, tmZ, i == 0 ? tmA_u : tmW_u, tmO, W, ldw, (char*)dB + (size_t)r0 * ldb * esize, ldb, r0, rows, (int)n, r0, b,
                    j0, Ybuf[i & 1], norm_part, up, ctrl, samp + i, st);
      }
      const int up_t1 = t1, up_p1 = t1 > 0 ? ceil_div(t1, up.tpc) : 0, up_tpc2 = tpc2;
      mark(RRF_PHASE_STOP, i);
      stop_kernel<<<1, 256, 0, st>>>(norm_part, up.P, b, p->max_rank, p->estimator, fixed ? 1 : 0, tr_sub, tr_dir, ctrl,
                                     done_after, 0, predicting ? samp : nullptr, predict);
      if (j0 >= 0 && predicting) {
        // the panel of pass i+2, sampled on its own if the loop goes on and the update had been told to skip it;
        // its first b rows are the rows above that panel which the fix-up needs
        const SamplePlan sp2 = plan_sample(gsms, rows - b, n, esize, ops->s_kbs);
        ops->sample(tmW_s, tmO, Ybuf[i & 1], r0 + b, rows - b, (int)n, j0, sp2, ctrl, samp + i, nullptr, st);
        alt_prev = PanelSource{};
        alt_prev.nseg = sp2.nseg;
        alt_prev.seg_stride = (long long)(rows - b) * b;
        alt_prev.ldy = b;
        alt_prev.row_off = b;
      }
      cudaEventRecord(evU(i), st);
      up_prev = up;
      pv_t1 = up_t1;
      pv_p1 = up_p1;
      pv_tpc2 = up_tpc2;
    }
  }
  mark(RRF_PHASE_SKIPPED, steps);   // closing event
  RRF_NVTX_CLOSE(nvtx_open);
  return RRF_OK;
  };

  // The sequence of launches depends only on the arguments.  The first call with a given set is
  // enqueued directly; if the next call repeats it, the sequence is captured into a graph, and every
  // further repeat is one graph launch (no per-kernel launch cost on the host).
  std::vector<unsigned char> key;
  {
    auto put = [&](const void* ptr, size_t nbytes) {
      const unsigned char* c = static_cast<const unsigned char*>(ptr);
      key.insert(key.end(), c, c + nbytes);
    };
    const void* ptrs[6] = {dA, dOmegaT, dV, dT, dB, d_workspace};
    const long long lds[4] = {lda, ldo, ldv, ldb};
    const int ints[4] = {look_ctas, h->profiling, h->f32_engine, h->tc_chunk};
    put(p, sizeof(*p));
    put(ptrs, sizeof(ptrs));
    put(lds, sizeof(lds));
    put(&workspace_bytes, sizeof(workspace_bytes));
    put(ints, sizeof(ints));
  }
  const bool graphs_ok = !h->graph_off && !(p->flags & RRF_FLAG_NO_GRAPH);
  bool launched = false;
  if (graphs_ok && h->gexec != nullptr && key == h->gkey) {
    marks = h->gmarks;
    nev = marks.size();
    steps_run = h->gsteps;
    launched = cudaGraphLaunch(h->gexec, user_st) == cudaSuccess;
    if (!launched) h->graph_off = 1;
  } else if (graphs_ok && key == h->gcand) {
    if (h->gexec != nullptr) cudaGraphExecDestroy(h->gexec);
    if (h->graph != nullptr) cudaGraphDestroy(h->graph);
    h->gexec = nullptr;
    h->graph = nullptr;
    h->gkey.clear();
    st = h->cap;
    capturing = true;
    if (!inplace && h->cand_steps > 0) steps_run = std::min(steps, h->cand_steps + 1);
    rrf_status_t cs = RRF_ERR_CUDA;
    if (cudaStreamBeginCapture(st, cudaStreamCaptureModeRelaxed) == cudaSuccess) {
      cs = enqueue();
      cudaGraph_t g = nullptr;
      const cudaError_t ce = cudaStreamEndCapture(st, &g);
      if (cs == RRF_OK && ce == cudaSuccess && g != nullptr &&
          cudaGraphInstantiate(&h->gexec, g, 0) == cudaSuccess) {
        h->graph = g;
        h->gkey = key;
        h->gmarks = marks;
        h->gsteps = steps_run;
        launched = cudaGraphLaunch(h->gexec, user_st) == cudaSuccess;
      } else if (g != nullptr) {
        cudaGraphDestroy(g);
      }
    }
    if (!launched) {               // capture is not available here: enqueue directly from now on
      steps_run = steps;
      cudaGetLastError();
      if (h->gexec != nullptr) cudaGraphExecDestroy(h->gexec);
      if (h->graph != nullptr) cudaGraphDestroy(h->graph);
      h->gexec = nullptr;
      h->graph = nullptr;
      h->gkey.clear();
      h->graph_off = 1;
      if (cs != RRF_OK && cs != RRF_ERR_CUDA) return fail(cs);
    }
    capturing = false;
    st = user_st;
  }
  const bool direct = !launched;
  if (!launched) {
    marks.clear();
    nev = 0;
    steps_run = steps;
    s = enqueue();
    if (s != RRF_OK) return fail(s);
    h->gcand = key;
  }
  st = user_st;
  cudaError_t e = cudaGetLastError();
  Ctrl hc;
  if (e == cudaSuccess) e = cudaMemcpyAsync(&hc, ctrl, sizeof(Ctrl), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e == cudaSuccess && !direct && steps_run < steps && !hc.done && hc.status >= 0) {
    // the graph held fewer passes than this input needs: drop it and run the call in full
    if (h->gexec != nullptr) cudaGraphExecDestroy(h->gexec);
    if (h->graph != nullptr) cudaGraphDestroy(h->graph);
    h->gexec = nullptr;
    h->graph = nullptr;
    h->gkey.clear();
    h->gcand.clear();
    marks.clear();
    nev = 0;
    steps_run = steps;
    s = enqueue();
    if (s != RRF_OK) return fail(s);
    e = cudaGetLastError();
    if (e == cudaSuccess) e = cudaMemcpyAsync(&hc, ctrl, sizeof(Ctrl), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  }
  if (e != cudaSuccess) {
    h->last_cuda = (int)e;
    out->cuda_error = (int)e;
    return fail(RRF_ERR_CUDA);
  }
  if (direct) h->cand_steps = (hc.done && hc.status >= 0) ? hc.steps : -1;
  if (h->profiling && nev > 1) {
    std::memset(&h->profile, 0, sizeof(h->profile));
    for (size_t q = 0; q + 1 < nev; ++q) {
      float ms = 0.f;
      if (cudaEventElapsedTime(&ms, h->events[q], h->events[q + 1]) != cudaSuccess) continue;
      const int phase = marks[q].second >= hc.steps ? (int)RRF_PHASE_SKIPPED : marks[q].first;
      h->profile.ms[phase] += ms;
      h->profile.launches[phase] += 1;
    }
  }
  out->status = hc.status;
  out->k = hc.k;
  out->steps = hc.steps;
  out->normA2 = hc.normA2;
  out->sigma2 = hc.sigma2;
  out->E_sub = hc.E_sub;
  out->E_dir = hc.E_dir;
  out->queues = look_ctas > 0 ? 2 : 1;
  {
    // kernels this call put on the device (passes after the stop included: they start and return)
    const int lag = look_ctas > 0 ? 2 : 1;
    // without the predictor every executed pass that has a later panel to sample samples it
    out->fused_samples = predicting ? hc.fused_samples : std::min(hc.steps, std::max(0, steps - lag));
    const int sl = steps_run;      // passes whose kernels were launched
    if (unchanged)
      out->kernel_launches = (dOmegaT == nullptr ? 1 : 0) + 1 + 4 * sl + 3 * sl * (sl - 1) / 2;
    else
    out->kernel_launches = (sampled ? sl : 0) + 1 + (dOmegaT == nullptr ? 1 : 0) + 1 + ((look_ctas > 0 && steps > 1) ? 1 : 0) +
                           ((look_ctas > 0 || tree) ? 5 : 6) * sl +   // look-ahead, tree kernel: the panel kernel builds T itself
                           (predicting ? std::max(0, std::min(sl, steps - lag)) : 0) +
                           ((p->dtype == RRF_F32 && h->f32_engine == 1 && get_ops(p->dtype, b)->has_upd_tc)   // TF32 planes of Zt, OmegaT's rows
                                ? sl + std::max(0, std::min(sl, steps - lag)) : 0);
  }
  out->extra_samples = hc.extra_samples;
  out->panel_ctas = look_ctas;
  if (hc.steps > 0) {
    if (h_E_sub_trace != nullptr) cudaMemcpy(h_E_sub_trace, tr_sub, sizeof(double) * hc.steps, cudaMemcpyDeviceToHost);
    if (h_E_dir_trace != nullptr) cudaMemcpy(h_E_dir_trace, tr_dir, sizeof(double) * hc.steps, cudaMemcpyDeviceToHost);
  }
  out->n_est = hc.n_est;
  if (hc.n_est > 0 && h_E_est_trace != nullptr)
    cudaMemcpy(h_E_est_trace, tr_est, sizeof(double) * hc.n_est, cudaMemcpyDeviceToHost);
  return (rrf_status_t)hc.status;
}

// ------------------------------------------------------------------------------------------
// Column-major view (the LAPACK / MAGMA convention of the paper's setting).  A column-major matrix is its
// transpose stored row by row, so the entry points below transpose on the way in and on the way out and run
// the row-major path in between, on a working copy that the update overwrites anyway.
// ------------------------------------------------------------------------------------------
static cudaError_t launch_transpose(const rrf_ctx* h, int dtype, long long rows, long long cols, const void* src,
                                    long long lds, void* dst, long long ldd, cudaStream_t st) {
  if (rows == 0 || cols == 0) return cudaSuccess;
  const long long d = dtype == RRF_F64 ? 32 : 64;      // the kernel's tile side
  const long long tiles = ((rows + d - 1) / d) * ((cols + d - 1) / d);
  const int grid = (int)std::min<long long>(tiles, (long long)h->sms * 16);
  if (dtype == RRF_F64)
    transpose_kernel<double><<<grid, 256, 0, st>>>((const double*)src, lds, rows, cols, (double*)dst, ldd);
  else
    transpose_kernel<float><<<grid, 256, 0, st>>>((const float*)src, lds, rows, cols, (float*)dst, ldd);
  return cudaGetLastError();
}

rrf_status_t rrf_transpose(rrf_handle_t h, int32_t dtype, int64_t rows, int64_t cols, const void* dSrc, int64_t lds,
                           void* dDst, int64_t ldd, void* cuda_stream) {
  if (h == nullptr || (dtype != RRF_F64 && dtype != RRF_F32) || rows < 0 || cols < 0 || lds < cols || ldd < rows)
    return RRF_ERR_INVALID_ARG;
  if (rows > 0 && cols > 0 && (dSrc == nullptr || dDst == nullptr || dSrc == dDst)) return RRF_ERR_INVALID_ARG;
  const cudaError_t e = launch_transpose(h, dtype, rows, cols, dSrc, lds, dDst, ldd, (cudaStream_t)cuda_stream);
  if (e != cudaSuccess) {
    h->last_cuda = (int)e;
    return RRF_ERR_CUDA;
  }
  return RRF_OK;
}

struct ColMajorLayout {
  rrf_params_t q;          // the row-major run in the middle
  size_t inner, at, v, t, total;
  long long ldat;
};
static rrf_status_t colmajor_layout(const rrf_params_t* p, ColMajorLayout* L) {
  const rrf_status_t s = check_params(p);
  if (s != RRF_OK) return s;
  if (p->flags & RRF_FLAG_INPLACE) return RRF_ERR_INVALID_ARG;   // the input is read-only here
  L->q = *p;
  if (!(p->flags & RRF_FLAG_NO_UPDATE)) L->q.flags |= RRF_FLAG_INPLACE;   // the transposed copy is the working matrix
  const rrf_status_t s2 = check_params(&L->q);
  if (s2 != RRF_OK) return s2;
  const size_t esize = p->dtype == RRF_F64 ? 8 : 4;
  const long long pad = 16 / (long long)esize;
  L->ldat = (p->n + pad - 1) / pad * pad;
  RunLayout R;
  run_layout(&L->q, true, &R);
  size_t off = align_up(R.total, 256);
  L->inner = off;
  L->at = off;
  off += align_up((size_t)p->m * (size_t)L->ldat * esize, 256);
  L->v = off;
  off += align_up((size_t)p->m * (size_t)p->max_rank * esize, 256);
  L->t = off;
  off += align_up((size_t)p->b * (size_t)p->max_rank * esize, 256);
  L->total = off;
  return RRF_OK;
}

rrf_status_t rrf_colmajor_workspace_bytes(const rrf_params_t* p, size_t* bytes) {
  if (bytes == nullptr) return RRF_ERR_INVALID_ARG;
  ColMajorLayout L;
  const rrf_status_t s = colmajor_layout(p, &L);
  if (s != RRF_OK) return s;
  *bytes = L.total;
  return RRF_OK;
}

rrf_status_t rrf_run_colmajor(rrf_handle_t h, const rrf_params_t* p, const void* dA, int64_t lda, const void* dOmega,
                              int64_t ldo, void* dV, int64_t ldv, void* dT, void* dB, int64_t ldb, void* d_workspace,
                              size_t workspace_bytes, void* cuda_stream, rrf_result_t* out, double* h_E_sub_trace,
                              double* h_E_dir_trace, double* h_E_est_trace) {
  if (out == nullptr) return RRF_ERR_INVALID_ARG;
  std::memset(out, 0, sizeof(*out));
  auto fail = [&](rrf_status_t s) {
    out->status = s;
    return s;
  };
  if (h == nullptr) return fail(RRF_ERR_INVALID_ARG);
  ColMajorLayout L;
  const rrf_status_t s = colmajor_layout(p, &L);
  if (s != RRF_OK) return fail(s);
  const bool unchanged = (p->flags & RRF_FLAG_NO_UPDATE) != 0;
  if (dA == nullptr || dV == nullptr || dT == nullptr || (dB == nullptr && !unchanged) || d_workspace == nullptr)
    return fail(RRF_ERR_INVALID_ARG);
  if (lda < p->m || ldv < p->m || (dB != nullptr && ldb < p->max_rank)) return fail(RRF_ERR_INVALID_ARG);
  if (reinterpret_cast<uintptr_t>(d_workspace) & 255u) return fail(RRF_ERR_INVALID_ARG);
  if (workspace_bytes < L.total) return fail(RRF_ERR_WORKSPACE);
  cudaStream_t st = (cudaStream_t)cuda_stream;
  unsigned char* ws = (unsigned char*)d_workspace;
  void* At = ws + L.at;
  void* Vr = ws + L.v;
  void* Tr = ws + L.t;
  auto cuda_fail = [&](cudaError_t e) {
    h->last_cuda = (int)e;
    out->cuda_error = (int)e;
    return fail(RRF_ERR_CUDA);
  };
  // column-major m x n with leading dimension lda = row-major n x m with the same leading dimension
  cudaError_t e = launch_transpose(h, p->dtype, p->n, p->m, dA, lda, At, L.ldat, st);
  if (e != cudaSuccess) return cuda_fail(e);
  const rrf_status_t r = rrf_run(h, &L.q, At, L.ldat, dOmega, ldo, Vr, p->max_rank, Tr, unchanged ? nullptr : At, L.ldat,
                                 ws, L.inner, cuda_stream, out, h_E_sub_trace, h_E_dir_trace, h_E_est_trace);
  if (r < 0) return r;
  const int k = out->k;
  e = launch_transpose(h, p->dtype, p->m, k, Vr, p->max_rank, dV, ldv, st);
  // T_i goes to columns i b ... of a column-major b x max_rank array with leading dimension b
  if (e == cudaSuccess) e = launch_transpose(h, p->dtype, p->b, k, Tr, p->max_rank, dT, p->b, st);
  if (e == cudaSuccess && !unchanged) e = launch_transpose(h, p->dtype, k, p->n, At, L.ldat, dB, ldb, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) return cuda_fail(e);
  out->kernel_launches += 1 + (k > 0 ? (unchanged ? 2 : 3) : 0);
  return r;
}

}  // extern "C"

// ------------------------------------------------------------------------------------------
// rrf_panel_qr_static: panel QR for callers that cannot allocate (see include/rrf.h).
// The scratch is a fixed array in the device image.  In host code its name is only a stand-in
// for the symbol, not a device address: the address is looked up once per device with
// cudaGetSymbolAddress and that pointer is what the kernels receive.
// ------------------------------------------------------------------------------------------
namespace rrf {

constexpr long long kStaticMaxRows = 65536;
constexpr size_t kStaticCtrlBytes = 256;                    // Ctrl (status, stop flag, barrier counter)
constexpr size_t kStaticScratchBytes = 512 * 1024;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

struct StaticDevice {
  std::once_flag once;     // the set-up below runs once per device, whichever host thread calls first
  cudaError_t err;
  unsigned char* ptr;      // device address of g_static_scratch on this device
  int sms;
  int panel_smem_max;
};
constexpr int kStaticMaxDevices = 64;
static StaticDevice g_static_dev[kStaticMaxDevices];

// Once per device, with that device current: symbol address, device limits, kernel attributes.
static cudaError_t static_setup(int dev, StaticDevice* sd) {
  void* ptr = nullptr;
  cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
  if (e != cudaSuccess) return e;
  int smem_optin = 0;
  e = cudaDeviceGetAttribute(&sd->sms, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return e;
  e = cudaDeviceGetAttribute(&smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  if (e != cudaSuccess) return e;
  int cluster_unused = 0;
  e = setup_panel_kernels(smem_optin, &sd->panel_smem_max, &cluster_unused);
  if (e != cudaSuccess) return e;
  sd->ptr = static_cast<unsigned char*>(ptr);
  return cudaSuccess;
}

}  // namespace rrf

extern "C" rrf_status_t rrf_panel_qr_static(int32_t dtype, int64_t rows, int32_t b, const void* dY, int64_t ldy,
                                            void* dV, int64_t ldv, void* dT, int64_t ldt, void* cuda_stream) {
  if (dY == nullptr || dV == nullptr || dT == nullptr) return RRF_ERR_INVALID_ARG;
  if (!b_ok(dtype, b) || rows < b || ldy < b || ldv < b || ldt < b || ldy > 0x7fffffffLL) return RRF_ERR_INVALID_ARG;
  if (rows > kStaticMaxRows) return RRF_ERR_WORKSPACE;      // beyond the built-in scratch's stated limit
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kStaticMaxDevices) return RRF_ERR_CUDA;
  StaticDevice* sd = &g_static_dev[dev];
  std::call_once(sd->once, [&] { sd->err = static_setup(dev, sd); });
  if (sd->err != cudaSuccess || sd->ptr == nullptr) return RRF_ERR_CUDA;
  if (sd->sms > kMaxSms || kStaticCtrlBytes + direct_scratch_bytes(sd->sms, b) > kStaticScratchBytes)
    return RRF_ERR_WORKSPACE;
  rrf_ctx tmp{};                                            // host-side plan parameters only
  tmp.device = dev;
  tmp.sms = sd->sms;
  tmp.panel_smem_max = sd->panel_smem_max;
  PanelPlan pp;
  if (!plan_panel(&tmp, rows, b, &pp)) return RRF_ERR_WORKSPACE;   // panel too tall for on-chip storage
  cudaStream_t st = (cudaStream_t)cuda_stream;
  Ctrl* ctrl = reinterpret_cast<Ctrl*>(sd->ptr);
  PanelScratch ps = carve_panel(sd->ptr + kStaticCtrlBytes, sd->sms, b, false);
  ps.bar = &ctrl->bar;
  // the array keeps the last call's contents: the stop flag, the status and the barrier counter
  // must start at zero; everything else is written by the kernels before it is read
  if (cudaMemsetAsync(ctrl, 0, kStaticCtrlBytes, st) != cudaSuccess) return RRF_ERR_CUDA;
  PanelSource src{};
  src.slots = 0;
  src.nseg = 1;
  src.seg_stride = 0;
  src.ldy = (int)ldy;
  const rrf_status_t s = launch_panel(&tmp, dtype, dY, src, rows, b, dV, ldv, dT, ldt, ps, ctrl, &ctrl->done, st);
  if (s != RRF_OK) return s;
  int status = 0;
  if (cudaMemcpyAsync(&status, &ctrl->status, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess)
    return RRF_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return RRF_ERR_CUDA;
  return (rrf_status_t)status;
}

#ifdef RRF_TSQR_TRACE
extern "C" int rrf_debug_trace_panel(unsigned long long* out) {
  return (int)cudaMemcpyFromSymbol(out, rrf::g_pcl_trace, sizeof(unsigned long long) * 16);
}
extern "C" int rrf_debug_trace(unsigned long long* out) {
  return (int)cudaMemcpyFromSymbol(out, rrf::g_tsqr_trace, sizeof(unsigned long long) * 64);
}
#endif
