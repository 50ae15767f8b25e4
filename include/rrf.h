/*
 * rrf.h - C ABI of the B200 (sm_100a) blocked adaptive randomized range finder.
 *
 * The library computes, entirely on one GPU, the factorisation A ~= Q B of the
 * paper's problem statement (Eqs. "A ~= Q Q^T A, Q^T Q = I_k" and "B = Q^T A"):
 * an orthonormal basis Q (m x k) kept as Householder block reflectors
 * Q = Q_0 Q_1 ... Q_{i-1}, Q_l = I - V_l T_l V_l^T (Eq. "Q_i = I_m - V_i T_i V_i^T"),
 * the projected matrix B (k x n), and the rank k found from a Frobenius
 * tolerance (Algorithm 2, "Householder Blocked Adaptive Randomized Range Finder").
 *
 * Conventions shared by every call
 *   - Every matrix pointer is DEVICE memory, row-major (C order): element (i, j) of a
 *     matrix with leading dimension ld is p[i*ld + j].  Leading dimensions are in
 *     elements.  Pointers must be 16-byte aligned and ld*sizeof(element) must be a
 *     multiple of 16 bytes (the tiles are fetched by TMA).
 *   - The caller owns every buffer and the CUDA stream.  The library allocates device
 *     memory only in rrf_create (a few hundred bytes of status words) and, temporarily,
 *     in the measurement aid rrf_measure_peak.
 *   - Scalars and result structs are HOST memory.
 *   - Every call returns an rrf_status_t; nothing throws, nothing exits.  Arguments are
 *     validated before anything is launched.  Device-side waits are bounded: a wait
 *     that gives up reports RRF_ERR_TIMEOUT and leaves the context usable.
 *   - Block size b must be one of 16, 32, 64, 128 (32, 64, 128 in single precision);
 *     max_rank must be a multiple of b and at most min(m, n)  (the paper assumes all
 *     dimensions divisible by b; here only max_rank has to be).  m and n are arbitrary.
 */
#ifndef RRF_H_
#define RRF_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct rrf_ctx* rrf_handle_t;

typedef enum { RRF_F64 = 0, RRF_F32 = 1 } rrf_dtype_t;

typedef enum {
  RRF_OK = 0,
  RRF_MAX_RANK_REACHED = 1,   /* success with information: rank cap hit before the tolerance */
  RRF_ERR_INVALID_ARG = -1,
  RRF_ERR_WORKSPACE = -2,     /* workspace too small, or (tree kernel, static entry point) a panel too tall for on-chip storage */
  RRF_ERR_CUDA = -3,          /* a CUDA call failed; the raw code is in rrf_result_t.cuda_error */
  RRF_ERR_TIMEOUT = -4,       /* a bounded device-side wait gave up */
  RRF_ERR_NONFINITE = -5      /* A contains NaN or Inf */
} rrf_status_t;

/* Flags for rrf_params_t.flags */
#define RRF_FLAG_INPLACE 1u     /* A itself is the working matrix (it is overwritten) */
#define RRF_FLAG_FIXED_RANK 2u  /* ignore the tolerance, always run to max_rank (fixed-rank mode) */
#define RRF_FLAG_ONE_QUEUE 4u   /* force the sequential schedule: panel, V^T W, update one after the other */
#define RRF_FLAG_SAMPLE_ALWAYS 32u /* every update samples a later panel (no prediction of the last passes) */
#define RRF_FLAG_SAMPLE_NEVER 64u  /* no update samples; every panel comes from the separate sample kernel
                                      (slower; exercises the path a wrong prediction takes).  Ignored in
                                      single precision and for b = 128, where the updates always sample */
#define RRF_FLAG_NO_GRAPH 16u    /* always enqueue the kernels one by one (by default a call that repeats the
                                   previous call's arguments is captured into a CUDA graph and replayed) */
#define RRF_FLAG_PANEL_TREE 128u /* b <= 64: factor the panels with the tree kernel (see rrf_panel_qr_tree) instead of
                                    the kernel that pays one grid barrier per column.  Off by default: it is the
                                    slower of the two on the sizes measured so far.  The look-ahead schedule is
                                    then used only if RRF_FLAG_TWO_QUEUES asks for it */
#define RRF_FLAG_PANEL_BLOCKED 512u /* factor the panels with the blocked kernel (see rrf_panel_qr_blocked) where it
                                      fits.  Off by default: slower than the column-by-column kernel in whole runs */
#define RRF_FLAG_NO_UPDATE 256u /* the variant of the paper's outlook that leaves A unchanged and returns no B: each
                                  panel is sampled from A itself and pulled through the reflector blocks found so
                                  far.  One pass over A per block instead of three.  Needs estimator 2 or 3, or
                                  RRF_FLAG_FIXED_RANK; dB may be NULL; sequential schedule, per-column panel kernel */
#define RRF_FLAG_TWO_QUEUES 8u  /* use the look-ahead schedule whenever the panel can be confined to a few SMs,
                                   also where the built-in rule would pick the sequential one */

typedef struct {
  int32_t dtype;            /* rrf_dtype_t: element type of A, Omega, V, T, B, Q */
  int32_t b;                /* block size */
  int32_t max_rank;         /* rank cap, multiple of b, <= min(m, n) */
  int32_t estimator;        /* 0: stop on the residual norm ||W[r0+b:, :]||_F^2 (default);
                               1: stop on the paper's E <- E - ||B_i||_F^2 (Algorithm 2, line 9);
                               2, 3: sampled rules, evaluated on panel i = W Omega_i before block i is applied and
                               ending the loop with k = i b if E <= sigma^2 (W: the residual left by i blocks):
                               2: E = ||Y_i||_F^2 / b, an unbiased estimate of ||W||_F^2;
                               3: E = (200/pi) max_j ||Y_i[:, j]||^2 >= ||W||_2^2 with probability 1 - 10^-b
                                  (a bound on the SPECTRAL norm of the residual, the norm of Eq. "tolerance").
                               If the rank cap ends the loop under 2 or 3 the status is RRF_MAX_RANK_REACHED:
                               nothing has certified the last block. */
  int64_t m, n;             /* A is m x n */
  double tol;               /* the tolerance sigma of Algorithm 2 ... */
  int32_t tol_is_relative;  /* ... taken as tol*||A||_F if non-zero */
  uint32_t flags;
  uint64_t seed;            /* seed of the built-in Gaussian generator (used when dOmegaT == NULL) */
  int32_t tune_panel_ctas;  /* look-ahead schedule: SMs given to the panel chain; 0 = the library's own rule */
  int32_t tune_gate;        /* look-ahead schedule: 0 = own rule, 1 = start each panel as early as its inputs
                               allow, 2 = hold it back until T^T Z of the pass is done (V^T W keeps every SM) */
} rrf_params_t;

typedef struct {
  int32_t status;           /* rrf_status_t of the run */
  int32_t k;                /* rank found: steps * b */
  int32_t steps;            /* block steps executed */
  int32_t cuda_error;       /* raw cudaError_t when status == RRF_ERR_CUDA */
  double normA2;            /* ||A||_F^2 */
  double sigma2;            /* squared absolute tolerance the loop compared against */
  double E_sub;             /* final value of Algorithm 2's E = ||A||_F^2 - sum ||B_i||_F^2 */
  double E_dir;             /* final ||W[k:, :]||_F^2 = ||A - Q B||_F^2 */
  int32_t queues;           /* schedule used: 1 = sequential, 2 = look-ahead (panel QR of the next block runs
                               beside the update of the current one) */
  int32_t panel_ctas;       /* look-ahead: SMs the panel kernel was confined to; sequential: 0 */
  int32_t fused_samples;    /* passes whose update also sampled a later panel */
  int32_t extra_samples;    /* panels the separate sample kernel had to provide (wrong "the loop will end"
                               predictions, or RRF_FLAG_SAMPLE_NEVER) */
  int32_t kernel_launches;  /* kernels of this library the call put on the device, passes after the stop
                               included (their kernels start, read the stop flag and return) */
  int32_t n_est;            /* estimators 2, 3: estimates evaluated (steps + 1 if an estimate ended the loop) */
} rrf_result_t;

/* Create / destroy a context bound to one CUDA device.  rrf_create makes `device`
 * current, queries its limits and allocates the context's status words.  A handle keeps per-call
 * state (events, a side stream, the captured graph of the last repeated call): use it from one thread
 * at a time, and do not overlap two rrf_run calls on the same handle. */
rrf_status_t rrf_create(rrf_handle_t* out, int device);
rrf_status_t rrf_destroy(rrf_handle_t h);

/* Bytes of device workspace rrf_run needs for these parameters (Algorithm 2 keeps B in
 * place of A; unless RRF_FLAG_INPLACE is set the working copy lives in the workspace). */
rrf_status_t rrf_workspace_bytes(const rrf_params_t* p, size_t* bytes);

/*
 * rrf_run - Algorithm 2, every step on the device.
 *
 *   dA       m x n input (lda >= n).  Read-only unless RRF_FLAG_INPLACE.
 *   dOmegaT  max_rank x n (ldo >= n): row j is the j-th Gaussian sample vector, i.e. the
 *            transpose of the n x max_rank matrix whose column block i is Omega_i of
 *            Algorithm 2 line 6.  NULL: drawn on the device from p->seed.
 *   dV       m x max_rank (ldv >= max_rank): Householder vectors, unit lower trapezoidal,
 *            block column i holds V_i in rows i*b.. and zeros above.  Columns >= k are
 *            unspecified on return.
 *   dT       b x max_rank, leading dimension max_rank: T_i (upper triangular) in columns i*b...;
 *            columns >= k are unspecified on return (the look-ahead schedule factors one panel
 *            past the stop).
 *   dB       max_rank x n (ldb >= n): rows 0..k-1 are B = Q^T A.  With RRF_FLAG_INPLACE,
 *            dB may alias dA (ldb == lda).
 *   d_workspace / workspace_bytes   at least rrf_workspace_bytes(), 256-byte aligned.
 *   cuda_stream   a cudaStream_t (NULL: the default stream).  All work is ordered after what
 *            is on it and the call synchronises it once, at the end, to read back the result.
 *            Part of the work runs on a stream the handle owns, forked from and joined back
 *            to cuda_stream with events.
 *   h_E_sub_trace, h_E_dir_trace   optional HOST arrays of max_rank/b doubles receiving
 *            both stopping quantities after every block step.
 *   h_E_est_trace   optional HOST array of max_rank/b + 1 doubles: under estimator 2 or 3, entry i is
 *            the estimate of the residual left by i blocks (out->n_est entries).
 *
 * The loop `while E > sigma^2` runs on the device: each kernel of a block step first
 * reads a device flag and returns at once when the stop rule has fired, so there is no
 * host round-trip per block.  Returns RRF_OK / RRF_MAX_RANK_REACHED, or an error (out->status
 * is the same value).
 *
 * Schedule (Section "Implementation" of the paper, Figure "DAG").  One queue: panel QR, V^T W,
 * T^T Z and the update follow one another.  Two queues: the panel of block i+1 is sampled one
 * block early, corrected with block i's reflectors and factored on a few SMs while the update of
 * block i runs on the others; this needs b <= 64 and a panel that fits in the shared memory of
 * at most a third of the SMs.  The library picks the faster one for the sizes given; the flags
 * RRF_FLAG_ONE_QUEUE / RRF_FLAG_TWO_QUEUES override that, and out->queues / out->panel_ctas say
 * what ran.  The two schedules compute the same quantities up to rounding.
 * A call whose arguments (parameters, pointers, leading dimensions, workspace) repeat those of
 * the previous call on this handle is captured into a CUDA graph and replayed on later repeats;
 * the buffers' CONTENTS may change freely between calls.  RRF_FLAG_NO_GRAPH disables this.
 *
 * Resuming.  A run made with RRF_FLAG_INPLACE that ended with RRF_MAX_RANK_REACHED at k0 = out->k leaves the
 * residual in rows k0.. of dA, and the blocks still to come are Algorithm 2 on that residual.  To carry on up to a
 * larger cap K call rrf_run again with m - k0 rows, max_rank = K - k0, the absolute tolerance
 * tol = sqrt(out->sigma2) (tol_is_relative = 0), RRF_FLAG_INPLACE, and every pointer moved on:
 * dA and dB to row k0, dV to row k0 and column k0 of an m x K array whose rows above k0 are zero in the new
 * columns, dOmegaT to its row k0 (or rrf_fill_omega with first_vec = k0), dT to a b x (K - k0) array.  The second
 * call's k, steps and traces continue the first one's; its normA2 is the residual's.  (The Python binding's
 * rrf_resume does exactly this.)
 */
rrf_status_t rrf_run(rrf_handle_t h, const rrf_params_t* p,
                     void* dA, int64_t lda,
                     const void* dOmegaT, int64_t ldo,
                     void* dV, int64_t ldv,
                     void* dT,
                     void* dB, int64_t ldb,
                     void* d_workspace, size_t workspace_bytes,
                     void* cuda_stream, rrf_result_t* out,
                     double* h_E_sub_trace, double* h_E_dir_trace, double* h_E_est_trace);

/*
 * Column-major view of Algorithm 2 (the LAPACK / MAGMA storage of the paper's Section "Implementation").
 *
 * rrf_run_colmajor takes and returns every matrix stored column by column:
 *   dA      m x n, lda >= m, read-only (RRF_FLAG_INPLACE is rejected);
 *   dOmega  n x max_rank, ldo >= n (16-byte aligned, ldo a multiple of 16 bytes): column block i is Omega_i.
 *           This is the same memory as rrf_run's dOmegaT.  NULL: drawn from p->seed;
 *   dV      m x max_rank, ldv >= m; columns >= k unspecified;
 *   dT      b x max_rank, leading dimension b: T_i in columns i*b ...;
 *   dB      max_rank x n, ldb >= max_rank: the leading k x n block is B = Q^T A (may be NULL with RRF_FLAG_NO_UPDATE).
 * No alignment is asked of dA, dV, dT, dB.  The call transposes A into a row-major working copy in the workspace
 * (rrf_colmajor_workspace_bytes: rrf_run's workspace plus m*n + m*max_rank + b*max_rank elements), runs rrf_run
 * on it in place with the same parameters, schedule and result fields, and transposes the k computed columns of
 * V and T and the k rows of B into the caller's arrays; it costs one extra read and write of A and of the results.
 * It synchronises the stream before it returns.  Values are those of rrf_run on the same matrices.
 *
 * rrf_transpose: dDst (cols x rows, ldd >= rows) = dSrc^T for dSrc rows x cols (lds >= cols), both row-major, not
 * in place - equivalently a change between row- and column-major storage of one matrix.  It is what a caller with
 * column-major data puts around rrf_apply_qt, rrf_apply_q, rrf_form_q and rrf_subspace_transfer, which are row-major
 * only.  Does not synchronise the stream.
 */
rrf_status_t rrf_colmajor_workspace_bytes(const rrf_params_t* p, size_t* bytes);
rrf_status_t rrf_run_colmajor(rrf_handle_t h, const rrf_params_t* p,
                              const void* dA, int64_t lda,
                              const void* dOmega, int64_t ldo,
                              void* dV, int64_t ldv,
                              void* dT,
                              void* dB, int64_t ldb,
                              void* d_workspace, size_t workspace_bytes,
                              void* cuda_stream, rrf_result_t* out,
                              double* h_E_sub_trace, double* h_E_dir_trace, double* h_E_est_trace);
rrf_status_t rrf_transpose(rrf_handle_t h, int32_t dtype, int64_t rows, int64_t cols, const void* dSrc, int64_t lds,
                           void* dDst, int64_t ldd, void* cuda_stream);

/*
 * rrf_panel_qr - Algorithm 2 line 7 on its own (LAPACK geqrt semantics): Householder QR of a
 * tall device panel Y (rows x b, ldy >= b) into V (rows x b, ldv >= b, unit lower trapezoidal,
 * explicit ones and zeros) and the compact-WY factor T (b x b, ldt >= b, upper triangular) with
 * H_0 ... H_{b-1} = I - V T V^T.  Reflector convention: beta = -sign(alpha) ||x||, v_0 = 1,
 * tau = (beta - alpha)/beta.  R is not returned.  Workspace: rrf_panel_workspace_bytes().
 * Any height: a panel whose slabs do not fit in the SMs' shared memory (more than about 32000 x 128 or
 * 47000 x 64 doubles on 148 SMs) is factored by the blocked kernel with its slabs in global memory.
 * Does not synchronise the stream; a timeout of the in-kernel grid barrier is reported by
 * the next rrf_last_status() call.
 */
rrf_status_t rrf_panel_workspace_bytes(int32_t dtype, int64_t rows, int32_t b, size_t* bytes);
rrf_status_t rrf_panel_qr(rrf_handle_t h, int32_t dtype, int64_t rows, int32_t b,
                          const void* dY, int64_t ldy, void* dV, int64_t ldv,
                          void* dT, int64_t ldt,
                          void* d_workspace, size_t workspace_bytes, void* cuda_stream);

/* rrf_panel_qr_blocked - the same call with the blocked kernel: the columns are factored in micro-panels of eight
 * (a column step touches eight columns of the slab instead of all b), each finished micro-panel is applied to the
 * rest of the panel as a block reflector on the FP64 tensor cores, and the CTAs exchange their partial sums through
 * flagged words in global memory instead of a grid barrier followed by a read.  Same V and T up to rounding.  Falls
 * back to the column-by-column kernel when the slab and its small matrices do not fit in shared memory. */
rrf_status_t rrf_panel_qr_blocked(rrf_handle_t h, int32_t dtype, int64_t rows, int32_t b,
                                  const void* dY, int64_t ldy, void* dV, int64_t ldv,
                                  void* dT, int64_t ldt,
                                  void* d_workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * rrf_panel_qr_tree - the same factorisation (Algorithm 2 line 7) by another route, for b <= 64: a tall-skinny QR
 * over row slabs (every CTA factors its slab on its own, the b x b triangular factors are reduced up a tree
 * of Householder QRs) followed by a reconstruction of the panel's Householder vectors and of T from the explicit
 * orthonormal factor.  It needs 2 * levels - 1 grid barriers instead of b, is built from orthogonal
 * transformations only, and returns the same V and T as rrf_panel_qr up to rounding, except where a column is
 * exactly zero below its pivot (LAPACK then takes H = I; this route returns another valid reflector).
 * Same arguments, workspace and error behaviour as rrf_panel_qr; RRF_ERR_WORKSPACE if the slabs and tree nodes
 * need more CTAs than the device has SMs (about 40000 rows for b = 64).
 */
rrf_status_t rrf_panel_qr_tree(rrf_handle_t h, int32_t dtype, int64_t rows, int32_t b,
                               const void* dY, int64_t ldy, void* dV, int64_t ldv,
                               void* dT, int64_t ldt,
                               void* d_workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * rrf_panel_qr_static - the same factorisation as rrf_panel_qr for callers that cannot allocate.
 * (The paper has no counterpart: it is an addition for embedding.)
 *
 * Who needs it: code that runs where device allocation is off limits - inside another
 * framework's memory plan where every byte is pre-assigned, in a plug-in or a real-time loop
 * that must not call cudaMalloc (which may synchronise the whole device and can fail late), or
 * before any allocator exists.  Such a caller has no handle (rrf_create allocates) and no
 * workspace to hand over.  This entry point needs neither: its scratch - the per-CTA partial
 * sums, the pivot row, the Gram rows, tau, the barrier counter and the status word of the
 * panel kernel - lives in one fixed 512 KiB array in the library's device image, which every GPU
 * that loads the library holds until the process exits.  It calls no cudaMalloc, cudaFree or
 * any other allocating routine; the caller still passes the input and the outputs.
 *
 * Limits: b in {16, 32, 64, 128} (32.. in single precision), b <= rows <= 65536, and the panel
 * must fit on chip (rows*b*8 bytes spread over the SMs, as for rrf_panel_qr); a larger request
 * returns RRF_ERR_WORKSPACE and launches nothing.
 *
 * The first call on each device looks up the array's device address (with that device current)
 * and raises the kernels' shared-memory limits; make that first call before starting any stream
 * capture.  That one-time set-up is guarded (std::call_once per device), so first calls from
 * several host threads are safe.  Every call on a device shares the one array and finds the
 * previous call's contents in it: the entry point clears the words that must start at zero
 * itself, but two calls whose kernels overlap on the GPU (different streams, or different host
 * threads) race on it - serialise them.
 * Unlike rrf_panel_qr, EVERY call copies the device-side status back and synchronises
 * `cuda_stream` before returning (RRF_OK, or RRF_ERR_TIMEOUT if the bounded grid barrier gave
 * up), so it blocks the calling thread until the panel is factored.
 */
rrf_status_t rrf_panel_qr_static(int32_t dtype, int64_t rows, int32_t b,
                                 const void* dY, int64_t ldy, void* dV, int64_t ldv,
                                 void* dT, int64_t ldt, void* cuda_stream);

/*
 * rrf_apply_qt / rrf_apply_q - C <- Q^T C or C <- Q C for a device matrix C (m x ncols,
 * ldc >= ncols) with Q = Q_0 ... Q_{k/b-1} given by V (m x k) and T (b x k, leading dimension
 * ldt) as rrf_run returns them (Algorithm 2 line 8 and Eq. "Q_i = I_m - V_i T_i V_i^T": Q is applied
 * one block reflector after the other, each as three GEMMs).  Workspace: rrf_apply_workspace_bytes().
 * rrf_form_q writes the explicit basis Q = Q I[:, 0:k] (m x k, ldq >= k).  None of the three
 * synchronises the stream.
 */
rrf_status_t rrf_apply_workspace_bytes(int32_t dtype, int64_t m, int64_t ncols, int32_t b, size_t* bytes);
rrf_status_t rrf_apply_qt(rrf_handle_t h, int32_t dtype, int64_t m, int32_t b, int32_t k,
                          const void* dV, int64_t ldv, const void* dT, int64_t ldt,
                          void* dC, int64_t ldc, int64_t ncols,
                          void* d_workspace, size_t workspace_bytes, void* cuda_stream);
rrf_status_t rrf_apply_q(rrf_handle_t h, int32_t dtype, int64_t m, int32_t b, int32_t k,
                         const void* dV, int64_t ldv, const void* dT, int64_t ldt,
                         void* dC, int64_t ldc, int64_t ncols,
                         void* d_workspace, size_t workspace_bytes, void* cuda_stream);
rrf_status_t rrf_form_q(rrf_handle_t h, int32_t dtype, int64_t m, int32_t b, int32_t k,
                        const void* dV, int64_t ldv, const void* dT, int64_t ldt,
                        void* dQ, int64_t ldq,
                        void* d_workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Building blocks of the column-sharded variant (outlook of the paper: "extensions to distributed matrix
 * layouts"; driver: paper_2608_28941_b200/sharded.py).  With the columns of A split over the GPUs, A = [A_1 .. A_P],
 * and the rows of Omega split to match, a block step needs one exchange: the m_i x b panel Y_i = sum_p W_p Omega_{i,p}
 * (an all-reduce, left to the caller's communication library); everything else is local.
 *
 * rrf_sample_panel: dY (rows x b, dense, leading dimension b) = C (rows x n, ldc) * OmegaT (b x n, ldo)^T, i.e. line 7
 *   of Algorithm 2 for one rank's column block.  Workspace: rrf_sample_workspace_bytes(), 256-byte aligned.
 * rrf_frobenius_sq: *d_out (a double in DEVICE memory) = squared Frobenius norm of C (rows x cols, ldc), summed in a fixed
 *   order in double precision; rows may be 0.  Workspace: 8 * 4 * (number of SMs) bytes (5 KB is always enough).
 * Neither synchronises the stream.
 */
rrf_status_t rrf_sample_workspace_bytes(int32_t dtype, int64_t rows, int32_t b, size_t* bytes);
rrf_status_t rrf_sample_panel(rrf_handle_t h, int32_t dtype, int64_t rows, int64_t n, int32_t b,
                              const void* dC, int64_t ldc, const void* dOmegaT, int64_t ldo, void* dY,
                              void* d_workspace, size_t workspace_bytes, void* cuda_stream);
rrf_status_t rrf_frobenius_sq(rrf_handle_t h, int32_t dtype, int64_t rows, int64_t cols, const void* dC, int64_t ldc,
                       double* d_out, void* d_workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * rrf_subspace_transfer - the subspace-consistency transform of the paper's Section "Towards
 * Efficient Low-Rank Deep Learning": a low-rank optimiser state M (k_old x ncols) held in the basis
 * Q_old of the previous step is re-expressed in the current basis Q_new,
 *     Mout (k_new x ncols) = Q_new^T (Q_old M),
 * both bases given by their reflectors (V m x k, T b x k) as rrf_run returns them, for the same m
 * and b; k_old and k_new may differ (the adaptive ranks of two training steps).  Computed as
 * [M; 0] (m x ncols) -> Q_old [M; 0] -> Q_new^T (.) -> first k_new rows, with the same kernels as
 * rrf_apply_q / rrf_apply_qt.  M and Mout are device matrices (ldm, ldmo >= ncols, 16-byte aligned
 * rows); they may not overlap.  Workspace: rrf_transfer_workspace_bytes(), 256-byte aligned.  Does
 * not synchronise the stream.
 */
rrf_status_t rrf_transfer_workspace_bytes(int32_t dtype, int64_t m, int64_t ncols, int32_t b, size_t* bytes);
rrf_status_t rrf_subspace_transfer(rrf_handle_t h, int32_t dtype, int64_t m, int32_t b,
                                   int32_t k_old, const void* dV_old, int64_t ldv_old,
                                   const void* dT_old, int64_t ldt_old,
                                   int32_t k_new, const void* dV_new, int64_t ldv_new,
                                   const void* dT_new, int64_t ldt_new,
                                   const void* dM, int64_t ldm, int64_t ncols,
                                   void* dMout, int64_t ldmo,
                                   void* d_workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * rrf_fill_omega - Algorithm 2 line 6: fill dOmegaT (nvec x n, ldo >= n) with i.i.d. standard
 * Gaussians.  Counter-based: element (j, c) depends only on (seed, j, c) - Philox-4x32-10 keyed
 * by the seed with counter (c/2, j), Box-Muller in double precision, rounded to dtype - so any
 * block of vectors can be regenerated independently.  Does not synchronise the stream.
 */
rrf_status_t rrf_fill_omega(rrf_handle_t h, int32_t dtype, uint64_t seed, int64_t n, int32_t nvec,
                            int32_t first_vec, void* dOmegaT, int64_t ldo, void* cuda_stream);

/*
 * rrf_set_single_engine - choose the tensor-core path of the single-precision product Z = V_i^T W
 * (Algorithm 2 line 8) for every later call on this handle that computes it (rrf_run, rrf_apply_q,
 * rrf_apply_qt, rrf_form_q, rrf_subspace_transfer).  Double precision is not affected.
 *   engine 0  mma.sync m16n8k8, 3xTF32, every k-step added round-to-nearest in registers (default)
 *   engine 1  tcgen05.mma kind::tf32, 3xTF32 operand planes in shared memory, accumulator in tensor
 *             memory; chunk_tiles > 0 bounds the number of 64-row tiles summed inside tensor memory
 *             (whose additions do not round to nearest) before a round-to-nearest add into registers,
 *             0 keeps a whole accumulator there.
 * Host-side setting, no device work.  Returns RRF_ERR_INVALID_ARG for other values.
 */
rrf_status_t rrf_set_single_engine(rrf_handle_t h, int32_t engine, int32_t chunk_tiles);

/*
 * Measurement aids (the paper reports wall times only; these have no counterpart in it).
 *
 * rrf_set_profiling(h, 1) makes every following rrf_run record a CUDA event on its stream
 * before each kernel it enqueues; rrf_get_profile then returns, for the last run, the device
 * time and the number of launches of each phase over the block steps that actually executed
 * (passes skipped by the device-side stop flag are reported under RRF_PHASE_SKIPPED).
 * rrf_measure_peak runs a register-resident arithmetic loop on all SMs for about `ms`
 * milliseconds and reports the achieved rate: kind 0 = FP64 tensor-core mma (m16n8k8),
 * 1 = FP64 FMA, 2 = FP32 FMA, 3 = TF32 tensor-core mma (m16n8k8).  It synchronises the device.
 */
enum {
  RRF_PHASE_INIT = 0,     /* Algorithm 2 lines 1-4 (and the Gaussian fill when Omega is generated) */
  RRF_PHASE_SAMPLE = 1,   /* line 7: Y = W[r0:, :] Omega_i */
  RRF_PHASE_PANEL = 2,    /* line 7: panel Householder QR */
  RRF_PHASE_TFACTOR = 3,  /* line 7: compact-WY T_i */
  RRF_PHASE_VTW = 4,      /* line 8: Z = V_i^T W */
  RRF_PHASE_TZ = 5,       /* line 8: Z <- T_i^T Z */
  RRF_PHASE_UPDATE = 6,   /* line 8: W -= V_i Z, with the norms of line 9 */
  RRF_PHASE_STOP = 7,     /* lines 9, 10 and the test of line 5 */
  RRF_PHASE_SKIPPED = 8,  /* launches of passes after the stop, which return at once */
  RRF_NPHASES = 9
};
typedef struct {
  double ms[RRF_NPHASES];
  int32_t launches[RRF_NPHASES];
  int32_t pad;
} rrf_profile_t;
rrf_status_t rrf_set_profiling(rrf_handle_t h, int32_t enable);
rrf_status_t rrf_get_profile(rrf_handle_t h, rrf_profile_t* out);
rrf_status_t rrf_measure_peak(rrf_handle_t h, int32_t kind, double ms, double* tflops);

/*
 * rrf_selftest_timeout - failure-detection self test (no counterpart in the paper).  Launches one
 * small CTA that waits, with the library's bounded grid-barrier wait shortened to `limit_ms`
 * milliseconds, for an arrival that never comes.  The wait gives up, the kernel records
 * RRF_ERR_TIMEOUT in the handle's device status word and returns normally: nothing traps, faults or
 * hangs, and the context stays usable.  The next rrf_last_status() call reports and clears it.
 */
rrf_status_t rrf_selftest_timeout(rrf_handle_t h, double limit_ms, void* cuda_stream);

/* Status word of the handle's device side (set by bounded waits), read with one small
 * device-to-host copy after synchronising `cuda_stream`; clears it. */
rrf_status_t rrf_last_status(rrf_handle_t h, void* cuda_stream);

const char* rrf_status_string(rrf_status_t s);

#ifdef __cplusplus
}
#endif
#endif /* RRF_H_ */
