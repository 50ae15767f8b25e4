"""GPU parity: the CUDA library, called through the C ABI, against the CPU oracle on the
same seeded inputs.  Bars:
  k, status, steps: exact;  B and Q: relative max-norm 1e-10 (f64) / 1e-4 (f32);
  ||Q^T Q - I||_F <= 1e-12 (f64) / 1e-5 (f32).
Q's late column blocks are ill-conditioned functions of the input (two correct float64
implementations differ there by far more than 1e-10), so per block the Q bar is
max(bar, 10 x the oracle's own permutation envelope); every well-posed quantity gets the
plain bar."""
import numpy as np
import pytest
import torch

from oracle import rrf_oracle as orc
from paper_2608_28941_b200 import rrf, workloads as wl
from philox_ref import omega_reference as _omega_reference

pytestmark = pytest.mark.gpu

TOL = {"f64": dict(rel=1e-10, orth=1e-12), "f32": dict(rel=1e-4, orth=1e-5)}
ESTIMATORS = ["direct", "subtractive", "sampled_fro", "sampled_spectral"]
ALGOS = [pytest.param("column", id="per-column"), pytest.param("blocked", id="blocked"), pytest.param("tree", id="tree")]


@pytest.fixture(scope="module")
def h():
    hd = rrf.rrf_create(0)
    yield hd
    rrf.rrf_destroy(hd)


def _tdtype(w):
    return torch.float64 if w.dtype == "f64" else torch.float32


def _pad_cols(x: np.ndarray, mult: int) -> torch.Tensor:
    """Device copy of x whose leading dimension is a multiple of `mult` elements."""
    r, c = x.shape
    ld = (c + mult - 1) // mult * mult
    buf = torch.zeros((r, ld), dtype=torch.from_numpy(x).dtype, device="cuda")
    buf[:, :c] = torch.from_numpy(x).cuda()
    return buf[:, :c]


def run_both(h, w, estimator=0, flags=0, A=None, Om=None):
    if A is None:
        A, _ = wl.make_matrix(w)
    if Om is None:
        Om = wl.make_omega(w)
    A = np.ascontiguousarray(A.astype(w.np_dtype))
    Om_t = np.ascontiguousarray(Om.astype(w.np_dtype))
    mult = 2 if w.dtype == "f64" else 4
    dA = _pad_cols(A, mult)
    dOmT = _pad_cols(np.ascontiguousarray(Om_t.T), mult)
    g = rrf.rrf_run(h, dA, w.b, w.tol, w.max_rank, omegaT=dOmT, estimator=estimator, flags=flags)
    o = orc.rrf(A.astype(np.float64), Om_t.astype(np.float64), w.b, w.tol, w.max_rank, estimator=ESTIMATORS[estimator])
    return g, o, A, Om_t


def relmax(x, ref):
    d = np.max(np.abs(x - ref)) if ref.size else 0.0
    s = np.max(np.abs(ref)) if ref.size else 1.0
    return d / s if s > 0 else d


def check_run(h, w, g, o, A, Om, q_envelope=True, estimator="direct"):
    tol = TOL[w.dtype]
    assert g.k == o.k and g.steps == o.steps and g.status == o.status, (g.k, o.k, g.status, o.status)
    k, b = g.k, w.b
    assert np.isclose(g.normA2, o.normA2, rtol=1e-12 if w.dtype == "f64" else 1e-6)
    if k == 0:
        return
    B = g.B[:k].cpu().numpy().astype(np.float64)
    assert relmax(B, o.B) <= tol["rel"], ("B", relmax(B, o.B))
    u = 1.1e-16 if w.dtype == "f64" else 6e-8
    d = 2 * max(w.m, w.n) * u * np.sqrt(o.normA2)     # Frobenius size of the residual's rounding noise
    A64 = A.astype(np.float64)
    # The oracle's own envelope: the same problem with another summation order (float64: columns of A
    # and rows of Omega permuted; float32: the same steps in plain float32 on the CPU).
    op = None
    if q_envelope and w.dtype == "f64":
        op = orc.permuted_rerun(A64, Om.astype(np.float64), b, w.tol, w.max_rank, seed=1, estimator=estimator)
        assert op.k == o.k
    elif q_envelope:
        op = orc.rrf(A, Om, b, w.tol, w.max_rank, dtype=np.float32, estimator=estimator)
        if op.k != o.k:
            op = None
    # Stopping quantities after every block: 1e-9 relative, plus what the oracle's own trace moves under
    # the reordering (x10; x3 against the float32 rerun), plus the effect on the squared norm of a
    # perturbation of the residual of Frobenius size d0 = 4 u ||A||_F (a few ulps of A).
    d0 = 4 * u * np.sqrt(o.normA2)
    for i, (a, c) in enumerate(zip(g.E_dir_trace, o.E_dir)):
        if w.rank and w.noise_std == 0.0 and (i + 1) * b >= w.rank:
            # the generated rank is used up: what is left is the rounding noise of the updates, whose
            # norm depends on the summation order; it must stay at the noise level
            assert 0.0 <= a <= 100 * c + d * d, ("E_dir at rank exhaustion", i, a, c)
            continue
        slack = 1e-9 * c + 2 * np.sqrt(c) * d0 + d0 * d0
        if op is not None:
            slack += (10 if w.dtype == "f64" else 3) * abs(op.E_dir[i] - c)
        assert abs(a - c) <= slack, ("E_dir", i, a, c, slack)
    # Q explicitly, on the device
    Qg = rrf.rrf_form_q(h, g.V, g.T, b, k).cpu().numpy().astype(np.float64)
    Qo = orc.form_q(o.V, o.T, b)
    orth = np.linalg.norm(Qg.T @ Qg - np.eye(k))
    assert orth <= tol["orth"], ("orth", orth)
    # Q*B and the residual are well-posed: full bar
    assert relmax(Qg @ B, Qo @ o.B) <= 10 * tol["rel"], ("QB", relmax(Qg @ B, Qo @ o.B))
    res = np.linalg.norm(A64 - Qg @ B)
    assert abs(res ** 2 - o.E_dir[-1]) <= 1e-6 * o.E_dir[-1] + 2 * np.sqrt(o.E_dir[-1]) * d + d * d
    if o.status == orc.RRF_OK:
        assert res <= w.tol * np.sqrt(o.normA2) * (1 + 1e-6)
    # Q element-wise, block by block, against the oracle's own envelope
    env = None
    if op is not None:
        env = orc.form_q(op.V.astype(np.float64), op.T.astype(np.float64), b)
    worst = 0.0
    for i in range(k // b):
        blk = slice(i * b, (i + 1) * b)
        d = np.max(np.abs(Qg[:, blk] - Qo[:, blk])) / np.max(np.abs(Qo))
        bar = tol["rel"]
        if env is not None:
            mult = 10 if w.dtype == "f64" else 3
            bar = max(bar, mult * np.max(np.abs(env[:, blk] - Qo[:, blk])) / np.max(np.abs(Qo)))
        # a block sampled from a residual of relative size rho is only determined to about u / rho, and what
        # it contributes to Q B is weighted by rho: weighted that way a tenth of the plain bar is required
        rho = np.sqrt((o.E_dir[i - 1] if i > 0 else o.normA2) / o.normA2)
        assert d <= bar or d * rho <= 0.1 * tol["rel"], ("Q block", i, d, bar, rho)
        worst = max(worst, d)
    return worst


# ------------------------------------------------------------------ building blocks


@pytest.mark.parametrize("rows,b,dtype", [(200, 16, "f64"), (1024, 16, "f64"), (4096, 32, "f64"),
                                          (8192, 64, "f64"), (5001, 64, "f64"), (300, 128, "f64"),
                                          (20000, 128, "f64"), (4096, 64, "f32"), (777, 32, "f32"),
                                          (60000, 32, "f64"), (45000, 64, "f64"),       # slabs of 512 / 320 rows
                                          # one thread-block cluster: 1, 2, 16 CTAs; its largest panel, one row more
                                          # (cooperative grid again); b = 128 keeps the shared-memory loop
                                          (64, 64, "f64"), (100, 32, "f64"), (4096, 64, "f64"), (4097, 64, "f64"),
                                          (4095, 16, "f64"), (2048, 128, "f64"), (2049, 128, "f64"), (3000, 64, "f32")])
@pytest.mark.parametrize("algo", ALGOS)
def test_panel_qr_matches_oracle(h, rows, b, dtype, algo):
    tree, blocked = algo == "tree", algo == "blocked"
    if tree and (b > 64 or rows * b > 35000 * 64):
        pytest.skip("the tree kernel takes b <= 64 and at most one slab or node per SM")
    rng = np.random.default_rng(rows + b)
    Y = rng.standard_normal((rows, b))
    if dtype == "f32":
        Y = Y.astype(np.float32)
    V, T = rrf.rrf_panel_qr(h, torch.from_numpy(Y).cuda(), tree=tree, blocked=blocked)
    Vo, tau, To, _ = orc.panel_qr(Y.astype(np.float64))
    tol = 1e-12 if dtype == "f64" else 2e-6
    assert np.max(np.abs(V.cpu().numpy() - Vo)) <= tol
    assert np.max(np.abs(T.cpu().numpy() - To)) <= tol * 10


@pytest.mark.parametrize("algo", ALGOS)
@pytest.mark.parametrize("zero", [0.0, -0.0])
def test_panel_qr_with_a_zero_first_pivot(h, zero, algo):
    # the reflector of a zero pivot takes the sign of the zero on both sides (LAPACK's SIGN)
    rng = np.random.default_rng(17)
    Y = rng.standard_normal((700, 16))
    Y[0, 0] = zero
    V, T = rrf.rrf_panel_qr(h, torch.from_numpy(Y).cuda(), tree=algo == "tree", blocked=algo == "blocked")
    Vo, tau, To, _ = orc.panel_qr(Y)
    assert np.max(np.abs(V.cpu().numpy() - Vo)) <= 1e-12
    assert np.max(np.abs(T.cpu().numpy() - To)) <= 1e-11
    assert np.sign(Vo[1, 0]) == np.sign(Y[1, 0]) * (1.0 if np.copysign(1.0, zero) > 0 else -1.0)


@pytest.mark.parametrize("rows,b", [(65536, 128), (131072, 64), (40000, 128)])
def test_panels_taller_than_shared_memory(h, rows, b):
    # slabs that do not fit on chip are factored from global memory (blocked kernel); any height goes
    rng = np.random.default_rng(rows)
    Y = rng.standard_normal((rows, b))
    V, T = rrf.rrf_panel_qr(h, torch.from_numpy(Y).cuda())
    Vo, tau, To, _ = orc.panel_qr(Y)
    assert np.max(np.abs(V.cpu().numpy() - Vo)) <= 1e-12
    assert np.max(np.abs(T.cpu().numpy() - To)) <= 1e-11


@pytest.mark.parametrize("algo", ALGOS)
def test_panel_qr_zero_column_and_rank_deficient(h, algo):
    rng = np.random.default_rng(0)
    Y = rng.standard_normal((500, 16))
    Y[:, 3] = 0.0
    Y[:, 7] = Y[:, 2] * 2.0          # exactly dependent column
    Y[5:, 0] = 0.0                   # nothing to annihilate below... except rows 1..4
    V, T = rrf.rrf_panel_qr(h, torch.from_numpy(Y).cuda(), tree=algo == "tree", blocked=algo == "blocked")
    Vg, Tg = V.cpu().numpy(), T.cpu().numpy()
    Q = np.eye(500) - Vg @ Tg @ Vg.T
    assert np.linalg.norm(Q.T @ Q - np.eye(500)) < 1e-12
    R = Q.T @ Y
    assert np.max(np.abs(np.tril(R, -1))) < 1e-12


@pytest.mark.parametrize("m,ncols,b,k,dtype", [(600, 300, 16, 64, "f64"), (1000, 131, 32, 96, "f64"),
                                               (2048, 512, 64, 256, "f64"), (700, 260, 128, 256, "f64"),
                                               (1024, 520, 64, 128, "f32")])
def test_apply_and_form_q_match_oracle(h, m, ncols, b, k, dtype):
    rng = np.random.default_rng(m + ncols)
    n0 = k + 40
    A = rng.standard_normal((m, n0))
    Om = rng.standard_normal((n0, k))
    o = orc.rrf(A, Om, b, 0.0, k)
    npdt = np.float64 if dtype == "f64" else np.float32
    mult = 2 if dtype == "f64" else 4
    V = _pad_cols(o.V.astype(npdt), mult)
    T = _pad_cols(o.T.astype(npdt), mult)
    Cm = rng.standard_normal((m, ncols))
    tol = 1e-12 if dtype == "f64" else 3e-5
    got = rrf.rrf_apply_qt(h, V, T, b, k, _pad_cols(Cm.astype(npdt), mult)).cpu().numpy()
    assert relmax(got, orc.apply_qt(o.V, o.T, b, Cm)) <= tol
    got = rrf.rrf_apply_q(h, V, T, b, k, _pad_cols(Cm.astype(npdt), mult)).cpu().numpy()
    assert relmax(got, orc.apply_q(o.V, o.T, b, Cm)) <= tol
    Q = rrf.rrf_form_q(h, V, T, b, k).cpu().numpy()
    assert relmax(Q, orc.form_q(o.V, o.T, b)) <= tol


@pytest.mark.parametrize("m,n,b,k_old,k_new,ncols,dtype", [(700, 400, 16, 48, 80, 333, "f64"),
                                                          (1500, 900, 64, 192, 128, 1000, "f64"),
                                                          (1024, 640, 32, 96, 96, 520, "f32")])
def test_subspace_transfer_matches_oracle(h, m, n, b, k_old, k_new, ncols, dtype):
    # the bases of two unrelated matrices (two "training steps"), different ranks
    rng = np.random.default_rng(m + k_old)
    Om = rng.standard_normal((n, max(k_old, k_new)))
    old = orc.rrf(rng.standard_normal((m, n)), Om, b, 0.0, k_old)
    new = orc.rrf(rng.standard_normal((m, n)), Om, b, 0.0, k_new)
    M = rng.standard_normal((k_old, ncols))
    npdt = np.float64 if dtype == "f64" else np.float32
    mult = 2 if dtype == "f64" else 4
    dev = lambda x: _pad_cols(np.ascontiguousarray(x.astype(npdt)), mult)
    got = rrf.rrf_subspace_transfer(h, dev(old.V), dev(old.T), k_old, dev(new.V), dev(new.T), k_new, b, dev(M))
    want = orc.subspace_transfer(old.V, old.T, new.V, new.T, b, M)
    assert got.shape == (k_new, ncols)
    assert relmax(got.cpu().numpy().astype(np.float64), want) <= (1e-12 if dtype == "f64" else 3e-5)


# ------------------------------------------------------------------ whole runs


SCHEDULES = [pytest.param(rrf.RRF_FLAG_ONE_QUEUE, id="one-queue"), pytest.param(rrf.RRF_FLAG_TWO_QUEUES, id="two-queues")]


@pytest.mark.parametrize("sched", SCHEDULES)
def test_cfg1_full(h, sched):
    w = wl.CONFIGS["cfg1"]
    g, o, A, Om = run_both(h, w, flags=sched)
    assert o.k == 256 and o.status == orc.RRF_MAX_RANK_REACHED
    assert g.queues == (1 if sched == rrf.RRF_FLAG_ONE_QUEUE else 2)
    check_run(h, w, g, o, A, Om)


@pytest.mark.parametrize("name,kw", [
    ("cfg1", dict(m=512, n=384, max_rank=128)),
    ("cfg2", dict(m=1536, n=1280, max_rank=512)),
    ("cfg2", dict(m=1000, n=1111, max_rank=256)),           # ragged tiles in both dimensions
    ("cfg3", dict(m=1024, n=1024, max_rank=512)),
    ("cfg5", dict(m=2048, n=1024, max_rank=512, rank=384)),
    ("cfg4", dict(m=1024, n=2752, max_rank=256, rank=64)),
    ("cfg4b", dict(m=1024, n=2752, max_rank=256, rank=64)),
    ("cfg4", dict(m=1024, n=1500, max_rank=128, rank=48, b=32)),      # other fp32 block sizes
    ("cfg4b", dict(m=1200, n=1024, max_rank=256, rank=128, b=128)),
    ("cfg1", dict(m=900, n=700, max_rank=256, b=128)),                 # fp64, widest block, ragged
])
@pytest.mark.parametrize("sched", SCHEDULES)
def test_reduced_configs(h, name, kw, sched):
    w = wl.CONFIGS[name].scaled(**kw)
    g, o, A, Om = run_both(h, w, flags=sched)
    # the look-ahead schedule needs the panel (plus its staging) in a few SMs' shared memory
    assert g.queues == (2 if sched == rrf.RRF_FLAG_TWO_QUEUES and w.b <= 64 else 1)
    check_run(h, w, g, o, A, Om)


@pytest.mark.parametrize("sched", SCHEDULES)
@pytest.mark.parametrize("sampling", [pytest.param(rrf.RRF_FLAG_SAMPLE_ALWAYS, id="always-fused"),
                                      pytest.param(rrf.RRF_FLAG_SAMPLE_NEVER, id="never-fused")])
@pytest.mark.parametrize("name,kw", [("cfg2", dict(m=1536, n=1280, max_rank=512)),
                                     ("cfg3", dict(m=1024, n=1024, max_rank=512)),
                                     ("cfg1", dict(m=900, n=700, max_rank=256))])
def test_panel_from_either_sampler(h, name, kw, sched, sampling):
    # the update samples a later panel unless the stop rule predicts that the loop ends first; a panel
    # skipped wrongly comes from the separate sample kernel.  Both extremes must give the oracle's result.
    w = wl.CONFIGS[name].scaled(**kw)
    g, o, A, Om = run_both(h, w, flags=sched | sampling)
    if sampling == rrf.RRF_FLAG_SAMPLE_NEVER:
        assert g.fused_samples == 0 and g.extra_samples >= g.steps - (2 if g.queues == 2 else 1)
    else:
        assert g.extra_samples == 0 and g.fused_samples >= g.steps - (2 if g.queues == 2 else 1)
    check_run(h, w, g, o, A, Om)


@pytest.mark.parametrize("sched", SCHEDULES)
@pytest.mark.parametrize("name,kw", [("cfg2", dict(m=1536, n=1280, max_rank=512)),
                                     ("cfg3", dict(m=1024, n=1024, max_rank=384)),
                                     ("cfg4", dict(m=1024, n=2752, max_rank=256, rank=64))])
def test_each_block_factors_the_residual_it_was_given(h, name, kw, sched):
    # Block by block, without the conditioning that compounds over a run: stop the GPU after i blocks
    # (in place, so the residual W it leaves can be read back), sample Y_i = W[i b:, :] Omega_i from THAT
    # residual on the CPU, factor it with the oracle, and compare with block i of the full GPU run at
    # the plain bar (1e-10 / 1e-4, scaled by the panel's own condition number only; under the look-ahead
    # schedule the panel was sampled one update earlier, from a residual that was larger by the factor
    # `amp`, whose rounding noise it carries).
    w = wl.CONFIGS[name].scaled(**kw)
    A, _ = wl.make_matrix(w)
    Om = wl.make_omega(w).astype(w.np_dtype)
    dOmT = torch.from_numpy(np.ascontiguousarray(Om.T)).cuda()
    full = rrf.rrf_run(h, torch.from_numpy(A).cuda(), w.b, w.tol, w.max_rank, omegaT=dOmT,
                       flags=sched | rrf.RRF_FLAG_FIXED_RANK)
    assert full.k == w.max_rank
    Vf, Tf = full.V.cpu().numpy().astype(np.float64), full.T.cpu().numpy().astype(np.float64)
    b = w.b
    bar = TOL[w.dtype]["rel"]
    E = [full.normA2] + list(full.E_dir_trace)      # E[j]: squared residual norm after j blocks
    for i in (1, 2, 3):
        dA = torch.from_numpy(A).cuda()
        part = rrf.rrf_run(h, dA, b, w.tol, i * b, omegaT=dOmT[:i * b],
                           flags=sched | rrf.RRF_FLAG_FIXED_RANK | rrf.RRF_FLAG_INPLACE, B=dA[:i * b])
        assert part.k == i * b
        Wres = dA[i * b:].cpu().numpy().astype(np.float64)
        Y = Wres @ Om[:, i * b:(i + 1) * b].astype(np.float64)
        Vo, _, To, R = orc.panel_qr(Y)
        cond = np.linalg.cond(R)
        amp = np.sqrt(E[i - 1] / E[i]) if full.queues == 2 else 1.0
        tol = bar * max(1.0, cond / 100.0) * amp
        dv = np.max(np.abs(Vf[i * b:, i * b:(i + 1) * b] - Vo))
        dt = np.max(np.abs(Tf[:, i * b:(i + 1) * b] - To))
        assert dv <= tol and dt <= 10 * tol, (i, dv, dt, cond)


@pytest.mark.parametrize("sched", SCHEDULES)
@pytest.mark.parametrize("name,kw", [("cfg1", dict(m=512, n=384, max_rank=128)),
                                     ("cfg2", dict(m=1536, n=1280, max_rank=512)),
                                     ("cfg3", dict(m=1024, n=1024, max_rank=512)),
                                     ("cfg2", dict(m=6000, n=1111, max_rank=256)),      # several tree levels
                                     ("cfg4", dict(m=1024, n=2752, max_rank=256, rank=64))])
@pytest.mark.parametrize("panel", [pytest.param(rrf.RRF_FLAG_PANEL_TREE, id="tree"), pytest.param(rrf.RRF_FLAG_PANEL_BLOCKED, id="blocked")])
def test_whole_runs_with_the_other_panel_kernels(h, name, kw, sched, panel):
    # the opt-in panel kernels (tall-skinny QR + reconstruction; micro-panels of eight columns) under both schedules
    w = wl.CONFIGS[name].scaled(**kw)
    g, o, A, Om = run_both(h, w, flags=sched | panel)
    assert g.queues == (2 if sched == rrf.RRF_FLAG_TWO_QUEUES else 1)
    check_run(h, w, g, o, A, Om)


@pytest.mark.parametrize("sched", SCHEDULES)
@pytest.mark.parametrize("estimator", [2, 3])
@pytest.mark.parametrize("name,kw,tol", [("cfg2", dict(m=1536, n=1280, max_rank=512), 3e-3),
                                         ("cfg1", dict(m=900, n=700, max_rank=256), 1e-3),
                                         ("cfg4b", dict(m=1024, n=2752, max_rank=256, rank=64), 1e-2)])
def test_sampled_stopping_rules_match_the_oracle(h, name, kw, tol, estimator, sched):
    # the rules that look at the sampled panel instead of B or the updated matrix: same k, same estimates
    w = wl.CONFIGS[name].scaled(**kw)
    w = w.__class__(**{**w.__dict__, "tol": tol})
    g, o, A, Om = run_both(h, w, estimator=estimator, flags=sched)
    assert len(g.E_est_trace) == len(o.E_est) and g.status == o.status
    rt = 1e-9 if w.dtype == "f64" else 1e-4
    assert np.allclose(g.E_est_trace, o.E_est, rtol=rt, atol=rt * 1e-6 * o.normA2), (g.E_est_trace, o.E_est)
    if estimator == 2 or name != "cfg4b":
        assert 0 < g.k < w.max_rank and g.status == rrf.RRF_OK
    check_run(h, w, g, o, A, Om, estimator=ESTIMATORS[estimator])


@pytest.mark.parametrize("name,kw,tol", [("cfg2", dict(m=1536, n=1280, max_rank=512), 3e-3),
                                         ("cfg1", dict(m=900, n=700, max_rank=256), 1e-3),
                                         ("cfg5", dict(m=2048, n=1024, max_rank=512, rank=384), 1e-4),
                                         ("cfg4b", dict(m=1024, n=2752, max_rank=256, rank=64), 1e-2)])
def test_variant_that_leaves_a_unchanged(h, name, kw, tol):
    # no update of A, no B: panels are sampled from A and pulled through the reflectors found so far
    w = wl.CONFIGS[name].scaled(**kw)
    A, _ = wl.make_matrix(w)
    Om = wl.make_omega(w).astype(w.np_dtype)
    dA = torch.from_numpy(A).cuda()
    keep = dA.clone()
    dOmT = torch.from_numpy(np.ascontiguousarray(Om.T)).cuda()
    g = rrf.rrf_run(h, dA, w.b, tol, w.max_rank, omegaT=dOmT, estimator=2, flags=rrf.RRF_FLAG_NO_UPDATE)
    o = orc.rrf(A.astype(np.float64), Om.astype(np.float64), w.b, tol, w.max_rank, estimator="sampled_fro",
                schedule="a_unchanged")
    oi = orc.rrf(A.astype(np.float64), Om.astype(np.float64), w.b, tol, w.max_rank, estimator="sampled_fro")
    assert torch.equal(dA, keep) and g.B is None
    assert (g.k, g.steps, g.status) == (o.k, o.steps, o.status) and 0 < g.k < w.max_rank
    rt = 1e-9 if w.dtype == "f64" else 1e-4
    assert np.allclose(g.E_est_trace, o.E_est, rtol=rt, atol=rt * 1e-6 * o.normA2)
    k, b = g.k, w.b
    Qg = rrf.rrf_form_q(h, g.V, g.T, b, k).cpu().numpy().astype(np.float64)
    Qo = orc.form_q(o.V, o.T, b)
    tl = TOL[w.dtype]
    assert np.linalg.norm(Qg.T @ Qg - np.eye(k)) <= tl["orth"]
    A64 = A.astype(np.float64)
    # the projection is what a user of this variant gets: Q Q^T A against the oracle's, and the residual it leaves
    assert relmax(Qg @ (Qg.T @ A64), Qo @ (Qo.T @ A64)) <= 10 * tl["rel"]
    assert np.linalg.norm(A64 - Qg @ (Qg.T @ A64)) <= tol * np.sqrt(o.normA2) * 3.0
    prev = [oi.normA2] + oi.E_dir
    for i in range(k // b):
        blk = slice(i * b, (i + 1) * b)
        d = np.max(np.abs(Qg[:, blk] - Qo[:, blk])) / np.max(np.abs(Qo))
        rho = np.sqrt(prev[i] / oi.normA2)
        assert d <= tl["rel"] or d * rho <= tl["rel"], (i, d, rho)
    # fixed-rank mode of the same variant
    gf = rrf.rrf_run(h, dA, w.b, tol, w.max_rank, omegaT=dOmT, flags=rrf.RRF_FLAG_NO_UPDATE | rrf.RRF_FLAG_FIXED_RANK)
    of = orc.rrf(A.astype(np.float64), Om.astype(np.float64), w.b, tol, w.max_rank, schedule="a_unchanged",
                 fixed_rank=True, estimator="sampled_fro")
    assert gf.k == of.k == w.max_rank and gf.status == of.status
    Qf = rrf.rrf_form_q(h, gf.V, gf.T, b, gf.k).cpu().numpy().astype(np.float64)
    assert np.linalg.norm(Qf.T @ Qf - np.eye(gf.k)) <= tl["orth"]
    Qof = orc.form_q(of.V, of.T, b)
    assert relmax(Qf @ (Qf.T @ A64), Qof @ (Qof.T @ A64)) <= 10 * tl["rel"]


def test_single_precision_subtractive_rule_leaves_the_track_near_384_on_the_device(h):
    # The paper's stability experiment (1024 x 1024, singular values 1 ... 1e-14, b = 64, single precision) on the
    # GPU: Algorithm 2 line 9 (estimator 1) follows the residual for a few blocks and then stops tracking it
    # (cancellation: it stalls, or turns negative), while the residual norm itself (always recorded) and the
    # sampled Frobenius rule keep following the singular values down to the single-precision floor.
    rng = np.random.default_rng(2024)
    n, b, cap = 1024, 64, 640
    U, _ = np.linalg.qr(rng.standard_normal((n, n)))
    Vv, _ = np.linalg.qr(rng.standard_normal((n, n)))
    sv = np.logspace(0, -14, n)
    A = ((U * sv) @ Vv.T).astype(np.float32)
    Om = rng.standard_normal((n, cap)).astype(np.float32)
    dA, dOmT = torch.from_numpy(A).cuda(), torch.from_numpy(np.ascontiguousarray(Om.T)).cuda()
    g = rrf.rrf_run(h, dA, b, 0.0, cap, omegaT=dOmT, estimator=1, flags=rrf.RRF_FLAG_FIXED_RANK)
    o = orc.rrf(A, Om, b, 0.0, cap, dtype=np.float32)
    assert g.k == cap
    tail2 = np.array([np.sum(sv[(i + 1) * b:] ** 2) for i in range(cap // b)])   # Eckart-Young tails
    e_dir, e_sub = np.array(g.E_dir_trace), np.array(g.E_sub_trace)
    # the first blocks: both quantities are the residual (within 20 %) ...
    assert np.all(np.abs(e_sub[:3] - e_dir[:3]) <= 0.2 * e_dir[:3])
    # ... by block 6 (k = 384) and after, the subtractive one is off by more than a factor of two or negative
    lost = (e_sub[5:] <= 0.0) | (np.abs(e_sub[5:] - e_dir[5:]) > e_dir[5:])
    assert lost.all(), (e_sub, e_dir)
    # the residual norm keeps following the spectrum until the fp32 floor (about 1e-13 of ||A||^2)
    floor = 1e-12 * g.normA2
    assert np.all(e_dir >= 0.5 * tail2) and np.all(e_dir <= 100.0 * tail2 + floor)
    # same loss in the oracle's single-precision rerun (the paper's observation, pinned on the CPU too)
    o_sub, o_dir = np.array(o.E_sub), np.array(o.E_dir)
    assert ((o_sub[5:] <= 0.0) | (np.abs(o_sub[5:] - o_dir[5:]) > o_dir[5:])).all()
    # the sampled rule (estimator 2) looks at panel i = residual after i blocks: stays within its spread of it
    g2 = rrf.rrf_run(h, dA, b, 0.0, cap, omegaT=dOmT, estimator=2, flags=rrf.RRF_FLAG_FIXED_RANK)
    est = np.array(g2.E_est_trace)
    prev = np.concatenate([[g2.normA2], np.array(g2.E_dir_trace)[:-1]])
    ok = prev > floor
    assert np.all(est[ok] >= 0.3 * prev[ok]) and np.all(est[ok] <= 3.0 * prev[ok])


def test_schedules_agree_and_stop_mid_way(h):
    # stops after a few blocks: the look-ahead has factored one panel too many by then, which must
    # not show in k, B, the traces, or the defined part of V and T
    w = wl.CONFIGS["cfg2"].scaled(m=2048, n=1536, max_rank=512)
    A, _ = wl.make_matrix(w)
    Om = wl.make_omega(w)
    dA, dOmT = torch.from_numpy(A).cuda(), torch.from_numpy(np.ascontiguousarray(Om.T)).cuda()
    g1 = rrf.rrf_run(h, dA, w.b, 1e-2, w.max_rank, omegaT=dOmT, flags=rrf.RRF_FLAG_ONE_QUEUE)
    g2 = rrf.rrf_run(h, dA, w.b, 1e-2, w.max_rank, omegaT=dOmT, flags=rrf.RRF_FLAG_TWO_QUEUES)
    assert (g1.queues, g2.queues) == (1, 2) and g2.panel_ctas > 0
    assert 0 < g1.k < w.max_rank and g1.k == g2.k and g1.status == g2.status == rrf.RRF_OK
    k = g1.k
    assert relmax(g2.B[:k].cpu().numpy(), g1.B[:k].cpu().numpy()) <= 1e-10
    assert np.allclose(g1.E_dir_trace, g2.E_dir_trace, rtol=1e-9)
    Q1 = rrf.rrf_form_q(h, g1.V, g1.T, w.b, k).cpu().numpy()
    Q2 = rrf.rrf_form_q(h, g2.V, g2.T, w.b, k).cpu().numpy()
    assert relmax(Q2 @ g2.B[:k].cpu().numpy(), Q1 @ g1.B[:k].cpu().numpy()) <= 1e-10


@pytest.mark.parametrize("sched", SCHEDULES)
def test_subtractive_estimator_and_fixed_rank(h, sched):
    w = wl.CONFIGS["cfg2"].scaled(m=1024, n=768, max_rank=256)
    g, o, A, Om = run_both(h, w, estimator=1, flags=sched)
    check_run(h, w, g, o, A, Om, q_envelope=False)
    assert np.allclose(g.E_sub_trace, o.E_sub, rtol=1e-6, atol=1e-18 * o.normA2)
    dA, dOmT = torch.from_numpy(A).cuda(), torch.from_numpy(np.ascontiguousarray(Om.T)).cuda()
    ga = rrf.rrf_run(h, dA, w.b, 1e-2, w.max_rank, omegaT=dOmT, flags=sched)
    assert ga.k < w.max_rank and ga.status == rrf.RRF_OK
    gf = rrf.rrf_run(h, dA, w.b, 1e-2, w.max_rank, omegaT=dOmT, flags=sched | rrf.RRF_FLAG_FIXED_RANK)
    assert gf.k == w.max_rank and gf.status == rrf.RRF_OK   # tolerance met on the way, ran to the cap
    assert torch.equal(gf.B[:ga.k], ga.B[:ga.k])
    gf = rrf.rrf_run(h, dA, w.b, 1e-9, w.max_rank, omegaT=dOmT, flags=sched | rrf.RRF_FLAG_FIXED_RANK)
    assert gf.k == w.max_rank and gf.status == rrf.RRF_MAX_RANK_REACHED


def test_edge_cases(h):
    # zero matrix: rank 0, nothing launched past the init
    Z = torch.zeros((256, 128), dtype=torch.float64, device="cuda")
    OmT = torch.randn((64, 128), dtype=torch.float64, device="cuda")
    g = rrf.rrf_run(h, Z, 16, 1e-3, 64, omegaT=OmT)
    assert g.k == 0 and g.steps == 0 and g.status == rrf.RRF_OK
    # max_rank == b (one block) and max_rank == min(m, n) (run to completion, P7)
    w = wl.CONFIGS["cfg1"].scaled(m=160, n=96, max_rank=16)
    g, o, A, Om = run_both(h, w)
    check_run(h, w, g, o, A, Om)
    w = wl.CONFIGS["cfg1"].scaled(m=160, n=96, max_rank=96)
    w = w.__class__(**{**w.__dict__, "tol": 0.0})
    g, o, A, Om = run_both(h, w)
    assert g.k == 96
    check_run(h, w, g, o, A, Om, q_envelope=True)
    # non-finite input is reported, not propagated
    Abad = torch.randn((128, 128), dtype=torch.float64, device="cuda")
    Abad[3, 5] = float("nan")
    g = rrf.rrf_run(h, Abad, 16, 1e-3, 64, omegaT=torch.randn((64, 128), dtype=torch.float64, device="cuda"),
                    check=False)
    assert g.status == rrf.RRF_ERR_NONFINITE and g.k == 0


@pytest.mark.parametrize("sched", SCHEDULES)
def test_inplace_aliasing_b(h, sched):
    w = wl.CONFIGS["cfg2"].scaled(m=768, n=512, max_rank=128)
    g, o, A, Om = run_both(h, w, flags=sched)
    dA = torch.from_numpy(A).cuda()
    gi = rrf.rrf_run(h, dA, w.b, w.tol, w.max_rank, omegaT=torch.from_numpy(np.ascontiguousarray(Om.T)).cuda(),
                     flags=sched | rrf.RRF_FLAG_INPLACE, B=dA[:w.max_rank])
    assert gi.k == g.k
    assert torch.equal(dA[:g.k], g.B[:g.k])


def test_runs_are_bitwise_reproducible(h):
    w = wl.CONFIGS["cfg2"].scaled(m=1536, n=1024, max_rank=256)
    g1, o, A, Om = run_both(h, w)
    g2, _, _, _ = run_both(h, w)
    assert g1.k == g2.k and g1.E_dir_trace == g2.E_dir_trace and g1.E_sub_trace == g2.E_sub_trace
    k = g1.k
    assert torch.equal(g1.B[:k], g2.B[:k]) and torch.equal(g1.V[:, :k], g2.V[:, :k]) and torch.equal(g1.T[:, :k], g2.T[:, :k])


def test_graph_replay_follows_the_data(h):
    # Repeating a call with the same buffers replays a captured CUDA graph (third call on); the replay
    # must read the buffers' current contents and give what a direct enqueue gives, bit for bit.
    w = wl.CONFIGS["cfg2"].scaled(m=1280, n=1024, max_rank=256)
    A1, _ = wl.make_matrix(w)
    A2 = np.ascontiguousarray(A1[::-1] * 0.5 + np.roll(A1, 7, axis=1))
    Om = wl.make_omega(w)
    dA = torch.empty((w.m, w.n), dtype=torch.float64, device="cuda")
    dOmT = torch.from_numpy(np.ascontiguousarray(Om.T)).cuda()
    p = rrf.make_params(rrf.RRF_F64, w.m, w.n, w.b, w.tol, w.max_rank)
    ws = torch.empty(rrf.rrf_workspace_bytes(p), dtype=torch.uint8, device="cuda")
    V = torch.empty((w.m, w.max_rank), dtype=torch.float64, device="cuda")
    T = torch.empty((w.b, w.max_rank), dtype=torch.float64, device="cuda")
    B = torch.empty((w.max_rank, w.n), dtype=torch.float64, device="cuda")

    def run(A, flags):
        dA.copy_(torch.from_numpy(A))
        g = rrf.rrf_run(h, dA, w.b, w.tol, w.max_rank, omegaT=dOmT, V=V, T=T, B=B, workspace=ws, flags=flags)
        return g.k, g.status, list(g.E_dir_trace), B[:g.k].clone(), V[:, :g.k].clone(), T[:, :g.k].clone()

    for sched in (rrf.RRF_FLAG_ONE_QUEUE, rrf.RRF_FLAG_TWO_QUEUES):
        ref1 = run(A1, sched | rrf.RRF_FLAG_NO_GRAPH)
        ref2 = run(A2, sched | rrf.RRF_FLAG_NO_GRAPH)
        for A, ref in ((A1, ref1), (A1, ref1), (A1, ref1), (A2, ref2), (A1, ref1), (A2, ref2)):
            got = run(A, sched)          # direct, capture, then replays; the data changes under the graph
            assert got[:3] == ref[:3]
            assert all(torch.equal(x, y) for x, y in zip(got[3:], ref[3:]))


def test_runs_on_a_caller_stream(h):
    # all work is ordered on the caller's stream, also when the launches come from a replayed graph:
    # the input is produced on that stream right before the call and the output consumed right after
    w = wl.CONFIGS["cfg2"].scaled(m=1024, n=896, max_rank=192)
    A, _ = wl.make_matrix(w)
    Om = wl.make_omega(w)
    dOmT = torch.from_numpy(np.ascontiguousarray(Om.T)).cuda()
    dA0 = torch.from_numpy(A).cuda()
    ref = rrf.rrf_run(h, dA0, w.b, w.tol, w.max_rank, omegaT=dOmT, flags=rrf.RRF_FLAG_NO_GRAPH)
    refB = ref.B[:ref.k].clone()
    p = rrf.make_params(rrf.RRF_F64, w.m, w.n, w.b, w.tol, w.max_rank)
    ws = torch.empty(rrf.rrf_workspace_bytes(p), dtype=torch.uint8, device="cuda")
    V = torch.empty((w.m, w.max_rank), dtype=torch.float64, device="cuda")
    T = torch.empty((w.b, w.max_rank), dtype=torch.float64, device="cuda")
    B = torch.empty((w.max_rank, w.n), dtype=torch.float64, device="cuda")
    dA = torch.empty_like(dA0)
    side = torch.cuda.Stream()
    torch.cuda.synchronize()
    with torch.cuda.stream(side):
        for _ in range(4):
            dA.zero_()
            dA.add_(dA0)                 # the input only exists once this has run on `side`
            g = rrf.rrf_run(h, dA, w.b, w.tol, w.max_rank, omegaT=dOmT, V=V, T=T, B=B, workspace=ws)
            out = B[:g.k] * 1.0          # consumer on the same stream
            assert g.k == ref.k and torch.equal(out, refB)
    torch.cuda.synchronize()


def test_kernels_behind_a_timed_out_wait_return_at_once(h):
    # a wait that gives up also raises the stop flag, so work already enqueued behind it does not run on
    # half-written data (and cannot wait out its own limit): here a panel QR enqueued after the self test
    import ctypes as C
    lib = rrf.load()
    Y = torch.randn((512, 16), dtype=torch.float64, device="cuda")
    V = torch.full_like(Y, 7.0)
    T = torch.full((16, 16), 7.0, dtype=torch.float64, device="cuda")
    need = C.c_size_t()
    lib.rrf_panel_workspace_bytes(rrf.RRF_F64, 512, 16, C.byref(need))
    ws = torch.empty(need.value, dtype=torch.uint8, device="cuda")
    st = rrf._stream()
    assert lib.rrf_selftest_timeout(h, C.c_double(20.0), st) == rrf.RRF_OK          # enqueue only
    assert lib.rrf_panel_qr(h, rrf.RRF_F64, 512, 16, C.c_void_p(Y.data_ptr()), 16, C.c_void_p(V.data_ptr()), 16,
                            C.c_void_p(T.data_ptr()), 16, C.c_void_p(ws.data_ptr()), ws.numel(), st) == rrf.RRF_OK
    assert rrf.rrf_last_status(h) == rrf.RRF_ERR_TIMEOUT            # synchronises, reports, clears
    assert float(V.min()) == 7.0 and float(T.max()) == 7.0          # the panel kernels saw the flag and left at once
    Vg, Tg = rrf.rrf_panel_qr(h, Y)                                 # and the context works again
    Vo, _, To, _ = orc.panel_qr(Y.cpu().numpy())
    assert np.max(np.abs(Vg.cpu().numpy() - Vo)) <= 1e-12


def test_bounded_wait_times_out_and_context_survives(h):
    # a wait that nothing satisfies gives up after its limit and reports it; no trap, no hang
    assert rrf.rrf_selftest_timeout(h, 20.0) == rrf.RRF_ERR_TIMEOUT
    assert rrf.rrf_last_status(h) == rrf.RRF_OK                     # reported once, then cleared
    Y = torch.randn((512, 16), dtype=torch.float64, device="cuda")
    V, T = rrf.rrf_panel_qr(h, Y)                                   # the context is still usable
    Vo, _, To, _ = orc.panel_qr(Y.cpu().numpy())
    assert np.max(np.abs(V.cpu().numpy() - Vo)) <= 1e-12


def test_invalid_arguments_are_rejected(h):
    A = torch.randn((128, 96), dtype=torch.float64, device="cuda")
    for kw in (dict(b=24, max_rank=48), dict(b=16, max_rank=40), dict(b=16, max_rank=112), dict(b=16, max_rank=0)):
        with pytest.raises(rrf.RrfError) as e:
            rrf.rrf_run(h, A, kw["b"], 1e-3, kw["max_rank"])
        assert e.value.status == rrf.RRF_ERR_INVALID_ARG
    odd = torch.randn((128, 97), dtype=torch.float64, device="cuda")       # ld = 97 doubles: not 16-byte rows
    with pytest.raises(rrf.RrfError):
        rrf.rrf_run(h, odd, 16, 1e-3, 32)
    assert rrf.rrf_last_status(h) == rrf.RRF_OK
    # the tallest panel of the largest configuration (32768 x 128) does fit
    V, T = rrf.rrf_panel_qr(h, torch.randn((32768, 128), dtype=torch.float64, device="cuda"))
    assert torch.isfinite(V).all() and float(V[0, 0]) == 1.0 and torch.count_nonzero(torch.triu(V[:128], 1)) == 0


# ------------------------------------------------------------------ built-in Gaussian generator


def test_fill_omega_matches_host_generator(h):
    seed, n, nvec = 0x1234_5678_9abc_def0, 1001, 48
    O = rrf.rrf_fill_omega(h, n, nvec, seed).cpu().numpy()
    ref = _omega_reference(seed, n, nvec)
    assert np.max(np.abs(O - ref)) < 1e-13                 # same bits up to libm ulps
    O2 = rrf.rrf_fill_omega(h, n, 8, seed, first_vec=16).cpu().numpy()
    assert np.array_equal(O2, O[16:24])                    # counter-based: any block on its own
    big = rrf.rrf_fill_omega(h, 4096, 256, 7).cpu().numpy()
    assert abs(big.mean()) < 5e-3 and abs(big.std() - 1) < 5e-3
    assert abs(np.mean(big ** 4) - 3.0) < 0.05
    O32 = rrf.rrf_fill_omega(h, n, nvec, seed, dtype=torch.float32).cpu().numpy()
    assert np.array_equal(O32, ref.astype(np.float32)) or np.max(np.abs(O32 - ref)) < 1e-6


def test_run_with_builtin_omega(h):
    w = wl.CONFIGS["cfg2"].scaled(m=1024, n=1024, max_rank=256)
    A, _ = wl.make_matrix(w)
    dA = torch.from_numpy(A).cuda()
    g = rrf.rrf_run(h, dA, w.b, w.tol, w.max_rank, seed=42)
    OmT = rrf.rrf_fill_omega(h, w.n, w.max_rank, 42).cpu().numpy()
    o = orc.rrf(A, OmT.T, w.b, w.tol, w.max_rank)
    assert g.k == o.k and g.status == o.status
    assert relmax(g.B[:g.k].cpu().numpy(), o.B) <= 1e-10


# ------------------------------------------------------------------ column-sharded driver (one rank on one GPU)


@pytest.mark.parametrize("name,kw", [("cfg2", dict(m=1536, n=1280, max_rank=512)), ("cfg1", dict(m=900, n=700, max_rank=256)),
                                     ("cfg4b", dict(m=1024, n=2752, max_rank=256, rank=64))])
def test_column_sharded_driver_as_a_single_rank(h, name, kw):
    # the multi-GPU variant's code path (sample, exchange, panel QR, local update, norms) with a one-rank "exchange";
    # its host logic across ranks is covered on the CPU with gloo (tests/test_column_sharded_cpu.py)
    from paper_2608_28941_b200 import sharded
    w = wl.CONFIGS[name].scaled(**kw)
    A, _ = wl.make_matrix(w)
    Om = wl.make_omega(w).astype(w.np_dtype)
    mult = 2 if w.dtype == "f64" else 4
    g = sharded.rrf_run_column_sharded(h, _pad_cols(A, mult), _pad_cols(np.ascontiguousarray(Om.T), mult), w.b, w.tol, w.max_rank)
    o = orc.rrf(A.astype(np.float64), Om.astype(np.float64), w.b, w.tol, w.max_rank)
    assert (g.k, g.steps, g.status) == (o.k, o.steps, o.status)
    tl = TOL[w.dtype]
    assert relmax(g.B[:g.k].cpu().numpy().astype(np.float64), o.B) <= tl["rel"]
    assert np.allclose(g.E_dir_trace, o.E_dir, rtol=1e-8 if w.dtype == "f64" else 1e-3, atol=1e-24 * o.normA2)
    Q = rrf.rrf_form_q(h, _pad_cols(g.V[:, :g.k].cpu().numpy(), mult), _pad_cols(g.T[:, :g.k].cpu().numpy(), mult), w.b, g.k)
    Q = Q.cpu().numpy().astype(np.float64)
    assert np.linalg.norm(Q.T @ Q - np.eye(g.k)) <= tl["orth"]
    assert relmax(Q @ g.B[:g.k].cpu().numpy().astype(np.float64), orc.form_q(o.V, o.T, w.b) @ o.B) <= 10 * tl["rel"]


@pytest.mark.parametrize("sched", [rrf.RRF_FLAG_ONE_QUEUE, rrf.RRF_FLAG_TWO_QUEUES], ids=["one-queue", "two-queues"])
@pytest.mark.parametrize("dtype", ["f64", "f32"])
def test_replayed_graph_that_holds_fewer_passes_than_the_new_input_needs(h, sched, dtype):
    """A graph captured for a repeated call holds only the passes that call needed.  The same buffers then get an
    input of higher rank: the replay ends with the loop still open, and the call must be run again in full and give
    the oracle's answer for the NEW input (and the old answer again when the old input comes back)."""
    m, n, b, max_rank = 900, 700, 32, 256
    tol = 1e-6 if dtype == "f64" else 1e-3
    npdt = np.float64 if dtype == "f64" else np.float32
    rng = np.random.default_rng(5)

    def lowrank(r):
        return (rng.standard_normal((m, r)) @ rng.standard_normal((r, n)) / np.sqrt(r)).astype(npdt)

    A_small, A_big = lowrank(40), lowrank(150)
    Om = rng.standard_normal((n, max_rank)).astype(npdt)
    dA = torch.empty((m, n), dtype=torch.float64 if dtype == "f64" else torch.float32, device="cuda")
    dOmT = torch.from_numpy(np.ascontiguousarray(Om.T)).cuda()
    V = torch.empty((m, max_rank), dtype=dA.dtype, device="cuda")
    T = torch.empty((b, max_rank), dtype=dA.dtype, device="cuda")
    B = torch.empty((max_rank, n), dtype=dA.dtype, device="cuda")
    need = rrf.rrf_workspace_bytes(rrf.make_params(rrf.RRF_F64 if dtype == "f64" else rrf.RRF_F32, m, n, b, tol, max_rank))
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")

    def run():
        return rrf.rrf_run(h, dA, b, tol, max_rank, omegaT=dOmT, flags=sched, V=V, T=T, B=B, workspace=ws)

    def check(A):
        o = orc.rrf(A.astype(np.float64), Om.astype(np.float64), b, tol, max_rank)
        g = run()
        assert (g.k, g.steps, g.status) == (o.k, o.steps, o.status), (g.k, o.k)
        Bg = g.B[:g.k].cpu().numpy().astype(np.float64)
        assert relmax(Bg, o.B) <= TOL[dtype]["rel"]
        return g.k

    dA.copy_(torch.from_numpy(A_small))
    k_small = check(A_small)           # enqueued directly
    assert check(A_small) == k_small   # captured, holding k_small / b + 1 passes
    assert check(A_small) == k_small   # replayed
    dA.copy_(torch.from_numpy(A_big))
    k_big = check(A_big)               # replayed, found too short, run in full
    assert k_big > k_small + b
    assert check(A_big) == k_big       # captured anew
    dA.copy_(torch.from_numpy(A_small))
    assert check(A_small) == k_small   # the longer graph serves the shorter input
