"""The two tensor-core paths of the single-precision products of Algorithm 2 line 8
(mma.sync 3xTF32 and tcgen05 3xTF32 with the accumulator in tensor memory):

  * both against a float64 statement of  C <- (I - V T^T V^T) C  (what rrf_apply_qt computes per block),
    at sizes where every CTA walks many tiles and every ring of the tcgen05 kernels wraps several times;
  * the error of the tcgen05 path as a function of the chunk length (how many 64-row tiles are summed in
    tensor memory, whose additions do not round to nearest, between round-to-nearest adds);
  * whole runs of Algorithm 2 on both paths against the oracle, and against each other.
"""
import numpy as np
import pytest
import torch

from oracle import rrf_oracle as orc
from paper_2608_28941_b200 import rrf, workloads as wl

pytestmark = pytest.mark.gpu

MMA, TC = 0, 1


@pytest.fixture()
def h():
    hd = rrf.rrf_create(0)
    yield hd
    rrf.rrf_destroy(hd)


def _reflector_like(m, k, b, gen):
    """V: unit lower trapezoidal blocks scaled like Householder vectors; T: upper triangular blocks."""
    V = torch.randn(m, k, dtype=torch.float64, device="cuda", generator=gen) / m ** 0.5
    T = torch.zeros(b, k, dtype=torch.float64, device="cuda")
    for l in range(k // b):
        blk = V[:, l * b:(l + 1) * b]
        blk[:l * b] = 0
        sub = blk[l * b:(l + 1) * b]
        sub.copy_(torch.tril(sub, -1) + torch.eye(b, dtype=torch.float64, device="cuda"))
        T[:, l * b:(l + 1) * b] = torch.triu(torch.randn(b, b, dtype=torch.float64, device="cuda", generator=gen))
    return V, T


def _apply_error(h, m, n, b, k, engine, chunk, seed=0):
    gen = torch.Generator(device="cuda").manual_seed(seed)
    V, T = _reflector_like(m, k, b, gen)
    Cm = torch.randn(m, n, dtype=torch.float64, device="cuda", generator=gen)
    V32, T32, C32 = V.float().contiguous(), T.float().contiguous(), Cm.float().contiguous()
    ref = C32.double()
    for l in range(k // b):
        Vl, Tl = V32[:, l * b:(l + 1) * b].double(), T32[:, l * b:(l + 1) * b].double()
        ref = ref - Vl @ (Tl.T @ (Vl.T @ ref))
    rrf.rrf_set_single_engine(h, engine, chunk)
    X = C32.clone()
    rrf.rrf_apply_qt(h, V32, T32, b, k, X)
    torch.cuda.synchronize()
    assert rrf.rrf_last_status(h) == 0
    return ((X.double() - ref).norm() / ref.norm()).item()


@pytest.mark.parametrize("engine", [MMA, TC])
@pytest.mark.parametrize("m,n,b,k", [(4096, 11008, 64, 128), (8192, 4096, 32, 64), (8192, 4096, 128, 256),
                                      (1000, 520, 64, 128), (777, 1300, 32, 96)])
def test_block_reflector_application_in_single_precision(h, engine, m, n, b, k):
    # a few units of float32 round-off per block; the bar is the one the whole-run tests use for B and Q
    err = _apply_error(h, m, n, b, k, engine, chunk=2)
    assert err <= 5e-6, err


def test_error_of_the_tensor_memory_accumulator_against_chunk_length(h):
    """The longer a sum stays in tensor memory the larger its error (its additions truncate), so the error grows
    with the chunk length; every length stays far below the 1e-4 bar of the single-precision parity tests, and
    short chunks are as accurate as the path that adds every k-step in registers."""
    m, n, b, k = 4096, 4096, 64, 128
    base = _apply_error(h, m, n, b, k, MMA, 0)
    errs = {c: _apply_error(h, m, n, b, k, TC, c) for c in (1, 2, 4, 16, 0)}
    assert base <= 1e-6
    assert errs[1] <= 3 * base + 1e-7
    assert errs[1] <= errs[4] <= errs[16] <= errs[0] * 1.05
    assert errs[0] <= 1e-4 / 3


def test_engine_setting_is_validated(h):
    with pytest.raises(rrf.RrfError):
        rrf.rrf_set_single_engine(h, 2, 0)
    with pytest.raises(rrf.RrfError):
        rrf.rrf_set_single_engine(h, 1, -1)


def _f32_workload(m, n, b, rank, decay, max_rank, tol):
    rng = np.random.default_rng(11)
    U, _ = np.linalg.qr(rng.standard_normal((m, rank)))
    W, _ = np.linalg.qr(rng.standard_normal((n, rank)))
    A = ((U * decay ** np.arange(rank)) @ W.T).astype(np.float32)
    Om = rng.standard_normal((n, max_rank)).astype(np.float32)
    return A, Om


@pytest.mark.parametrize("engine", [MMA, TC])
@pytest.mark.parametrize("flags", [rrf.RRF_FLAG_ONE_QUEUE, rrf.RRF_FLAG_TWO_QUEUES], ids=["one-queue", "two-queues"])
@pytest.mark.parametrize("b", [32, 64])
def test_whole_single_precision_runs_against_the_oracle_on_both_engines(h, engine, flags, b):
    m, n, max_rank, tol = 1500, 1100, 256, 3e-2
    A, Om = _f32_workload(m, n, b, 300, 0.985, max_rank, tol)
    o = orc.rrf(A.astype(np.float64), Om.astype(np.float64), b, tol, max_rank)
    dA = torch.from_numpy(A).cuda()
    dOmT = torch.from_numpy(np.ascontiguousarray(Om.T)).cuda()
    rrf.rrf_set_single_engine(h, engine, 2)
    for _ in range(3):                       # enqueued directly, captured into a graph, replayed
        g = rrf.rrf_run(h, dA, b, tol, max_rank, omegaT=dOmT, flags=flags)
        assert (g.k, g.steps, g.status) == (o.k, o.steps, o.status)
        k = g.k
        B = g.B[:k].cpu().numpy().astype(np.float64)
        assert np.max(np.abs(B - o.B)) <= 1e-4 * np.max(np.abs(o.B))
        Q = rrf.rrf_form_q(h, g.V, g.T, b, k).double()
        assert torch.linalg.norm(Q.T @ Q - torch.eye(k, dtype=torch.float64, device="cuda")).item() <= 1e-5
        np.testing.assert_allclose(np.array(g.E_dir_trace[:g.steps]), np.array(o.E_dir[:o.steps]), rtol=2e-3)


def test_last_pass_without_a_sample_at_full_width(h):
    """The pass that ends a run at the rank cap samples no further panel: its update releases its shared-memory
    stages sooner than any other, which is where a stage given back too early shows.  Both engines must leave the
    same residual and the same last rows of B."""
    w = wl.CONFIGS["cfg4"]
    A, _ = wl.make_matrix(w)
    dA = torch.from_numpy(np.ascontiguousarray(A.astype(np.float32))).cuda()
    OmT = torch.from_numpy(np.ascontiguousarray(wl.make_omega(w).astype(np.float32).T)).cuda()
    out = {}
    for engine in (MMA, TC):
        rrf.rrf_set_single_engine(h, engine, 2)
        Ac = dA.clone()
        g = rrf.rrf_run(h, Ac, w.b, w.tol, 128, omegaT=OmT[:128].contiguous(),
                        flags=rrf.RRF_FLAG_ONE_QUEUE | rrf.RRF_FLAG_INPLACE)
        out[engine] = (g.k, Ac, g.B[:g.k].clone())
    assert out[MMA][0] == out[TC][0] == 128
    # the bar of the parity tests (1e-4 of the largest entry of B); a tile computed from a stage that was
    # overwritten under it is off by the size of the entries themselves
    scale = out[MMA][2].abs().max().item()
    assert (out[MMA][1][128:] - out[TC][1][128:]).abs().max().item() <= 1e-4 * scale
    assert (out[MMA][2] - out[TC][2]).abs().max().item() <= 1e-4 * scale


def test_single_precision_runs_are_bitwise_reproducible(h):
    """Every reduction of the tcgen05 kernels and of the cluster panel kernel has a fixed order, and no result may
    depend on which CTA or message arrives first: two hundred runs on both schedules give the same bits."""
    rng = np.random.default_rng(3)
    m, n, b, max_rank = 2304, 3136, 64, 384
    A = (rng.standard_normal((m, 200)) @ rng.standard_normal((200, n)) / 14.0 + 1e-3 * rng.standard_normal((m, n))).astype(np.float32)
    dA = torch.from_numpy(A).cuda()
    dOmT = torch.from_numpy(rng.standard_normal((max_rank, n)).astype(np.float32)).cuda()
    rrf.rrf_set_single_engine(h, TC, 2)
    for flags in (rrf.RRF_FLAG_ONE_QUEUE, rrf.RRF_FLAG_TWO_QUEUES):
        ref = None
        for _ in range(200):
            g = rrf.rrf_run(h, dA, b, 1e-3, max_rank, omegaT=dOmT, flags=flags)
            cur = (g.k, g.status, g.V[:, :g.k].clone(), g.T[:, :g.k].clone(), g.B[:g.k].clone(), tuple(g.E_dir_trace[:g.steps]))
            if ref is None:
                ref = cur
                assert g.k >= 2 * b
            else:
                assert cur[0] == ref[0] and cur[1] == ref[1] and cur[5] == ref[5]
                assert torch.equal(cur[2], ref[2]) and torch.equal(cur[3], ref[3]) and torch.equal(cur[4], ref[4])
