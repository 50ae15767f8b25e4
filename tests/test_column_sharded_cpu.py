"""The column-sharded variant (one exchange of the m_i x b panel per block step), on the CPU.

The oracle's statement of it is pinned against the single-process oracle twice: with the ranks simulated in one
process (the all-reduce is a Python sum), and with two real gloo ranks, each of which sees only its own column block
and its own rows of Omega.  The same all-reduce wrapper is what the GPU driver hands to NCCL."""
import os
import sys
import threading

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from oracle import rrf_oracle as orc  # noqa: E402


def _problem(m=120, n=90, b=6, max_rank=48, seed=4):
    rng = np.random.default_rng(seed)
    p = min(m, n)
    u, _ = np.linalg.qr(rng.standard_normal((m, p)))
    v, _ = np.linalg.qr(rng.standard_normal((n, p)))
    A = (u * np.exp(-np.arange(p) / 5.0)) @ v.T
    Om = rng.standard_normal((n, max_rank))
    return A, Om, b, max_rank


class _Lockstep:
    """All-reduce among P threads of one process (the ranks run the algorithm in lock step)."""

    def __init__(self, P):
        self.P, self.slots, self.bar = P, [None] * P, threading.Barrier(P)

    def make(self, rank):
        def allreduce(x):
            self.slots[rank] = np.array(x, dtype=np.float64, copy=True)
            self.bar.wait()
            total = sum(self.slots[q] for q in range(self.P))      # rank order: every rank gets the same bits
            self.bar.wait()
            return total
        return allreduce


def test_sharded_oracle_equals_the_single_process_oracle_with_simulated_ranks():
    A, Om, b, max_rank = _problem()
    ref = orc.rrf(A, Om, b, 1e-3, max_rank)
    assert 0 < ref.k < max_rank
    cuts = [0, 25, 61, 90]                           # three ranks, uneven column blocks
    P = len(cuts) - 1
    ls = _Lockstep(P)
    out = [None] * P

    def run(p):
        out[p] = orc.rrf_column_sharded(A[:, cuts[p]:cuts[p + 1]], Om[cuts[p]:cuts[p + 1], :], b, 1e-3, max_rank, ls.make(p))

    th = [threading.Thread(target=run, args=(p,)) for p in range(P)]
    [t.start() for t in th]
    [t.join() for t in th]
    for p in range(P):
        r = out[p]
        assert (r.k, r.steps, r.status) == (ref.k, ref.steps, ref.status)
        assert np.allclose(r.E_dir, ref.E_dir, rtol=1e-10) and np.isclose(r.normA2, ref.normA2, rtol=1e-13)
        assert np.max(np.abs(r.V - ref.V)) < 1e-11 and np.max(np.abs(r.T - ref.T)) < 1e-11
        assert np.max(np.abs(r.B - ref.B[:, cuts[p]:cuts[p + 1]])) < 1e-12
        assert np.array_equal(r.V, out[0].V)         # replicated bit for bit: every rank factors the same panel


def _gloo_rank(rank, world, port, out):
    sys.path.insert(0, ROOT)
    from oracle import rrf_oracle as o2
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)

    def allreduce(x):
        t = torch.as_tensor(np.array(x, dtype=np.float64, copy=True)).reshape(-1).clone()
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
        r = t.numpy().reshape(np.shape(x))
        return r if np.ndim(x) else float(r)

    A, Om, b, max_rank = _problem()
    half = A.shape[1] // 2
    cols = slice(0, half) if rank == 0 else slice(half, A.shape[1])
    r = o2.rrf_column_sharded(A[:, cols], Om[cols, :], b, 1e-3, max_rank, allreduce)
    out[rank] = (r.k, r.status, list(r.E_dir), r.V.copy(), r.T.copy(), r.B.copy())
    dist.barrier()
    dist.destroy_process_group()


def test_sharded_oracle_on_two_gloo_ranks():
    world, port = 2, 29500 + os.getpid() % 400
    A, Om, b, max_rank = _problem()
    ref = orc.rrf(A, Om, b, 1e-3, max_rank)
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_gloo_rank, args=(world, port, out), nprocs=world, join=True)
        half = A.shape[1] // 2
        for rank, cols in ((0, slice(0, half)), (1, slice(half, A.shape[1]))):
            k, status, E, V, T, B = out[rank]
            assert (k, status) == (ref.k, ref.status)
            assert np.allclose(E, ref.E_dir, rtol=1e-10)
            assert np.max(np.abs(V - ref.V)) < 1e-11 and np.max(np.abs(T - ref.T)) < 1e-11
            assert np.max(np.abs(B - ref.B[:, cols])) < 1e-12
        assert np.array_equal(out[0][3], out[1][3])
