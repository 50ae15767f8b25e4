"""The panel QR entry point for callers that cannot allocate device memory.

Some embedders - a framework with a fixed memory plan, a plug-in or control loop that must
never call cudaMalloc - can use neither a handle (creating one allocates) nor a workspace.
rrf_panel_qr_static keeps its scratch in a fixed array inside the library instead.  This test
calls it through the C ABI several times in a row, on different panels, and checks every result
against the ordinary entry point and the CPU oracle: a later call must not be disturbed by what an earlier one left in
the shared array.  It lives in its own file, collected last, and also passes on its own."""
import numpy as np
import pytest
import torch

from oracle import rrf_oracle as orc
from paper_2608_28941_b200 import rrf

pytestmark = pytest.mark.gpu


def test_static_scratch_panel_qr_matches_workspace_version_twice():
    cases = [(6000, 64, torch.float64), (2500, 32, torch.float64), (4096, 64, torch.float32)]
    outs = []
    # the allocation-free calls come first, back to back, before this test creates any handle
    for call, (rows, b, dtype) in enumerate(cases):
        gen = torch.Generator(device="cuda").manual_seed(100 + call)
        Y = torch.randn((rows, b), dtype=dtype, device="cuda", generator=gen)
        V = torch.full_like(Y, float("nan"))
        T = torch.full((b, b), float("nan"), dtype=dtype, device="cuda")
        status = rrf.rrf_panel_qr_static(Y, V, T)
        assert status == rrf.RRF_OK
        outs.append((Y, V, T))
    h = rrf.rrf_create(0)
    try:
        for (rows, b, dtype), (Y, V, T) in zip(cases, outs):
            V_ref, T_ref = rrf.rrf_panel_qr(h, Y)
            tol = 1e-12 if dtype == torch.float64 else 2e-6
            assert torch.max(torch.abs(V - V_ref)).item() <= tol
            assert torch.max(torch.abs(T - T_ref)).item() <= 10 * tol
            # ... against the CPU oracle's panel factorisation of the same panel ...
            Vo, _, To, _ = orc.panel_qr(Y.cpu().numpy().astype("float64"))
            assert abs(V.double().cpu().numpy() - Vo).max() <= tol
            assert abs(T.double().cpu().numpy() - To).max() <= 10 * tol
            # ... and the factorisation itself is right: (I - V T V^T)^T Y is upper triangular
            Vd, Td, Yd = V.double(), T.double(), Y.double()
            R = Yd - Vd @ (Td.T @ (Vd.T @ Yd))
            assert torch.max(torch.abs(torch.tril(R, -1))).item() <= (1e-11 if dtype == torch.float64 else 1e-4)
    finally:
        rrf.rrf_destroy(h)


def test_static_scratch_rejects_oversized_panels():
    Y = torch.zeros((16, 16), dtype=torch.float64, device="cuda")
    V = torch.empty_like(Y)
    T = torch.empty((16, 16), dtype=torch.float64, device="cuda")
    lib = rrf.load()
    import ctypes as C
    too_tall = lib.rrf_panel_qr_static(rrf.RRF_F64, 70000, 16, C.c_void_p(Y.data_ptr()), 16, C.c_void_p(V.data_ptr()), 16,
                                       C.c_void_p(T.data_ptr()), 16, None)
    assert too_tall == rrf.RRF_ERR_WORKSPACE
    bad_b = lib.rrf_panel_qr_static(rrf.RRF_F64, 64, 24, C.c_void_p(Y.data_ptr()), 24, C.c_void_p(V.data_ptr()), 24,
                                    C.c_void_p(T.data_ptr()), 24, None)
    assert bad_b == rrf.RRF_ERR_INVALID_ARG
