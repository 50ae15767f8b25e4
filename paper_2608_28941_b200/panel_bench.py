"""Time the panel QR entry points on one Gaussian panel (CUDA events, warm device).

    python -m paper_2608_28941_b200.panel_bench --rows 8192 --b 64 [--dtype f64] [--algo column|blocked|tree|all] [--iters 50]

Prints one JSON line per algorithm: microseconds per call (launch to completion, back to back on one stream),
the bytes the panel occupies and the rate 2 * rows * b * w / time (one read of Y, one write of V), which is the
figure to hold against the HBM bandwidth.
"""
from __future__ import annotations

import argparse
import ctypes as C
import json

import torch

from . import rrf


def time_panel(h, Y: torch.Tensor, algo: str, iters: int) -> float:
    lib = rrf.load()
    rows, b = Y.shape
    dt = rrf._dtype_code(Y)
    need = C.c_size_t()
    lib.rrf_panel_workspace_bytes(dt, rows, b, C.byref(need))
    ws = torch.empty(need.value, dtype=torch.uint8, device=Y.device)
    V = torch.empty_like(Y)
    T = torch.empty((b, b), dtype=Y.dtype, device=Y.device)
    fn = {"column": lib.rrf_panel_qr, "blocked": lib.rrf_panel_qr_blocked, "tree": lib.rrf_panel_qr_tree}[algo]

    def call():
        s = fn(h, dt, rows, b, C.c_void_p(Y.data_ptr()), b, C.c_void_p(V.data_ptr()), b, C.c_void_p(T.data_ptr()), b,
               C.c_void_p(ws.data_ptr()), ws.numel(), rrf._stream())
        if s != rrf.RRF_OK:
            raise rrf.RrfError(s, "panel QR")

    for _ in range(5):
        call()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        call()
    e1.record()
    torch.cuda.synchronize()
    if rrf.rrf_last_status(h) != rrf.RRF_OK:
        raise RuntimeError("device-side status")
    return e0.elapsed_time(e1) / iters * 1e3


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--rows", type=int, default=8192)
    ap.add_argument("--b", type=int, default=64)
    ap.add_argument("--dtype", default="f64", choices=["f64", "f32"])
    ap.add_argument("--algo", default="all", choices=["column", "blocked", "tree", "all"])
    ap.add_argument("--iters", type=int, default=50)
    args = ap.parse_args()
    tdt = torch.float64 if args.dtype == "f64" else torch.float32
    gen = torch.Generator(device="cuda").manual_seed(args.rows + args.b)
    Y = torch.randn((args.rows, args.b), dtype=tdt, device="cuda", generator=gen)
    h = rrf.rrf_create(0)
    try:
        for algo in (["column", "blocked", "tree"] if args.algo == "all" else [args.algo]):
            if algo == "tree" and (args.b > 64 or args.rows * args.b > 35000 * 64):
                continue
            us = time_panel(h, Y, algo, args.iters)
            byts = 2.0 * args.rows * args.b * Y.element_size()
            print(json.dumps({"kernel": "panel_qr", "algo": algo, "rows": args.rows, "b": args.b, "dtype": args.dtype,
                              "us_per_call": us, "algorithmic_bytes": byts, "gb_per_s": byts / (us * 1e-6) / 1e9}))
    finally:
        rrf.rrf_destroy(h)


if __name__ == "__main__":
    main()
