"""Times one operation of the library on one synthetic case and prints a JSON line.

    python -m paper_2511_00874_b200.cases quantize --rows 16384 --cols 4096 --dtype f32
    python -m paper_2511_00874_b200.cases gemm --M 8192 --N 4096 --K 4096
    python -m paper_2511_00874_b200.cases layer --T 16384 --N 2304 --K 768

Used for the per-configuration sweeps and as the small, self-ending command that profiler
captures are taken on.  Timing is by CUDA events on the launching stream; between iterations a
buffer larger than L2 is rewritten unless the case's own inputs exceed L2.
"""
from __future__ import annotations

import argparse
import json
import statistics

import torch

from . import binding as B
from . import synth

L2_BYTES = 126 * 1024 * 1024


def _time(fn, iters, warmup, flush):
    scratch = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device="cuda") if flush else None
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    ms = []
    for _ in range(iters):
        if scratch is not None:
            scratch.fill_(1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        torch.cuda.synchronize()
        ms.append(e0.elapsed_time(e1))
    return statistics.median(ms), min(ms)


def case_quantize(a):
    dt = torch.float32 if a.dtype == "f32" else torch.bfloat16
    x = synth.with_outliers((a.rows, a.cols), a.seed, dt, "cuda")
    per_row = a.scale == "row"
    q = B.QSpec(a.bits, B.PER_ROW if per_row else B.PER_TENSOR, B.SR if a.round == "sr" else B.RTN, a.seed, 1)
    rm, tr = a.layouts in ("rm", "both"), a.layouts in ("tr", "both")
    crm = torch.empty((a.rows, a.cols), dtype=torch.int8, device="cuda") if rm else None
    ctr = torch.empty((a.cols, a.rows), dtype=torch.int8, device="cuda") if tr else None
    srm = torch.empty(a.rows if per_row else 1, device="cuda") if rm else None
    st = torch.empty(a.cols if per_row else 1, device="cuda") if tr else None
    ws = B.new_workspace(B.srq_quantize_workspace_bytes(a.rows, a.cols))
    fn = lambda: B.sr_quantize(x, q, crm, srm, ctr, st, ws)
    n = a.rows * a.cols
    e = x.element_size()
    med, best = _time(fn, a.iters, a.warmup, flush=n * e < 2 * L2_BYTES)
    assert B.srq_poll_status(ws) == 0
    nbytes = n * (2 * e + int(rm) + int(tr))       # absmax read + quantize read + code layouts written
    return {"op": "sr_quantize", "rows": a.rows, "cols": a.cols, "dtype": a.dtype, "bits": a.bits, "scale": a.scale,
            "round": a.round, "layouts": a.layouts, "ms": med, "ms_best": best, "algorithmic_bytes": nbytes,
            "GBps": nbytes / med / 1e6}


def case_gemm(a):
    g = torch.Generator(device="cuda").manual_seed(a.seed)
    A = torch.randint(-127, 128, (a.M, a.K), generator=g, dtype=torch.int8, device="cuda")
    Bm = torch.randint(-127, 128, (a.N, a.K), generator=g, dtype=torch.int8, device="cuda")
    one = torch.ones(1, device="cuda")
    out = torch.empty((a.M, a.N), device="cuda")
    ws = B.new_workspace(B.srq_gemm_workspace_bytes(a.M, a.N))
    fn = lambda: B.srq_gemm_i8(A, Bm, one, one, out, None, ws)
    small = (a.M + a.N) * a.K + 4 * a.M * a.N < 2 * L2_BYTES
    med, best = _time(fn, a.iters, a.warmup, flush=small)
    assert B.srq_poll_status(ws) == 0
    ops = 2.0 * a.M * a.N * a.K
    return {"op": "srq_gemm_i8", "M": a.M, "N": a.N, "K": a.K, "ms": med, "ms_best": best, "TOPS": ops / med / 1e9,
            "out_GBps": 4.0 * a.M * a.N / med / 1e6}


def case_layer(a):
    dt = torch.float32 if a.dtype == "f32" else torch.bfloat16
    A, W, dY = synth.layer_inputs(a.T, a.N, a.K, a.seed, dt, "cuda", std_dy=1e-3)
    sc = B.PER_ROW if a.scale == "row" else B.PER_TENSOR
    rd = B.SR if a.round == "sr" else B.RTN
    q = {k: B.QSpec(b, sc, rd, a.seed, i) for i, (k, b) in enumerate(
        [("a_fwd", a.bits_fwd), ("w_fwd", a.bits_fwd), ("a_bwd", a.bits_bwd), ("w_bwd", a.bits_bwd),
         ("dy", a.bits_bwd)])}
    Y = torch.empty((a.T, a.N), device="cuda")
    dA = torch.empty((a.T, a.K), device="cuda")
    dW = torch.empty((a.N, a.K), device="cuda")
    ws = B.new_workspace(B.srq_workspace_bytes(a.T, a.N, a.K))

    def fn():
        B.qlinear_fwd(A, W, q["a_fwd"], q["w_fwd"], Y, None, ws)
        B.qlinear_bwd_input(dY, W, q["dy"], q["w_bwd"], dA, None, ws)
        B.qlinear_bwd_weight(dY, A, q["dy"], q["a_bwd"], dW, None, ws)

    small = (A.numel() + dY.numel()) * A.element_size() < 2 * L2_BYTES
    med, best = _time(fn, a.iters, a.warmup, flush=small)
    assert B.srq_poll_status(ws) == 0
    ops = 6.0 * a.T * a.N * a.K
    return {"op": "layer fwd+bwd", "T": a.T, "N": a.N, "K": a.K, "dtype": a.dtype, "bits_fwd": a.bits_fwd,
            "bits_bwd": a.bits_bwd, "scale": a.scale, "round": a.round, "ms": med, "ms_best": best,
            "TOPS": ops / med / 1e9}


def main(argv=None):
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    sub = ap.add_subparsers(dest="op", required=True)
    for name in ("quantize", "gemm", "layer"):
        p = sub.add_parser(name)
        p.add_argument("--iters", type=int, default=20)
        p.add_argument("--warmup", type=int, default=3)
        p.add_argument("--seed", type=int, default=0)
        if name == "quantize":
            p.add_argument("--rows", type=int, default=16384)
            p.add_argument("--cols", type=int, default=4096)
            p.add_argument("--layouts", default="rm", choices=["rm", "tr", "both"])
            p.add_argument("--bits", type=int, default=8)
        if name == "gemm":
            p.add_argument("--M", type=int, default=8192)
            p.add_argument("--N", type=int, default=4096)
            p.add_argument("--K", type=int, default=4096)
        if name == "layer":
            p.add_argument("--T", type=int, default=16384)
            p.add_argument("--N", type=int, default=4096)
            p.add_argument("--K", type=int, default=4096)
            p.add_argument("--bits-fwd", dest="bits_fwd", type=int, default=8)
            p.add_argument("--bits-bwd", dest="bits_bwd", type=int, default=8)
        if name != "gemm":
            p.add_argument("--dtype", default="f32", choices=["f32", "bf16"])
            p.add_argument("--scale", default="tensor", choices=["tensor", "row"])
            p.add_argument("--round", default="sr", choices=["sr", "rtn"])
    a = ap.parse_args(argv)
    if not torch.cuda.is_available():
        raise SystemExit("a CUDA device is required (there is no CPU fallback)")
    res = {"quantize": case_quantize, "gemm": case_gemm, "layer": case_layer}[a.op](a)
    print(json.dumps(res))


if __name__ == "__main__":
    main()
