"""Times one operation of the library on one synthetic case and prints a JSON line.

    python -m paper_2511_00874_b200.cases quantize --rows 16384 --cols 4096 --dtype f32
    python -m paper_2511_00874_b200.cases gemm --M 8192 --N 4096 --K 4096
    python -m paper_2511_00874_b200.cases layer --T 16384 --N 2304 --K 768
    python -m paper_2511_00874_b200.cases mma-peak --k-blocks 2048 --seconds 2

    python -m paper_2511_00874_b200.cases sweep --config 3

`sweep` runs one of the synthetic workload families (2: quantizer sweep, 3: GPT-2-small shaped
layers, 4: Llama-style 1.1B layers in bf16 with per-row scales, 5: batch size against precision
on a 4096 x 4096 layer, with the error of the quantized weight gradient) and prints one JSON
line per case.  The single-case commands are also the small, self-ending commands that profiler
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
    q = B.QSpec(a.bits, B.PER_ROW if per_row else B.PER_TENSOR, {"sr": B.SR, "rtn": B.RTN, "sr8": B.SR8}[a.round], a.seed, 1,
                0, B.GRID_E4M3 if getattr(a, "grid", "int") == "e4m3" else B.GRID_INT)
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
            "round": a.round, "layouts": a.layouts, "grid": getattr(a, "grid", "int"), "ms": med, "ms_best": best, "algorithmic_bytes": nbytes,
            "GBps": nbytes / med / 1e6}


def case_gemm(a):
    g = torch.Generator(device="cuda").manual_seed(a.seed)
    A = torch.randint(-127, 128, (a.M, a.K), generator=g, dtype=torch.int8, device="cuda")
    Bm = torch.randint(-127, 128, (a.N, a.K), generator=g, dtype=torch.int8, device="cuda")
    one = torch.ones(1, device="cuda")
    out_bf16 = getattr(a, "out", "f32") == "bf16"
    out = torch.empty((a.M, a.N), dtype=torch.bfloat16 if out_bf16 else torch.float32, device="cuda")
    ws = B.new_workspace(B.srq_gemm_workspace_bytes(a.M, a.N))
    if getattr(a, "grid", "int") == "e4m3":
        A, Bm = A.view(torch.uint8), Bm.view(torch.uint8)
        A[(A & 0x7F) == 0x7F] = 0x38          # no NaN codes
        Bm[(Bm & 0x7F) == 0x7F] = 0x38
        fn = lambda: B.srq_gemm_e4m3(A, Bm, one, one, out, None, ws)
    elif out_bf16:
        fn = lambda: B.srq_gemm_i8_ex(A, Bm, one, one, out, None, None, ws)
    else:
        fn = lambda: B.srq_gemm_i8(A, Bm, one, one, out, None, ws)
    small = (a.M + a.N) * a.K + 4 * a.M * a.N < 2 * L2_BYTES
    med, best = _time(fn, a.iters, a.warmup, flush=small)
    assert B.srq_poll_status(ws) == 0
    ops = 2.0 * a.M * a.N * a.K
    return {"op": "srq_gemm_e4m3" if getattr(a, "grid", "int") == "e4m3" else "srq_gemm_i8", "M": a.M, "N": a.N, "K": a.K, "ms": med, "ms_best": best, "TOPS": ops / med / 1e9,
            "out": "bf16" if out_bf16 else "f32", "out_GBps": out.element_size() * a.M * a.N / med / 1e6}


def case_mma_peak(a):
    """The ceiling of the tensor pipe for the products' instruction (kind::i8, CTA pairs, M256 N256 K32):
    operands resident in shared memory, no global traffic.  `ms` is the median of single launches
    (burst clocks); with --seconds S the launch is also repeated back to back for S seconds, which
    is what the power limit sustains."""
    ws = B.new_workspace(256)
    ops = B.srq_selftest_mma_rate(ws, a.k_blocks)
    med, best = _time(lambda: B.srq_selftest_mma_rate(ws, a.k_blocks), a.iters, a.warmup, flush=False)
    assert B.srq_poll_status(ws) == 0
    r = {"op": "mma-peak", "k_blocks": a.k_blocks, "ops_per_launch": ops, "ms": med, "ms_best": best, "TOPS": ops / med / 1e9}
    if a.seconds > 0:
        n = max(3, int(a.seconds * 1e3 / med))
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(n):
            B.srq_selftest_mma_rate(ws, a.k_blocks)
        e1.record()
        torch.cuda.synchronize()
        assert B.srq_poll_status(ws) == 0
        r.update({"sustained_launches": n, "sustained_ms": e0.elapsed_time(e1) / n, "sustained_TOPS": ops * n / e0.elapsed_time(e1) / 1e9})
    return r


def _layer_fn(A, W, dY, q, Y, dA, dW, ws):
    def fn():
        B.qlinear_fwd(A, W, q["a_fwd"], q["w_fwd"], Y, None, ws)
        B.qlinear_bwd(dY, A, W, q["dy"], q["a_bwd"], q["w_bwd"], dA, dW, None, None, ws)
    return fn


def _layer_specs(bits_fwd, bits_bwd, sc, rd, seed, grid="int"):
    fmt = B.GRID_E4M3 if grid == "e4m3" else B.GRID_INT
    return {k: B.QSpec(b, sc, rd, seed, i, 0, fmt) for i, (k, b) in enumerate(
        [("a_fwd", bits_fwd), ("w_fwd", bits_fwd), ("a_bwd", bits_bwd), ("w_bwd", bits_bwd), ("dy", bits_bwd)])}


def case_layer(a):
    dt = torch.float32 if a.dtype == "f32" else torch.bfloat16
    A, W, dY = synth.layer_inputs(a.T, a.N, a.K, a.seed, dt, "cuda", std_dy=1e-3)
    sc = B.PER_ROW if a.scale == "row" else B.PER_TENSOR
    rd = {"sr": B.SR, "rtn": B.RTN, "sr8": B.SR8}[a.round]
    q = _layer_specs(a.bits_fwd, a.bits_bwd, sc, rd, a.seed, getattr(a, "grid", "int"))
    Y = torch.empty((a.T, a.N), device="cuda")
    dA = torch.empty((a.T, a.K), device="cuda")
    dW = torch.empty((a.N, a.K), device="cuda")
    ws = B.new_workspace(B.srq_workspace_bytes(a.T, a.N, a.K))
    fn = _layer_fn(A, W, dY, q, Y, dA, dW, ws)
    if getattr(a, "graph", False):
        # the calls only enqueue work on the stream, so a caller can record them once in a CUDA graph and
        # replay it: for small layers this removes most of the per-launch cost
        fn()                                     # first call outside the capture (one-time device set-up)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            fn()
        fn = g.replay
    small = (A.numel() + dY.numel()) * A.element_size() < 2 * L2_BYTES
    med, best = _time(fn, a.iters, a.warmup, flush=small)
    assert B.srq_poll_status(ws) == 0
    ops = 6.0 * a.T * a.N * a.K
    return {"op": "layer fwd+bwd", "T": a.T, "N": a.N, "K": a.K, "dtype": a.dtype, "bits_fwd": a.bits_fwd,
            "bits_bwd": a.bits_bwd, "scale": a.scale, "round": a.round, "grid": getattr(a, "grid", "int"), "graph": bool(getattr(a, "graph", False)),
            "ms": med, "ms_best": best, "TOPS": ops / med / 1e9}


# ---------------------------------------------------------------------------------------------
# workload families
# ---------------------------------------------------------------------------------------------
def _ns(**kw):
    return argparse.Namespace(**kw)


def sweep_quantizer(a):
    """Config 2: 2^20 .. 2^28 elements as [n / 4096, 4096], fp32 and bf16, bits 8 / 6 / 4, per tensor and
    per row, SR and RTN, seeds 0-3 (median over the seeds)."""
    for logn in (20, 22, 24, 26, 28):
        rows = (1 << logn) // 4096
        for dtype in ("f32", "bf16"):
            for bits in (8, 6, 4):
                for scale in ("tensor", "row"):
                    for rnd in ("sr", "rtn"):
                        ms, gb = [], []
                        for seed in range(4):
                            r = case_quantize(_ns(rows=rows, cols=4096, dtype=dtype, bits=bits, scale=scale, round=rnd,
                                                  layouts="rm", seed=seed, iters=a.iters, warmup=a.warmup))
                            ms.append(r["ms"]); gb.append(r["GBps"])
                        yield {"config": 2, "elements": 1 << logn, "dtype": dtype, "bits": bits, "scale": scale,
                               "round": rnd, "ms": statistics.median(ms), "GBps": statistics.median(gb)}


def sweep_gpt2(a):
    """Config 3: GPT-2-small shaped layers, fp32, 8-bit per-tensor SR on W, A and dY."""
    for name, (K, N) in synth.GPT2_SMALL_LAYERS.items():
        for batch in (1, 4, 16, 64):
            r = case_layer(_ns(T=batch * 1024, N=N, K=K, dtype="f32", bits_fwd=8, bits_bwd=8, scale="tensor", round="sr",
                               seed=0, iters=a.iters, warmup=a.warmup))
            r.update({"config": 3, "layer": name})
            yield r


def sweep_llama(a):
    """Config 4: Llama-style 1.1B layers, bf16 inputs, per-row scales, 8-bit forward, 4-bit SR backward."""
    for name, (K, N) in synth.LLAMA_1B_LAYERS.items():
        if name == "up":
            continue                     # same shape as gate
        for batch in (1, 8, 32):
            r = case_layer(_ns(T=batch * 2048, N=N, K=K, dtype="bf16", bits_fwd=8, bits_bwd=4, scale="row", round="sr",
                               seed=0, iters=a.iters, warmup=a.warmup))
            r.update({"config": 4, "layer": name + ("/up" if name == "gate" else "")})
            yield r


def _rounding_variance(x, bits):
    """Mean over the tensor of the variance SR adds to one element, D^2 p (1 - p) (per-tensor step)."""
    m = x.abs().max()
    qmax = float((1 << (bits - 1)) - 1)
    d = m / qmax
    t = x / d
    p = t - torch.floor(t)
    return float((d * d * (p * (1 - p)).mean()).item())


def sweep_batch_precision(a):
    """Config 5: 4096 x 4096 layer, tokens 512 .. 65536, bits 8 / 6 / 4 / 3, SR and RTN, 5 seeds.  Besides the
    throughput, the mean squared error of the quantized dW / T against the unquantized dY^T A / T
    (binary64), next to what the variance lemma (Lemma 3) predicts for SR:
    (E[A^2] var_dY + E[dY^2] var_A + var_A var_dY) / T with var_X the mean rounding variance of X."""
    N = K = 4096
    for T in (512, 1024, 2048, 4096, 8192, 16384, 32768, 65536):
        A, W, dY = synth.layer_inputs(T, N, K, 0, torch.float32, "cuda", std_dy=1e-3)
        ref = torch.zeros((N, K), dtype=torch.float64, device="cuda")
        for i in range(0, T, 8192):                        # binary64 in slices to bound memory
            ref += dY[i:i + 8192].double().t() @ A[i:i + 8192].double()
        ref /= T
        Y = torch.empty((T, N), device="cuda")
        dA = torch.empty((T, K), device="cuda")
        dW = torch.empty((N, K), device="cuda")
        ws = B.new_workspace(B.srq_workspace_bytes(T, N, K))
        ea2, edy2 = float((A.double() ** 2).mean()), float((dY.double() ** 2).mean())
        for bits in (8, 6, 4, 3):
            va, vdy = _rounding_variance(A, bits), _rounding_variance(dY, bits)
            predicted = (ea2 * vdy + edy2 * va + va * vdy) / T
            for rnd in ("sr", "rtn"):
                mses, times = [], []
                for seed in range(5):
                    q = _layer_specs(bits, bits, B.PER_TENSOR, B.SR if rnd == "sr" else B.RTN, seed)
                    fn = _layer_fn(A, W, dY, q, Y, dA, dW, ws)
                    med, _ = _time(fn, max(3, a.iters // 4), 2, flush=T < 8192)
                    times.append(med)
                    mses.append(float((((dW.double() / T) - ref) ** 2).mean()))
                assert B.srq_poll_status(ws) == 0
                ms = statistics.median(times)
                yield {"config": 5, "T": T, "bits": bits, "round": rnd, "ms": ms, "TOPS": 6.0 * T * N * K / ms / 1e9,
                       "dW_mse": statistics.mean(mses), "dW_mse_min": min(mses), "dW_mse_max": max(mses),
                       "lemma3_sr_variance": predicted, "dW_ref_mean_square": float((ref ** 2).mean())}
        del A, W, dY, Y, dA, dW, ws, ref


def case_sweep(a):
    gen = {2: sweep_quantizer, 3: sweep_gpt2, 4: sweep_llama, 5: sweep_batch_precision}[a.config](a)
    for r in gen:
        print(json.dumps(r), flush=True)
    return None


def main(argv=None):
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    sub = ap.add_subparsers(dest="op", required=True)
    for name in ("quantize", "gemm", "layer", "sweep", "mma-peak"):
        p = sub.add_parser(name)
        p.add_argument("--iters", type=int, default=20)
        p.add_argument("--warmup", type=int, default=3)
        p.add_argument("--seed", type=int, default=0)
        p.add_argument("--grid", default="int", choices=["int", "e4m3"])
        if name == "quantize":
            p.add_argument("--rows", type=int, default=16384)
            p.add_argument("--cols", type=int, default=4096)
            p.add_argument("--layouts", default="rm", choices=["rm", "tr", "both"])
            p.add_argument("--bits", type=int, default=8)
        if name == "gemm":
            p.add_argument("--M", type=int, default=8192)
            p.add_argument("--N", type=int, default=4096)
            p.add_argument("--K", type=int, default=4096)
            p.add_argument("--out", default="f32", choices=["f32", "bf16"], help="type the product is stored in (int grid only)")
        if name == "layer":
            p.add_argument("--T", type=int, default=16384)
            p.add_argument("--N", type=int, default=4096)
            p.add_argument("--K", type=int, default=4096)
            p.add_argument("--bits-fwd", dest="bits_fwd", type=int, default=8)
            p.add_argument("--bits-bwd", dest="bits_bwd", type=int, default=8)
            p.add_argument("--graph", action="store_true", help="record the step in a CUDA graph and time its replay")
        if name == "sweep":
            p.add_argument("--config", type=int, required=True, choices=[2, 3, 4, 5])
        if name == "mma-peak":
            p.add_argument("--k-blocks", dest="k_blocks", type=int, default=2048, help="128-byte blocks of contraction per CTA pair")
            p.add_argument("--seconds", type=float, default=0.0, help="also repeat the launch back to back for this long")
        if name not in ("gemm", "sweep", "mma-peak"):
            p.add_argument("--dtype", default="f32", choices=["f32", "bf16"])
            p.add_argument("--scale", default="tensor", choices=["tensor", "row"])
            p.add_argument("--round", default="sr", choices=["sr", "rtn", "sr8"])
    a = ap.parse_args(argv)
    if not torch.cuda.is_available():
        raise SystemExit("a CUDA device is required (there is no CPU fallback)")
    res = {"quantize": case_quantize, "gemm": case_gemm, "layer": case_layer, "sweep": case_sweep, "mma-peak": case_mma_peak}[a.op](a)
    if res is not None:
        print(json.dumps(res))


if __name__ == "__main__":
    main()
