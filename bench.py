#!/usr/bin/env python
"""Benchmark of the SR-quantized linear layer (forward + both backward products) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

With --gpus N > 1 and no launcher (torch.distributed.run sets RANK / WORLD_SIZE / MASTER_*), the
command starts its own N ranks, one per GPU; under a launcher it is one of the ranks.  Every rank
holds its own 65536-token shard (weak scaling); rank 0 prints the line.

One step = one pass of the whole hot path over one batch: qlinear_fwd (Alg. 1) and qlinear_bwd
(Alg. 2: both backward products) - five absmax reductions and quantizations, three int8
tensor-core products with dequantizing epilogues - on a 4096 x 4096 linear layer with 65536 tokens, fp32 inputs,
8-bit per-tensor stochastic rounding.  Prints one JSON line.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "sr_quantized_linear_fwd_bwd_tops"
UNIT = "TOPS"
WORKLOAD = "linear 4096->4096, tokens 65536, fp32 inputs, 8-bit per-tensor SR on A, W, dY (fwd + bwd)"
T_FULL, N_FULL, K_FULL = 65536, 4096, 4096

# DRAM bytes (read + write) of one gemm_i8_kernel launch of this workload (forward-shaped launch,
# M=65536 N=4096 K=4096) as a profiler capture counted them; not a quantity this run measures.
# None while the kernel has changed since the counters were taken.
GEMM_TRAFFIC_BYTES_PER_LAUNCH = 1332416000


def layer_ops(T, N, K):
    return 6.0 * T * N * K      # three products, 2 T N K integer operations each


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_burst": float(d["bf16_tflops"]),
                "bf16_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_burst": 1590.0, "bf16_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples taken while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.index)],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.splitlines():
            f = [t.strip() for t in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2])); pw.append(float(f[3]))
            except ValueError:
                continue
            for n, v in zip(names, f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        # samples under load: the upper half by power draw
        order = sorted(range(len(sm)), key=lambda i: pw[i])
        loaded = [sm[i] for i in order[len(order) // 2:]]
        return {"sm_mhz": statistics.median(loaded), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "samples": len(sm), "power_w_max": max(pw)}


# ---------------------------------------------------------------------------------------------
# CPU oracle timing (reported baseline and the --impl reference arm)
# ---------------------------------------------------------------------------------------------
def oracle_layer_seconds(T, N, K, seed=0):
    """Seconds the oracle takes for fwd + bwd_input + bwd_weight of a T-token slice."""
    import torch
    import oracle
    from paper_2511_00874_b200 import synth
    A, W, dY = synth.layer_inputs(T, N, K, seed, torch.float32, "cpu", std_dy=1e-3)
    A, W, dY = A.numpy(), W.numpy(), dY.numpy()
    q = [oracle.QSpec(8, oracle.PER_TENSOR, oracle.SR, seed, i) for i in range(5)]
    t0 = time.perf_counter()
    oracle.qlinear_fwd(A, W, q[0], q[1])
    oracle.qlinear_bwd_input(dY, W, q[4], q[3])
    oracle.qlinear_bwd_weight(dY, A, q[4], q[2])
    return time.perf_counter() - t0


def pick_oracle_sample(target_s):
    """(tokens, output features) of the slice of the layer the oracle can do in about target_s
    seconds on this host: as many tokens as fit; output features are cut only when even 256 tokens
    with the whole W (whose quantization does not shrink with the tokens) take longer."""
    Ns = N_FULL
    while True:
        # two probes separate the part that does not grow with the tokens (quantizing W) from the rest
        t1 = oracle_layer_seconds(64, Ns, K_FULL)
        t2 = oracle_layer_seconds(256, Ns, K_FULL)
        if t2 <= target_s or Ns <= 256:
            break
        Ns //= 2
    per_token = max((t2 - t1) / 192.0, 1e-9)
    fixed = max(t1 - 64 * per_token, 0.0)
    Ts = 256
    while Ts * 2 <= T_FULL and fixed + per_token * Ts * 2 <= target_s:
        Ts *= 2
    return Ts, Ns


def cpu_baseline(target_s=15.0):
    import oracle
    Ts, Ns = pick_oracle_sample(target_s)
    sec = oracle_layer_seconds(Ts, Ns, K_FULL)
    return {"value": layer_ops(Ts, Ns, K_FULL) / sec / 1e12, "unit": UNIT, "cores": oracle.num_threads(),
            "kind": "oracle", "seconds": sec,
            "sample": f"same layer (4096->{Ns} of 4096 output features, fp32, 8-bit per-tensor SR), first {Ts} of "
                      f"65536 tokens, fwd + bwd_input + bwd_weight, ops counted as 6*T*N*K"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    oracle.build()
    per_step = max(0.5, min(20.0, 150.0 / max(1, args.steps + args.warmup)))   # the whole run stays within minutes
    Ts, Ns = pick_oracle_sample(per_step)
    for _ in range(args.warmup):
        oracle_layer_seconds(Ts, Ns, K_FULL)
    t0 = time.perf_counter()
    for s in range(args.steps):
        oracle_layer_seconds(Ts, Ns, K_FULL, seed=s)
    sec = (time.perf_counter() - t0) / max(1, args.steps)
    val = layer_ops(Ts, Ns, K_FULL) / sec / 1e12
    sample = (f"CPU oracle on {oracle.num_threads()} host threads; each step = fwd + bwd of the first {Ts} of "
              f"65536 tokens and the first {Ns} of 4096 output features of the same layer (input generation included)")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int8", "data": "synthetic",
        "config": {"workload": WORKLOAD, "sample_tokens": Ts, "sample_out_features": Ns},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))


# ---------------------------------------------------------------------------------------------
# GPU arm
# ---------------------------------------------------------------------------------------------
def needs_spawn(gpus: int) -> bool:
    """True when this process must start the ranks itself: several GPUs asked for, no launcher."""
    from paper_2511_00874_b200 import dp
    return gpus > 1 and not dp.launched_by_env()


def _timed_loop(fn, seconds, est_ms, torch):
    """Runs fn back to back for about `seconds` (count fixed beforehand from est_ms, so that every rank
    runs the same number); returns (ms per call, calls) by CUDA events on the current stream."""
    n = max(3, int(seconds * 1e3 / max(est_ms, 1e-3)) + 1)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(n):
        fn(i)
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / n, n


def run_ours(args):
    import torch
    import torch.distributed as dist

    import paper_2511_00874_b200 as srq
    from paper_2511_00874_b200 import binding, dp, synth

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    binding.lib()                      # fails loudly if libsrq.so is missing
    local = int(os.environ.get("LOCAL_RANK", os.environ.get("RANK", "0")))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    rank, local, world = dp.init_from_env("nccl", dev)

    T, N, K = T_FULL, N_FULL, K_FULL
    shard = dp.TokenShard(rank, world, T)
    peaks = load_peaks()

    # each rank holds its own token shard (weak scaling); W is replicated
    A = synth.normal((T, K), 1.0, 1000 + 3 * rank, torch.float32, dev)
    dY = synth.normal((T, N), 1e-3, 1001 + 3 * rank, torch.float32, dev)
    W = synth.normal((N, K), 0.02, 7, torch.float32, dev)
    Y = torch.empty((T, N), device=dev)
    dA = torch.empty((T, K), device=dev)
    dW = torch.empty((N, K), device=dev)
    ws = srq.new_workspace(srq.srq_workspace_bytes(T, N, K), dev)

    # max |A| and max |dY|: found once per step, max-reduced over the token shards in ONE collective
    # (so that every rank uses the step sizes of the whole batch), and handed to the quantization points
    amax = torch.zeros(2, device=dev)
    amax_a, amax_dy = amax[0:1], amax[1:2]
    # Several ranks: the weight gradient sums over all shards.  While the int32 sums of the whole batch
    # cannot overflow, the ranks all-reduce the exact sums and scale the total once (bit for bit the
    # gradient one GPU computes on the whole batch); otherwise they all-reduce the fp32 gradients.
    exact_dw = world > 1 and dp.int32_sums_fit(world, T, 8, 8)
    sums = torch.empty((N, K), dtype=torch.int32, device=dev) if exact_dw else None
    step_dy, step_a = torch.empty(1, device=dev), torch.empty(1, device=dev)

    def specs(step):
        off_a, off_y = shard.index_offset(K), shard.index_offset(N)       # thresholds follow the global flat index
        return (srq.QSpec(8, srq.PER_TENSOR, srq.SR, step, 0, off_a, absmax=amax_a), srq.QSpec(8, srq.PER_TENSOR, srq.SR, step, 1),
                srq.QSpec(8, srq.PER_TENSOR, srq.SR, step, 2, off_a, absmax=amax_a), srq.QSpec(8, srq.PER_TENSOR, srq.SR, step, 3),
                srq.QSpec(8, srq.PER_TENSOR, srq.SR, step, 4, off_y, absmax=amax_dy))

    def step(i, a=A, w=W, dy=dY, y=Y, da=dA, dw=dW):
        qa_f, qw_f, qa_b, qw_b, qdy = specs(i)
        srq.srq_absmax(a, amax_a)
        srq.srq_absmax(dy, amax_dy)
        dp.reduce_absmax(amax, world)
        srq.qlinear_fwd(a, w, qa_f, qw_f, y, None, ws)
        if exact_dw:
            srq.qlinear_bwd_ex(dy, a, w, qdy, qa_b, qw_b, da, sums, None, None, ws,
                               dbg_weight=srq.DebugOut(scale_a=step_dy, scale_b=step_a))   # raw int32 sums of dW
            dp.reduce_sum(sums, world)
            srq.srq_dequant_i32(sums, step_dy, step_a, dw)
        else:
            srq.qlinear_bwd(dy, a, w, qdy, qa_b, qw_b, da, dw, None, None, ws)      # Alg. 2: both backward products
            dp.reduce_sum(dw, world)   # the batch average of the weight gradient spans all shards

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(v):
        if world == 1:
            return v
        t = torch.tensor([v], device=dev, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return t.item()

    quantizer = None
    if rank == 0:
        # ---- the quantizer alone on the largest tensor of the sweep (2^28 fp32 elements), timed before the
        # long loop so that it runs at the clocks of a kernel timed alone (it is issue-bound, so its speed
        # follows the SM clock, which the power cap lowers once the products run back to back)
        n_q = 1 << 28
        xq = synth.with_outliers((n_q // 4096, 4096), 11, torch.float32, dev)
        cq = torch.empty((n_q // 4096, 4096), dtype=torch.int8, device=dev)
        sq = torch.empty(1, device=dev)
        qws = srq.new_workspace(srq.srq_quantize_workspace_bytes(n_q // 4096, 4096), dev)
        for i in range(5):
            srq.sr_quantize(xq, srq.QSpec(8, 0, 0, i, 9), cq, sq, ws=qws)
        torch.cuda.synchronize()
        q_evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(30)]
        for i, (q0, q1) in enumerate(q_evs):
            q0.record()
            srq.sr_quantize(xq, srq.QSpec(8, 0, 0, i, 9), cq, sq, ws=qws)
            q1.record()
        torch.cuda.synchronize()
        q_ms = statistics.median(q0.elapsed_time(q1) for q0, q1 in q_evs)
        q_bytes = n_q * (4 + 4 + 1)       # absmax read + quantize read + one code layout written
        quantizer = {"bound": "hbm", "achieved": q_bytes / (q_ms * 1e-3) / 1e9, "peak": peaks["hbm_gbs"],
                               "unit": "GB/s", "frac": q_bytes / (q_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                               "ms": q_ms, "workload": "sr_quantize 2^28 fp32, per-tensor 8-bit SR, row-major codes "
                                                       "(absmax pass + quantize pass, 9 bytes per element)"}
        # the same tensor as bfloat16 (5 bytes per element): the case the quantizer's instruction mix, not
        # the memory, decides
        xb = xq.to(torch.bfloat16)
        del xq
        for i in range(5):
            srq.sr_quantize(xb, srq.QSpec(8, 0, 0, i, 9), cq, sq, ws=qws)
        torch.cuda.synchronize()
        for i, (q0, q1) in enumerate(q_evs):
            q0.record()
            srq.sr_quantize(xb, srq.QSpec(8, 0, 0, i, 9), cq, sq, ws=qws)
            q1.record()
        torch.cuda.synchronize()
        qb_ms = statistics.median(q0.elapsed_time(q1) for q0, q1 in q_evs)
        qb_bytes = n_q * (2 + 2 + 1)
        quantizer["bf16"] = {"achieved": qb_bytes / (qb_ms * 1e-3) / 1e9, "frac": qb_bytes / (qb_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                             "ms": qb_ms, "workload": "the same tensor as bfloat16 (5 bytes per element); bound by instruction "
                                                      "dispatch (Philox4x32-10 per four elements), not by HBM"}
        del xb, cq
    for i in range(args.warmup):
        step(i)
    st = srq.srq_poll_status(ws)
    if st != 0:
        raise SystemExit("device status after warm-up: " + srq.status_string(st))

    sampler = ClockSampler(local)
    barrier()
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    barrier()
    l0 = srq.launch_count()
    # the product kernels of the timed steps time themselves on the device (start of the first CTA's
    # work to the end of the last CTA, two atomics per CTA): the dominant kernel's duration INSIDE the step
    timer = srq.new_product_timer(3 * args.steps, dev)
    srq.srq_set_product_timer(timer)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(args.steps):
        step(args.warmup + i)
    e1.record()
    barrier()
    srq.srq_set_product_timer(None)
    launches = srq.launch_count() - l0
    in_step_ms = ((timer[:, 1] - timer[:, 0]).double() * 1e-6).reshape(args.steps, 3).mean(dim=0).tolist()   # fwd, bwd_input, bwd_weight
    ms = max_over_ranks(e0.elapsed_time(e1) / args.steps)
    clocks = sampler.stop() if rank == 0 else None
    st = srq.srq_poll_status(ws)
    if st != 0:
        raise SystemExit("device status after the timed region: " + srq.status_string(st))
    value = world * layer_ops(T, N, K) / (ms * 1e-3) / 1e12

    gathered = None
    if world > 1:
        # which process sat on which device (rank 0 puts the list into the line)
        gathered = [None] * world
        me = {"rank": rank, "local_rank": local, "device": torch.cuda.get_device_name(dev), "pid": os.getpid(),
              "uuid": str(torch.cuda.get_device_properties(dev).uuid), "index_offset_A": shard.index_offset(K)}
        dist.gather_object(me, gathered if rank == 0 else None, dst=0)

    result = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
              "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
              "vs_baseline": None, "dtype": "int8", "data": "synthetic",
              "config": {"workload": WORKLOAD, "tokens_per_gpu": T, "l2": "inputs (1 GiB each) are larger than L2",
                         "absmax": "max |A| and max |dY| are computed once per step (srq_absmax; max-reduced over ranks when "
                                   "N > 1) and handed to their quantization points; max |A| serves both of A's points",
                         "multi_gpu": ("token shards; per step one 2-element all-reduce(max) of the maxima and one all-reduce(sum) of "
                                       + ("the exact int32 sums of dW, scaled once afterwards" if exact_dw else
                                          "the fp32 dW (the int32 sums of the whole batch could overflow)")) if world > 1 else "single GPU",
                         "regime": "the timed region is --steps steps long: a short run is a burst figure (full clocks), "
                                   "see `sustained` for the same step under the power cap"},
              "gpu_launches": int(launches)}
    if gathered is not None and rank == 0:
        result["ranks"] = gathered

    # ---- the same step for at least two seconds: the figure a long training run sees (power cap, lower clocks)
    sus_sampler = ClockSampler(local)
    barrier()
    if rank == 0:
        sus_sampler.start()
    sus_ms, sus_n = _timed_loop(lambda i: step(2000 + i), args.sustained_seconds, ms, torch)
    barrier()
    sus_ms = max_over_ranks(sus_ms)
    sus_clocks = sus_sampler.stop() if rank == 0 else None
    result["sustained"] = {"ms_per_step": sus_ms, "value": world * layer_ops(T, N, K) / (sus_ms * 1e-3) / 1e12, "unit": UNIT,
                           "steps": sus_n, "clocks": sus_clocks}

    # ---- end to end through the public API with host buffers (every rank, max over ranks).
    # Every step copies its inputs from pinned host memory and its results back; the copies of
    # neighbouring steps overlap with the compute on two copy streams (two sets of device buffers).
    hA, hW, hdY = (t.cpu().pin_memory() for t in (A, W, dY))
    hY, hdA, hdW = (torch.empty_like(t, device="cpu").pin_memory() for t in (Y, dA, dW))
    e_steps = max(2, min(32, args.steps))      # enough steps that filling and draining the pipeline weigh little
    ins = [(A, W, dY), tuple(torch.empty_like(t) for t in (A, W, dY))]
    outs = [(Y, dA, dW), tuple(torch.empty_like(t) for t in (Y, dA, dW))]
    s_in, s_out, s_main = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.current_stream()
    ev_in = [torch.cuda.Event() for _ in range(e_steps)]
    ev_comp = [torch.cuda.Event() for _ in range(e_steps)]
    ev_out = [torch.cuda.Event() for _ in range(e_steps)]
    barrier()
    t0 = time.perf_counter()
    for i in range(e_steps):
        b = i % 2
        with torch.cuda.stream(s_in):
            if i >= 2:
                s_in.wait_event(ev_comp[i - 2])           # step i-2 no longer reads these inputs
            for d, h in zip(ins[b], (hA, hW, hdY)):
                d.copy_(h, non_blocking=True)
            ev_in[i].record(s_in)
        s_main.wait_event(ev_in[i])
        if i >= 2:
            s_main.wait_event(ev_out[i - 2])              # the results of step i-2 have left these outputs
        step(1000 + i, *ins[b], *outs[b])
        ev_comp[i].record(s_main)
        with torch.cuda.stream(s_out):
            s_out.wait_event(ev_comp[i])
            for h, d in zip((hY, hdA, hdW), outs[b]):
                h.copy_(d, non_blocking=True)
            ev_out[i].record(s_out)
    torch.cuda.synchronize()
    e_sec = max_over_ranks((time.perf_counter() - t0) / e_steps)
    h2d = sum(t.numel() * 4 for t in (hA, hW, hdY))
    d2h = sum(t.numel() * 4 for t in (hY, hdA, hdW))
    result["e2e"] = {"value": world * layer_ops(T, N, K) / e_sec / 1e12, "unit": UNIT, "h2d_bytes_per_step": h2d,
                     "d2h_bytes_per_step": d2h, "steps": e_steps, "ms_per_step": e_sec * 1e3,
                     "note": "per rank: pinned host A, W, dY copied in and Y, dA, dW copied out every step; "
                             "copies of neighbouring steps overlap with compute (host link bound)"}
    del hA, hW, hdY, hY, hdA, hdW, ins, outs

    if rank == 0:
        # ---- the dominant kernel: the three products of one step, on the codes the quantizer wrote
        one = torch.ones(1, device=dev)

        def codes(x, rows, cols, q, rm, tr):
            crm = torch.empty((rows, cols), dtype=torch.int8, device=dev) if rm else None
            ctr = torch.empty((cols, rows), dtype=torch.int8, device=dev) if tr else None
            s1, s2 = torch.empty(1, device=dev), torch.empty(1, device=dev)
            srq.sr_quantize(x, q, crm, s1 if rm else None, ctr, s2 if tr else None)
            return crm, ctr

        qs = specs(0)
        cA, cAt = codes(A, T, K, qs[0], True, True)
        cW, cWt = codes(W, N, K, qs[1], True, True)
        cdY, cdYt = codes(dY, T, N, qs[4], True, True)
        gemms = [(cA, cW, Y), (cdY, cWt, dA), (cdYt, cAt, dW)]
        gws = srq.new_workspace(max(srq.srq_gemm_workspace_bytes(o.shape[0], o.shape[1]) for _, _, o in gemms), dev)
        for a_, b_, o_ in gemms:
            srq.srq_gemm_i8(a_, b_, one, one, o_, None, gws)
        torch.cuda.synchronize()
        time.sleep(1.0)                          # let the clocks recover from the long loops above
        ops_per_launch = 2.0 * T * N * K

        # burst: every launch bracketed by its own CUDA events on the launching stream, a short series
        b_sampler = ClockSampler(local)
        b_sampler.start()
        time.sleep(0.5)                          # the sampler needs a moment before its first line
        reps = 20
        evs = [[(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in gemms]
               for _ in range(reps)]
        for r in range(reps):
            for j, (a_, b_, o_) in enumerate(gemms):
                evs[r][j][0].record()
                srq.srq_gemm_i8(a_, b_, one, one, o_, None, gws)
                evs[r][j][1].record()
        torch.cuda.synchronize()
        b_clocks = b_sampler.stop()
        gemm_ms = [statistics.mean(evs[r][j][0].elapsed_time(evs[r][j][1]) for r in range(reps)) for j in range(3)]
        launch_ms = statistics.mean(gemm_ms)
        achieved = ops_per_launch / (launch_ms * 1e-3) / 1e12
        peak_burst = 2.0 * peaks["bf16_burst"]        # int8 : bf16 dense nominal ratio is 2

        # sustained: the same three launches back to back for two seconds, against the sustained figure
        s_sampler = ClockSampler(local)
        s_sampler.start()

        def three(_):
            for a_, b_, o_ in gemms:
                srq.srq_gemm_i8(a_, b_, one, one, o_, None, gws)
        s_ms3, s_n = _timed_loop(three, args.sustained_seconds, 3.0 * launch_ms, torch)
        s_clocks = s_sampler.stop()
        s_achieved = ops_per_launch / (s_ms3 / 3.0 * 1e-3) / 1e12
        peak_sus = 2.0 * peaks["bf16_sustained"]
        # the tensor pipe on its own: the same instruction on operands resident in shared memory, no global
        # traffic (single launches, then two seconds back to back)
        mws = srq.new_workspace(256, dev)
        kb = 2048                                # about the duration of one product launch
        mma_ops = srq.srq_selftest_mma_rate(mws, kb)
        torch.cuda.synchronize()
        time.sleep(1.0)
        m_evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(20)]
        for m0, m1 in m_evs:
            m0.record()
            srq.srq_selftest_mma_rate(mws, kb)
            m1.record()
        torch.cuda.synchronize()
        mma_burst = mma_ops / (statistics.mean(m0.elapsed_time(m1) for m0, m1 in m_evs) * 1e-3) / 1e12
        mm_ms, _ = _timed_loop(lambda _i: srq.srq_selftest_mma_rate(mws, kb), args.sustained_seconds, mma_ops / (mma_burst * 1e12) * 1e3, torch)
        mma_sus = mma_ops / (mm_ms * 1e-3) / 1e12
        if srq.srq_poll_status(mws) != 0:
            raise SystemExit("tensor-pipe microbenchmark reported a device-side condition")
        # the headline figure: the products as they ran inside the timed steps; the peak follows the regime
        # of that region (a short region runs at burst clocks, a long one under the power cap)
        in_ms = statistics.mean(in_step_ms)
        in_achieved = ops_per_launch / (in_ms * 1e-3) / 1e12
        long_region = ms * args.steps >= 500.0
        in_peak = 2.0 * (peaks["bf16_sustained"] if long_region else peaks["bf16_burst"])
        result["roofline"] = {
            "bound": "tensor", "kernel": "gemm_i8_kernel", "achieved": in_achieved, "peak": in_peak, "unit": "TOPS",
            "frac": in_achieved / in_peak, "traffic": GEMM_TRAFFIC_BYTES_PER_LAUNCH,
            "traffic_source": "DRAM read + write bytes of one launch from a profiler capture (summary under profiles/), "
                              "not measured by this run",
            "regime": f"inside the {args.steps} timed steps ({ms * args.steps:.0f} ms region): device-side start-to-end time of "
                      f"each of the {3 * args.steps} product launches (srq_set_product_timer)",
            "peak_source": f"2 x {peaks['source']} {'sustained' if long_region else 'burst'} bf16 cuBLAS TFLOP/s (int8:bf16 nominal "
                           "ratio 2); sustained when the timed region is at least 0.5 s long",
            "frac_of_nominal_4500": in_achieved / 4500.0,
            "ms_per_launch": {"fwd": in_step_ms[0], "bwd_input": in_step_ms[1], "bwd_weight": in_step_ms[2]},
            "share_of_step": sum(in_step_ms) / ms,
            "ops_per_launch": ops_per_launch,
            "frac_of_mma_only": in_achieved / (mma_sus if long_region else mma_burst),
            "alone": {"achieved": achieved, "peak": peak_burst, "frac": achieved / peak_burst, "frac_of_mma_only": achieved / mma_burst,
                      "ms_per_launch": {"fwd": gemm_ms[0], "bwd_input": gemm_ms[1], "bwd_weight": gemm_ms[2]}, "clocks": b_clocks,
                      "regime": "burst: 60 launches, each timed alone by CUDA events on the launching stream",
                      "peak_source": f"2 x {peaks['source']} burst bf16 cuBLAS TFLOP/s"},
            "mma_only": {"burst_tops": mma_burst, "sustained_tops": mma_sus,
                         "what": "tcgen05.mma.cta_group::2.kind::i8 M256 N256 K32 on operands resident in shared memory, "
                                 "no global traffic (srq_selftest_mma_rate): the pipe's own ceiling at the clock the power limit allows"},
            "sustained": {"achieved": s_achieved, "peak": peak_sus, "frac": s_achieved / peak_sus,
                          "ms_per_launch": s_ms3 / 3.0, "launches": 3 * s_n, "clocks": s_clocks,
                          "frac_of_mma_only": s_achieved / mma_sus,
                          "peak_source": f"2 x {peaks['source']} sustained bf16 cuBLAS TFLOP/s",
                          "regime": f"the three products back to back for {args.sustained_seconds:g} s (power cap)"}}
        del cA, cAt, cW, cWt, cdY, cdYt

        result["quantizer"] = quantizer
        result["clocks"] = clocks
        if world == 1:
            result["cpu_baseline"] = cpu_baseline()
        print(json.dumps(result), flush=True)
    dp.finish()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--sustained-seconds", type=float, default=2.0,
                    help="length of the back-to-back loops that give the figures under the power cap")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    elif needs_spawn(args.gpus):
        from paper_2511_00874_b200 import dp
        sys.exit(dp.spawn_ranks(args.gpus, [os.path.abspath(__file__), *sys.argv[1:]]))
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
