"""Token sharding across ranks (world size 2, gloo, CPU): the recipe `bench.py --gpus N` uses.

Each rank holds half of the tokens of A and dY and a replica of W.  With
index_offset = first_row * cols every rank draws the thresholds its rows have in the unsharded
tensor, so (when the shards share the step size) its codes are the matching rows of the unsharded
codes; Y and dA need no exchange, and the int32 sums of dW add up exactly under one all-reduce.
The arithmetic is the oracle's; what is tested is the sharding rule and the collective.
"""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from oracle import PER_TENSOR, SR, QSpec

T, N, K = 96, 40, 56


def _inputs():
    g = torch.Generator().manual_seed(5)
    A = torch.randn(T, K, generator=g)
    W = torch.randn(N, K, generator=g) * 0.02
    dY = torch.randn(T, N, generator=g) * 1e-3
    # the same absmax in both shards, so that per-tensor step sizes coincide with the unsharded ones
    A[0, 0] = A[T // 2, 0] = 6.0
    dY[1, 1] = dY[T // 2 + 1, 1] = -7e-3
    return A.numpy(), W.numpy(), dY.numpy()


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        A, W, dY = _inputs()
        rows = T // world
        r0 = rank * rows
        a, dy = A[r0:r0 + rows], dY[r0:r0 + rows]
        qa = QSpec(8, PER_TENSOR, SR, 11, 2, index_offset=r0 * K)
        qdy = QSpec(8, PER_TENSOR, SR, 11, 4, index_offset=r0 * N)
        qw = QSpec(8, PER_TENSOR, SR, 11, 3)
        res_w = oracle.qlinear_bwd_weight(dy, a, qdy, qa)
        res_i = oracle.qlinear_bwd_input(dy, W, qdy, qw)
        acc = torch.from_numpy(res_w.acc.copy())
        dist.all_reduce(acc)                                  # exact: integer sums
        dW = torch.from_numpy(res_w.out.copy())
        dist.all_reduce(dW)
        # gather what the checks need on rank 0
        gathered = [None] * world
        dist.gather_object((res_w.codes_a, res_w.codes_b, res_w.scale_a, res_w.scale_b, res_i.out), gathered if rank == 0 else None)
        if rank == 0:
            full_w = oracle.qlinear_bwd_weight(dY, A, QSpec(8, PER_TENSOR, SR, 11, 4), QSpec(8, PER_TENSOR, SR, 11, 2))
            full_i = oracle.qlinear_bwd_input(dY, W, QSpec(8, PER_TENSOR, SR, 11, 4), qw)
            bad = []
            if not np.array_equal(np.concatenate([g[0] for g in gathered], axis=1), full_w.codes_a):
                bad.append("codes of dY^T [N, T]")
            if not np.array_equal(np.concatenate([g[1] for g in gathered], axis=1), full_w.codes_b):
                bad.append("codes of A^T [K, T]")
            if not all(np.array_equal(g[2], full_w.scale_a) and np.array_equal(g[3], full_w.scale_b) for g in gathered):
                bad.append("step sizes")
            if not np.array_equal(acc.numpy(), full_w.acc):
                bad.append("all-reduced int32 sums of dW")
            if not np.array_equal(np.concatenate([g[4] for g in gathered], axis=0), full_i.out):
                bad.append("dA rows")
            # the summed fp32 dW is the dequantized total up to the rounding of the two partial products
            tol = 2.0 ** -22 * np.abs(full_w.out).max()
            if not np.allclose(dW.numpy(), full_w.out, rtol=0, atol=tol):
                bad.append("all-reduced fp32 dW")
            out.put(bad)
    finally:
        dist.destroy_process_group()


def test_token_shards_reproduce_the_unsharded_layer():
    oracle.build()
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    assert out.get(timeout=5) == []


def _worker_per_row(rank, world, port, out):
    """Per-row step sizes: the operands of dW are scaled per column of dY / A, i.e. over the tokens.
    Each rank finds the column maxima of its shard, the ranks max-reduce them, and every rank
    quantizes with the reduced maxima (handed to the oracle as one extra row holding them, which
    makes its own column maxima the global ones; that row's codes are dropped)."""
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        A, W, dY = _inputs()
        rows = T // world
        r0 = rank * rows
        a, dy = A[r0:r0 + rows], dY[r0:r0 + rows]
        col_a = torch.from_numpy(np.abs(a).max(axis=0))
        col_dy = torch.from_numpy(np.abs(dy).max(axis=0))
        dist.all_reduce(col_a, op=dist.ReduceOp.MAX)
        dist.all_reduce(col_dy, op=dist.ReduceOp.MAX)
        from oracle import PER_ROW
        qa = QSpec(8, PER_ROW, SR, 11, 2, index_offset=r0 * K)
        qdy = QSpec(8, PER_ROW, SR, 11, 4, index_offset=r0 * N)
        # transposed layouts of the shard with the reduced maxima
        _, _, ca, sa = oracle.sr_quantize(np.concatenate([a, col_a.numpy()[None, :]], 0), qa, False, True)
        _, _, cdy, sdy = oracle.sr_quantize(np.concatenate([dy, col_dy.numpy()[None, :]], 0), qdy, False, True)
        ca, cdy = ca[:, :rows], cdy[:, :rows]
        acc = torch.from_numpy(oracle.gemm_i8_nt(cdy, ca).copy())
        dist.all_reduce(acc)
        gathered = [None] * world
        dist.gather_object((ca, cdy, sa, sdy, col_a.numpy(), col_dy.numpy()), gathered if rank == 0 else None)
        if rank == 0:
            full = oracle.qlinear_bwd_weight(dY, A, QSpec(8, PER_ROW, SR, 11, 4), QSpec(8, PER_ROW, SR, 11, 2))
            bad = []
            if not (np.array_equal(gathered[0][4], np.abs(A).max(axis=0)) and np.array_equal(gathered[0][5], np.abs(dY).max(axis=0))):
                bad.append("max-reduced column maxima")
            if not np.array_equal(np.concatenate([g[1] for g in gathered], axis=1), full.codes_a):
                bad.append("codes of dY^T [N, T]")
            if not np.array_equal(np.concatenate([g[0] for g in gathered], axis=1), full.codes_b):
                bad.append("codes of A^T [K, T]")
            if not all(np.array_equal(g[3], full.scale_a) and np.array_equal(g[2], full.scale_b) for g in gathered):
                bad.append("column step sizes")
            if not np.array_equal(acc.numpy(), full.acc):
                bad.append("all-reduced int32 sums of dW")
            out.put(bad)
    finally:
        dist.destroy_process_group()


def test_token_shards_with_per_row_steps_exchange_column_maxima():
    oracle.build()
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker_per_row, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    assert out.get(timeout=5) == []
