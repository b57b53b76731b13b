"""One rank of a two-rank data-parallel step on the CPU (gloo), started by dp.spawn_ranks.

It walks through what bench.py does on every rank -- read the launcher's variables, take the token
shard, max-reduce the per-tensor maxima of A and dY in ONE collective, quantize with
index_offset = first_row * cols, all-reduce the int32 sums of dW, scale them once -- with the
oracle's arithmetic in place of the CUDA library.  Rank 0 prints exactly one JSON line.
"""
import json
import os
import sys

import numpy as np
import torch
import torch.distributed as dist

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))

import oracle  # noqa: E402
from oracle import PER_TENSOR, SR, QSpec  # noqa: E402
from paper_2511_00874_b200 import dp  # noqa: E402

T_RANK, N, K = 48, 40, 56


def main():
    rank, local, world = dp.init_from_env("gloo")
    shard = dp.TokenShard(rank, world, T_RANK)
    g = torch.Generator().manual_seed(5)
    A = torch.randn(world * T_RANK, K, generator=g).numpy()
    dY = (torch.randn(world * T_RANK, N, generator=g) * 1e-3).numpy()
    a = A[shard.first_row:shard.first_row + T_RANK]
    dy = dY[shard.first_row:shard.first_row + T_RANK]

    amax = torch.tensor([np.abs(a).max(), np.abs(dy).max()], dtype=torch.float32)
    local_amax = amax.clone()
    dp.reduce_absmax(amax, world)                       # one collective for both operands

    off_a, off_dy = shard.index_offset(K), shard.index_offset(N)
    # the oracle takes a known maximum as one extra row holding it (its codes are dropped)
    qa = QSpec(8, PER_TENSOR, SR, 11, 2, index_offset=off_a)
    qdy = QSpec(8, PER_TENSOR, SR, 11, 4, index_offset=off_dy)
    a_ext = np.concatenate([a, np.full((1, K), amax[0].item(), np.float32)], 0)
    dy_ext = np.concatenate([dy, np.full((1, N), amax[1].item(), np.float32)], 0)
    _, _, ca, sa = oracle.sr_quantize(a_ext, qa, False, True)
    _, _, cdy, sdy = oracle.sr_quantize(dy_ext, qdy, False, True)
    ca, cdy = ca[:, :T_RANK], cdy[:, :T_RANK]
    assert dp.int32_sums_fit(world, T_RANK, 8, 8)
    acc = torch.from_numpy(oracle.gemm_i8_nt(cdy, ca).copy())
    dp.reduce_sum(acc, world)                           # exact: integer sums
    dW = oracle.dequant(acc.numpy(), sdy, sa)           # scaled once, from the total

    info = [None] * world
    dist.gather_object({"rank": rank, "local_rank": local, "first_row": shard.first_row, "index_offset_A": off_a,
                        "index_offset_dY": off_dy, "local_absmax": local_amax.tolist()}, info if rank == 0 else None)
    if rank == 0:
        full = oracle.qlinear_bwd_weight(dY, A, QSpec(8, PER_TENSOR, SR, 11, 4), QSpec(8, PER_TENSOR, SR, 11, 2))
        print(json.dumps({"n_gpus": world, "ranks": info, "reduced_absmax": amax.tolist(),
                          "true_absmax": [float(np.abs(A).max()), float(np.abs(dY).max())],
                          "dW_equal_to_unsharded": bool(np.array_equal(dW, full.out)),
                          "sums_equal_to_unsharded": bool(np.array_equal(acc.numpy(), full.acc))}), flush=True)
    dp.finish()


if __name__ == "__main__":
    if os.environ.get("SRQ_STUB_FAIL_RANK") == os.environ.get("RANK"):
        sys.exit(3)                                     # a rank that never joins: the launcher must end the others
    main()
