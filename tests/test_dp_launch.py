"""The multi-rank launch path of `bench.py --gpus N` without GPUs: dp.spawn_ranks starts the
ranks, each finds its shard from the launcher's variables, and rank 0 prints the one line."""
import json
import os
import subprocess
import sys

import oracle
from paper_2511_00874_b200 import dp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
STUB = os.path.join(ROOT, "tests", "_rank_stub.py")


def _run_spawner(n, extra_env=None):
    """spawn_ranks in a child interpreter, so that the ranks' output can be captured."""
    code = ("import sys; sys.path.insert(0, %r); from paper_2511_00874_b200 import dp; "
            "sys.exit(dp.spawn_ranks(%d, [%r], timeout=150))" % (ROOT, n, STUB))
    env = {k: v for k, v in os.environ.items() if k not in dp.LAUNCH_VARS}
    env.update(extra_env or {})
    return subprocess.run([sys.executable, "-c", code], capture_output=True, text=True, env=env, timeout=200)


def test_two_ranks_take_their_shards_and_rank0_prints_one_line():
    oracle.build()
    r = _run_spawner(2)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.strip()]
    assert len(lines) == 1, r.stdout
    out = json.loads(lines[0])
    assert out["n_gpus"] == 2
    ranks = sorted(out["ranks"], key=lambda d: d["rank"])
    assert [d["rank"] for d in ranks] == [0, 1] and [d["local_rank"] for d in ranks] == [0, 1]
    assert [d["first_row"] for d in ranks] == [0, 48]
    assert [d["index_offset_A"] for d in ranks] == [0, 48 * 56]          # first_row * cols of A[T, K]
    assert [d["index_offset_dY"] for d in ranks] == [0, 48 * 40]         # first_row * cols of dY[T, N]
    # one collective delivered both maxima, and they are those of the whole batch
    assert out["reduced_absmax"] == out["true_absmax"]
    for i in range(2):
        assert out["reduced_absmax"][i] == max(d["local_absmax"][i] for d in ranks)
    # integer sums add exactly, so the weight gradient scaled from the total equals the unsharded one
    assert out["sums_equal_to_unsharded"] and out["dW_equal_to_unsharded"]


def test_a_failing_rank_ends_the_launch_with_its_exit_code():
    r = _run_spawner(2, {"SRQ_STUB_FAIL_RANK": "1"})
    assert r.returncode == 3
    assert r.stdout.strip() == ""


def test_shard_offsets_and_the_int32_bound():
    s = dp.TokenShard(rank=3, world=8, tokens=65536)
    assert s.first_row == 3 * 65536 and s.index_offset(4096) == 3 * 65536 * 4096
    assert dp.int32_sums_fit(2, 65536, 8, 8) and not dp.int32_sums_fit(4, 65536, 8, 8)
    assert dp.int32_sums_fit(8, 65536, 8, 4) and not dp.int32_sums_fit(64, 65536, 8, 4)      # 8 * 65536 * 127 * 7 < 2^31


def test_bench_refuses_to_count_ranks_it_did_not_start(monkeypatch):
    """`bench.py --gpus N` with no launcher variables re-launches itself N times; with them it is a rank."""
    import importlib.util
    spec = importlib.util.spec_from_file_location("bench_under_test", os.path.join(ROOT, "bench.py"))
    bench = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(bench)
    for v in dp.LAUNCH_VARS:
        monkeypatch.delenv(v, raising=False)
    assert bench.needs_spawn(4) and not bench.needs_spawn(1)
    monkeypatch.setenv("WORLD_SIZE", "4")
    monkeypatch.setenv("RANK", "2")
    assert not bench.needs_spawn(4)
