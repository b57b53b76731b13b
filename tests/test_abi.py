"""The C-ABI library loads without a GPU, exports every symbol the header declares, and rejects
bad arguments on the host before touching CUDA."""
import ctypes
import os
import re

import pytest

import __graft_entry__ as entry
from paper_2511_00874_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    entry.build()
    return binding.lib()


def _declared():
    text = open(os.path.join(ROOT, "include", "srq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"\b([a-z_0-9]+)\s*\([^;{]*\)\s*;", text)
    return sorted(set(names))


def test_header_symbols_are_exported(L):
    names = _declared()
    assert set(binding.EXPORTS) == set(names), (names, binding.EXPORTS)
    for n in names:
        assert hasattr(L, n), n


def test_status_strings(L):
    seen = {binding.status_string(i) for i in range(8)}
    assert len(seen) == 8 and "ok" in seen
    assert "unknown" in binding.status_string(99)


def test_workspace_sizes_grow_with_the_problem(L):
    small = binding.srq_workspace_bytes(64, 256, 256)
    big = binding.srq_workspace_bytes(4096, 4096, 4096)
    assert 0 < small < big
    # room for both int8 code matrices of the largest pass at least
    assert big >= 2 * 4096 * 4096
    assert binding.srq_workspace_bytes(-1, 1, 1) == 0
    assert binding.srq_quantize_workspace_bytes(128, 128) >= 256 + 4 * 4 * 128
    assert binding.srq_gemm_workspace_bytes(768, 768) >= 256 + 768 * 768 * 4
    # at most the tiles of one partly filled round are split, so the need is bounded whatever the output
    assert binding.srq_gemm_workspace_bytes(65536, 4096) <= 256 + 160 * 128 * 256 * 4
    assert binding.srq_gemm_workspace_bytes(65536, 4096) == binding.srq_gemm_workspace_bytes(1 << 20, 1 << 14)


def test_host_side_argument_checks_need_no_device(L):
    q = binding.QSpec().c()
    fake = 4096          # an "aligned pointer"; the calls below must fail before using it
    f = L.sr_quantize
    r = lambda *a: int(f(*a))
    # null input, null workspace
    assert r(None, 0, 8, 8, 8, ctypes.byref(q), fake, 8, fake, None, 0, None, fake, 1 << 20, None) == binding.ERR_INVALID_ARG
    assert r(fake, 0, 8, 8, 8, ctypes.byref(q), fake, 8, fake, None, 0, None, None, 1 << 20, None) == binding.ERR_INVALID_ARG
    # no output layout requested; pitch smaller than extent; bad dtype
    assert r(fake, 0, 8, 8, 8, ctypes.byref(q), None, 0, None, None, 0, None, fake, 1 << 20, None) == binding.ERR_INVALID_ARG
    assert r(fake, 0, 8, 8, 4, ctypes.byref(q), fake, 8, fake, None, 0, None, fake, 1 << 20, None) == binding.ERR_INVALID_ARG
    assert r(fake, 7, 8, 8, 8, ctypes.byref(q), fake, 8, fake, None, 0, None, fake, 1 << 20, None) == binding.ERR_INVALID_ARG
    # misaligned input pointer, misaligned workspace
    assert r(fake + 4, 0, 8, 8, 8, ctypes.byref(q), fake, 8, fake, None, 0, None, fake, 1 << 20, None) == binding.ERR_INVALID_ARG
    assert r(fake, 0, 8, 8, 8, ctypes.byref(q), fake, 8, fake, None, 0, None, fake + 64, 1 << 20, None) == binding.ERR_INVALID_ARG
    # bits outside 2..8; bad enums
    for bits in (1, 9, 0, -3):
        qb = binding.QSpec(bits=bits).c()
        assert r(fake, 0, 8, 8, 8, ctypes.byref(qb), fake, 8, fake, None, 0, None, fake, 1 << 20, None) == binding.ERR_UNSUPPORTED
    qb = binding.QSpec(scale=5).c()
    assert r(fake, 0, 8, 8, 8, ctypes.byref(qb), fake, 8, fake, None, 0, None, fake, 1 << 20, None) == binding.ERR_INVALID_ARG
    # workspace too small
    assert r(fake, 0, 8, 8, 8, ctypes.byref(q), fake, 8, fake, None, 0, None, fake, 16, None) == binding.ERR_WORKSPACE


def test_the_static_entry_point_applies_the_same_checks_before_anything_is_enqueued(L):
    fake = 4096
    f = L.sr_quantize_static
    r = lambda q, x=fake: int(f(x, 0, 8, 8, 8, ctypes.byref(q), fake, 8, fake, None, 0, None, None, None))
    assert r(binding.QSpec(format=7).c()) == binding.ERR_INVALID_ARG                 # unknown grid
    assert r(binding.QSpec(format=binding.GRID_NONE).c()) == binding.ERR_INVALID_ARG  # a quantizer needs a grid
    assert r(binding.QSpec(bits=4, format=binding.GRID_E4M3).c()) == binding.ERR_UNSUPPORTED   # below E4M0
    assert r(binding.QSpec(round=binding.SR8, format=binding.GRID_E4M3).c()) == binding.ERR_UNSUPPORTED
    assert r(binding.QSpec(round=9).c()) == binding.ERR_INVALID_ARG
    q = binding.QSpec().c()
    q.absmax = fake + 2                                                               # misaligned known maximum
    assert r(q) == binding.ERR_INVALID_ARG
    assert r(binding.QSpec().c(), fake + 4) == binding.ERR_INVALID_ARG                # misaligned input
    assert int(f(fake, 0, 8, 8, 8, None, fake, 8, fake, None, 0, None, None, None)) == binding.ERR_INVALID_ARG


def test_dequant_i32_and_raw_sums_checks(L):
    fake = 4096
    d = L.srq_dequant_i32
    assert int(d(None, 8, 8, 8, fake, 0, fake, 0, fake, 8, 0, None)) == binding.ERR_INVALID_ARG
    assert int(d(fake, 4, 8, 8, fake, 0, fake, 0, fake, 8, 0, None)) == binding.ERR_INVALID_ARG      # pitch < N
    assert int(d(fake, 8, 8, 8, fake, 2, fake, 0, fake, 8, 0, None)) == binding.ERR_INVALID_ARG      # stride not 0 / 1
    assert int(d(fake, 8, 8, 8, fake, 0, fake, 0, fake + 2, 8, 0, None)) == binding.ERR_INVALID_ARG  # fp32 output misaligned
    assert int(d(fake, 8, 8, 8, fake, 0, fake, 0, fake, 8, 3, None)) == binding.ERR_INVALID_ARG
    assert int(d(fake, 8, 0, 8, fake, 0, fake, 0, fake, 8, 0, None)) == binding.OK                   # nothing to do
    o = binding._Output(1, 0, None, None, None, 0, None, 1)                                         # accumulate + raw sums
    g = L.srq_gemm_i8_ex
    assert int(g(fake, 32, fake, 32, 8, 8, 24, fake, 0, fake, 0, fake, 8, None, ctypes.byref(o), fake, 4096, None)) == binding.ERR_UNSUPPORTED


def test_every_kernel_waits_for_its_predecessor_first():
    """Kernels are launched as programmatic dependents of the kernel before them, which is only
    correct if a kernel's first act is the wait (pdl_enter).  Every __global__ function in the
    sources must therefore start with it, except those only ever launched the ordinary way."""
    src_dir = os.path.join(ROOT, "paper_2511_00874_b200", "csrc")
    plain_only = {"bounded_wait_probe_kernel", "clear_static_status"}      # launched with <<< >>>, no attribute
    seen = 0
    for name in sorted(os.listdir(src_dir)):
        text = open(os.path.join(src_dir, name)).read()
        for m in re.finditer(r"__global__\s+void(?:\s+__launch_bounds__\([^)]*(?:\([^)]*\))?[^)]*\))?\s+(\w+)\s*\(", text):
            kernel = m.group(1)
            body = text.index("{", m.end())
            first = text[body + 1:].lstrip().split("\n", 1)[0].strip()
            seen += 1
            if kernel in plain_only:
                assert ("launch_pdl(" + kernel) not in text, kernel
                continue
            if first.startswith("pdl_trigger();"):        # set-up first, then the wait, before any global access
                rest = text[body:text.index("\n}\n", body)]
                assert "pdl_wait();" in rest, f"{name}: {kernel} triggers but never waits"
                before = rest[:rest.index("pdl_wait();")]
                assert not re.search(r"__ldg|__ldc|\bP\.(out|s_row|s_col|acc_out|part|status)\b\s*[\[\+]|tma_load|tma_store|atomic", before), \
                    f"{name}: {kernel} touches global memory before its wait"
                continue
            assert first == "pdl_enter();", f"{name}: {kernel} starts with {first!r}"
    assert seen >= 12


def test_layer_calls_check_overflow_and_workspace_on_the_host(L):
    q8 = binding.QSpec(bits=8).c()
    q4 = binding.QSpec(bits=4).c()
    fake = 4096
    g = L.qlinear_bwd_weight
    # contraction over T: 133145 * 127 * 127 >= 2^31 is refused, 4-bit gradients lift the limit
    assert int(g(fake, fake, 0, 133145, 16, 16, ctypes.byref(q8), ctypes.byref(q8), fake, None, fake, 1 << 40, None)) == binding.ERR_ACC_OVERFLOW
    assert int(g(fake, fake, 0, 133145, 16, 16, ctypes.byref(q4), ctypes.byref(q8), fake, None, fake, 16, None)) == binding.ERR_WORKSPACE
    f = L.qlinear_fwd
    assert int(f(fake, fake, 0, 64, 64, 64, ctypes.byref(q8), ctypes.byref(q8), None, None, fake, 1 << 30, None)) == binding.ERR_INVALID_ARG
    assert int(f(fake, fake, 0, 64, 64, 64, ctypes.byref(q8), None, fake, None, fake, 1 << 30, None)) == binding.ERR_INVALID_ARG
    assert int(f(fake, fake, 0, 64, 64, 64, ctypes.byref(q8), ctypes.byref(q8), fake, None, fake, 1024, None)) == binding.ERR_WORKSPACE
    h = L.srq_gemm_i8
    # pitch not a multiple of 16 breaks the TMA rule
    assert int(h(fake, 24, fake, 32, 8, 8, 24, fake, 0, fake, 0, fake, 8, None, fake, 4096, None)) == binding.ERR_INVALID_ARG
    assert int(h(fake, 32, fake, 32, 8, 8, 24, fake, 0, fake, 2, fake, 8, None, fake, 4096, None)) == binding.ERR_INVALID_ARG


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "libsrq.so"))
    with pytest.raises(RuntimeError, match="no fallback"):
        binding.lib()


def test_split_planning_rule(L):
    """Host logic of the product: which tiles are split along the contraction and into how many parts."""
    plan = binding.srq_plan_splits
    for groups in (74, 148, 1, 7):
        for tiles in list(range(1, 40)) + [73, 74, 75, 148, 176, 222, 256, 512, 600, 4096]:
            for kb in (1, 8, 15, 16, 17, 32, 64, 512):
                full, s = plan(tiles, kb, groups)
                assert 0 <= full <= tiles and s >= 1
                if s == 1:
                    assert full == tiles                      # nothing split
                    continue
                assert full % groups == 0 and full < tiles      # whole rounds first, the rest is split
                per = -(-kb // s)
                assert per >= 8 and (s - 1) * per < kb          # every part has at least 8 k-blocks, none is empty
                assert (tiles - full) * s <= groups or s == kb // 8   # the split units fit into one round
    assert plan(256, 512, 74) == (222, 2)                   # dW of the benchmark layer: last 34 tiles in two parts
    assert plan(9, 512, 74) == (0, 8)                       # 768 x 768 output: every tile in eight parts
    assert plan(4096, 32, 74) == (4096, 1)                  # many rounds: not worth splitting
    assert plan(0, 1, 1) == (0, 0) and plan(5, 0, 3) == (0, 0)
