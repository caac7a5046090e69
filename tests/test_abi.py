"""The C-ABI library builds for sm_100a, loads without a GPU and exports every function that
include/meda.h declares; host-side argument checks answer before any CUDA call."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2502_17599_b200 import build, binding
    build.build()
    return binding.load_library()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "meda.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(meda_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound(lib):
    from paper_2502_17599_b200 import binding
    names = declared_functions()
    assert len(names) >= 11
    for name in names:
        assert hasattr(lib, name), name
        assert name in binding.EXPORTS, name
    assert sorted(binding.EXPORTS) == names


def test_status_strings(lib):
    from paper_2502_17599_b200 import binding
    assert binding.status_string(0) == "ok"
    seen = {binding.status_string(s) for s in range(-7, 1)}
    assert len(seen) == 8


def test_create_rejects_bad_arguments_before_touching_the_device(lib):
    from paper_2502_17599_b200 import binding as B
    good = dict(n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=64, n_tokens=100, window=8, dtype="bf16",
                global_budget=50, spans=((0, 10, 0), (10, 90, 1), (90, 100, 0)))

    def status_of(**kw):
        args = dict(good)
        args.update(kw)
        try:
            B.Context(**args)
        except B.MedaError as e:
            return e.status
        return 0

    assert status_of(n_q_heads=3) == B.MEDA_ERR_SHAPE
    assert status_of(head_dim=96) == B.MEDA_ERR_SHAPE
    assert status_of(window=101) == B.MEDA_ERR_SHAPE
    assert status_of(window=200, n_tokens=1000, spans=((0, 1000, 1),), global_budget=500) == B.MEDA_ERR_SHAPE
    # one head's cache of 4 GiB or more (32-bit byte offsets inside a head): 2^24 tokens x 256 dims x 4 bytes
    assert status_of(n_tokens=1 << 24, head_dim=256, dtype="f32", spans=((0, 1 << 24, 1),),
                     global_budget=1 << 20) == B.MEDA_ERR_SHAPE
    assert status_of(global_budget=3) == B.MEDA_ERR_BUDGET_INFEASIBLE
    assert status_of(global_budget=201) == B.MEDA_ERR_BUDGET_INFEASIBLE
    assert status_of(spans=((0, 10, 0), (11, 100, 1))) == B.MEDA_ERR_INVALID_ARG      # gap
    assert status_of(spans=((0, 10, 0), (10, 90, 2), (90, 100, 0))) == B.MEDA_ERR_INVALID_ARG  # bad modality
    assert status_of(spans=((0, 10, 0), (10, 90, 1))) == B.MEDA_ERR_INVALID_ARG        # does not cover
    assert status_of(entropy_mode=2) == B.MEDA_ERR_INVALID_ARG
    assert status_of(beta_recent=0, beta_important=0) == B.MEDA_ERR_INVALID_ARG


def test_null_handles_are_rejected(lib):
    assert lib.meda_poll_status(None, None) == -1
    assert lib.meda_allocate_budgets(None, None, None, None) == -1
    assert lib.meda_window_scores(None, 0, None, None, None, None, None, None) == -1
    assert lib.meda_workspace_bytes(None) == 0
    lib.meda_destroy(None)


def test_product_path_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2502_17599_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "import oracle" not in text and "from oracle" not in text, f


def test_tensor_core_kernels_keep_tensor_memory_loads_out_of_local_memory():
    """The tensor-core kernels keep a tcgen05.ld in flight while they work on the previous registers.  If
    the compiler spilled there, a destination register could be saved before its load has landed, which
    showed up as run-to-run differences when a variant of the arg-max kernel needed more registers than
    its block size allows.  The committed kernels must therefore compile without any spill."""
    import shutil
    import subprocess
    import tempfile
    from paper_2502_17599_b200 import build
    nvcc = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    with tempfile.TemporaryDirectory() as tmp:
        cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "--expt-relaxed-constexpr",
               "-Xptxas", "-v", "-cubin", "-o", os.path.join(tmp, "meda.cubin")] + build.sources()
        res = subprocess.run(cmd, capture_output=True, text=True)
    assert res.returncode == 0, res.stderr
    lines = (res.stdout + res.stderr).splitlines()
    hits = [i for i, line in enumerate(lines)
            if "Function properties" in line and any(name in line for name in (
                "nearest_kernel", "umma_stream_kernel", "window_stats_kernel", "window_sweep_kernel"))]
    assert len(hits) >= 9, "tensor-core kernels not found in the ptxas report"
    for i in hits:
        assert "0 bytes spill stores, 0 bytes spill loads" in lines[i + 1], (lines[i], lines[i + 1])


def test_bench_work_accounting_matches_the_kernels_switch_points():
    """bench.py splits the arg-max flops between the two kernels at the slot count the device code switches
    at, and counts one grouping pass per 9-bit digit of the prompt length."""
    import re
    import bench
    from paper_2502_17599_b200 import binding, workloads as W
    src = open(os.path.join(ROOT, "paper_2502_17599_b200", "csrc", "nearest_sm100.cuh")).read()
    assert int(re.search(r"kNearestSmallMaxS\s*=\s*(\d+)", src).group(1)) == binding.NEAREST_SMALL_MAX_S
    wl = W.WORKLOADS["long_video_128k"]
    n, d, hkv = wl.n_tokens, wl.head_dim, wl.n_kv_heads
    budgets = [36, binding.NEAREST_SMALL_MAX_S, binding.NEAREST_SMALL_MAX_S + 1, 67970]
    work = bench.algorithmic_work(wl, budgets)
    flops = lambda s: 2.0 * (n - s) * s * d * hkv
    assert work["nearest_small_flops"] == [flops(36), flops(binding.NEAREST_SMALL_MAX_S)]
    assert work["nearest_flops"] == [flops(binding.NEAREST_SMALL_MAX_S + 1), flops(67970)]
    assert work["group_bytes"][0] == 1 * 20 * hkv * n                 # 36 slots: one 9-bit digit, all n rows
    assert work["group_bytes"][3] == 2 * 20 * hkv * n                 # 67,970 slots: two digits
    assert all(b == hkv * n * d * 2 for b in work["stats_bytes"])
    # fp32 workloads have no streaming kernel: everything is the generic kernel's
    tiny = bench.algorithmic_work(W.WORKLOADS["tiny"], [100, 200])
    assert tiny["nearest_small_flops"] == [] and len(tiny["nearest_flops"]) == 2
