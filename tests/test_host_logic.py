"""Host-side logic that needs no GPU: the C ABI loads and exports what the header declares,
argument checks return error codes before any CUDA work, the workload recipes have the stated
shapes, and the multi-rank aggregation of the benchmark works over gloo with two ranks."""
import ctypes
import json
import os
import re
import subprocess
import sys

import numpy as np
import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2104_11125_b200 import build, binding
    build.build()
    return binding.lib()


def test_library_exports_every_declared_symbol(lib):
    from paper_2104_11125_b200 import binding
    header = open(os.path.join(ROOT, "include", "scalecom.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(scalecom_[a-z_]+)\s*\(", header))
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert getattr(lib, name) is not None


def test_binding_constants_equal_the_header_defines():
    """Every SCALECOM_OPT_ / _Q_ / _SELECTOR_ define of the header has a constant of the same value in the binding."""
    from paper_2104_11125_b200 import binding
    header = open(os.path.join(ROOT, "include", "scalecom.h")).read()
    defines = re.findall(r"#define\s+SCALECOM_((?:OPT|Q|SELECTOR)_[A-Z0-9_]+)\s+(-?\d+)", header)
    defines += re.findall(r"SCALECOM_(OK|ERR_[A-Z_]+)\s*=\s*(-?\d+)", header)      # the error enum
    assert len(defines) >= 28
    for name, value in defines:
        assert hasattr(binding, name), "binding lacks %s" % name
        assert getattr(binding, name) == int(value), name


def test_create_rejects_bad_arguments_without_touching_the_gpu(lib):
    from paper_2104_11125_b200 import binding as b
    bad = [
        (0, 1, 1, 0.1, 0.1), (2 ** 31, 1, 1, 0.1, 0.1), (10, 0, 1, 0.1, 0.1), (10, b.MAX_LEARNERS + 1, 1, 0.1, 0.1),
        (10, 1, 0, 0.1, 0.1), (10, 1, 11, 0.1, 0.1), (10, 1, 1, 0.0, 0.1), (10, 1, 1, -0.5, 0.1),
        (10, 1, 1, 1.5, 0.1), (10, 1, 1, float("nan"), 0.1), (10, 1, 1, 0.1, float("inf")), (10, 1, 1, 0.1, float("nan")),
    ]
    for args in bad:
        rc, h = b.scalecom_create(*args)
        assert rc == b.ERR_INVALID_ARG and h is None, args
    assert lib.scalecom_create(None, 10, 1, 1, 0.1, 0.1) == b.ERR_NULL_PTR


def test_null_handles_and_pointers_are_reported(lib):
    from paper_2104_11125_b200 import binding as b
    assert lib.scalecom_step(None, None, None, None, 0, None, None) == b.ERR_NULL_PTR
    assert lib.scalecom_step_host(None, None, None, None, 0, None, None) == b.ERR_NULL_PTR
    assert lib.scalecom_status(None) == b.ERR_NULL_PTR
    assert lib.scalecom_reset(None) == b.ERR_NULL_PTR
    assert lib.scalecom_set_stream(None, None) == b.ERR_NULL_PTR
    assert lib.scalecom_set_gathered(None, None) == b.ERR_NULL_PTR
    assert lib.scalecom_set_option(None, 1, 1) == b.ERR_NULL_PTR
    assert lib.scalecom_query(None, 1, None) == b.ERR_NULL_PTR
    assert lib.scalecom_apply_update(None, None, None, None, 0, 0.0) == b.ERR_NULL_PTR
    lib.scalecom_destroy(None)                                   # accepted
    # allocation-free entry point: size limits and NULLs are checked before any CUDA call
    x = (ctypes.c_float * 4)()
    p = ctypes.addressof(x)
    assert b.scalecom_topk_static(p, p, b.STATIC_MAX_D + 1, 1, p, None, None) == b.ERR_INVALID_ARG
    assert b.scalecom_topk_static(p, p, 4, 5, p, None, None) == b.ERR_INVALID_ARG
    assert b.scalecom_topk_static(p, p, 0, 0, p, None, None) == b.ERR_INVALID_ARG
    assert b.scalecom_topk_static(None, p, 4, 1, p, None, None) == b.ERR_NULL_PTR


def test_strerror_is_total(lib):
    from paper_2104_11125_b200 import binding as b
    seen = {b.strerror(c) for c in range(0, -9, -1)}
    assert len(seen) == 9 and "unknown error" not in seen
    assert b.strerror(-99) == "unknown error"


def test_missing_library_fails_loudly(tmp_path, monkeypatch):
    from paper_2104_11125_b200 import binding as b
    monkeypatch.setattr(b, "_lib", None)
    monkeypatch.setattr(b, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no fallback"):
        b.lib()


def test_workload_shapes():
    from paper_2104_11125_b200 import workloads as W
    seg = W.resnet50_segments()
    assert len(seg) == 161 and sum(seg) == 25_557_032 and min(seg) == 64 and max(seg) == 2_359_296
    assert (W.TINY.n, W.TINY.d, W.TINY.k) == (4, 1 << 20, 10_485)
    assert (W.RESNET50.n, W.RESNET50.k) == (8, 255_570)
    assert (W.TRANSFORMER.n, W.TRANSFORMER.d, W.TRANSFORMER.k) == (16, 61_000_000, 152_500)
    assert (W.LARGE.n, W.LARGE.d, W.LARGE.k) == (32, 354_000_000, 885_000)
    assert [W.sweep(n).n for n in W.SWEEP_N] == [8, 32, 64, 128]
    assert len(W.segments(W.LARGE)) == 24 and sum(s for _, s in W.segments(W.LARGE)) == W.LARGE.d
    for w in (W.RESNET50.scaled(50_001), W.LARGE.scaled(10_007), W.TRANSFORMER.scaled(999)):
        assert sum(s for _, s in W.segments(w)) == w.d


def test_workload_generators_are_seeded_and_correlated():
    from paper_2104_11125_b200 import workloads as W
    for base in (W.TINY, W.RESNET50, W.TRANSFORMER, W.LARGE):
        w = base.scaled(40_000, n=3)
        a = W.gradients(w, 2, "cpu")
        b = W.gradients(w, 2, "cpu")
        c = W.gradients(w, 3, "cpu")
        assert all(torch.equal(x, y) for x, y in zip(a, b))
        assert not torch.equal(a[0], c[0]) and not torch.equal(a[0], a[1])
        cos = torch.nn.functional.cosine_similarity(a[0], a[1], dim=0).item()
        assert abs(cos - 1.0 / (1.0 + w.c ** 2)) < 0.05            # g_i = shared + c * indep_i
        assert torch.equal(W.gradients(w, 2, "cpu", learners=[1])[0], a[1])
    t = W.TRANSFORMER.scaled(200_000)
    p = W.profile(t, "cpu")
    assert abs(p.laplace.float().mean().item() - 0.4) < 0.01


def test_bench_reference_arm_prints_the_contract_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
                          "--steps", "2", "--warmup", "1"], capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert out.returncode == 0, out.stderr
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "learner-elements/s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] == 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["steps"] == 2


def test_bench_reference_arm_keeps_the_workload_and_names_its_sample():
    """The reference arm reports the workload's own n, d, k (so that the two arms' configurations can be compared)
    and says in cpu_baseline.sample whether it ran whole steps or a bounded part of every vector."""
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
                          "--steps", "1", "--warmup", "0"], capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert out.returncode == 0, out.stderr
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert (line["config"]["n"], line["config"]["d"], line["config"]["k"]) == (4, 1 << 20, 10485)
    assert line["cpu_baseline"]["sample"].startswith("full steps of the workload")


def test_learner_sweep_fit_is_a_least_squares_line():
    import bench
    slope, icpt = bench.fit_line([8, 32, 64, 128], [0.05 * n + 0.07 for n in (8, 32, 64, 128)])
    assert abs(slope - 0.05) < 1e-12 and abs(icpt - 0.07) < 1e-12
    slope, icpt = bench.fit_line([1, 2, 3], [1.0, 2.0, 4.0])
    assert abs(slope - 1.5) < 1e-12 and abs(icpt - (7.0 / 3 - 3.0)) < 1e-12


_GLOO_WORKER = r"""
import os, sys
sys.path.insert(0, sys.argv[1])
import torch.distributed as dist
import bench
rank = int(os.environ["RANK"])
dist.init_process_group("gloo")
ms = [10.0 + rank, 3.0 - rank]
got = bench.max_over_ranks(ms)
assert got == [11.0, 3.0], got
val = bench.job_value(8, 1000, dist.get_world_size(), got[0])
assert abs(val - 8 * 1000 * 2 / 11e-3) < 1e-6
dist.barrier()
dist.destroy_process_group()
print("rank", rank, "ok")
"""


def test_replica_aggregation_over_two_gloo_ranks(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(_GLOO_WORKER)
    port = 29500 + os.getpid() % 2000
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script), ROOT], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT, text=True))
    for p in procs:
        out, _ = p.communicate(timeout=180)
        assert p.returncode == 0, out
