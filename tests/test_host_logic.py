"""CPU-only checks of the host logic: the shared library loads and exports every symbol the public
headers declare, the planner's shape -> order rule, argument rejection, and the benchmark's
multi-process plumbing (gloo, world size 2).  No compute call is made: there is no GPU here."""
import ctypes
import json
import os
import re
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def built_lib():
    import __graft_entry__ as entry
    entry.build()
    from paper_2609_25624_b200 import binding
    return binding


def declared_symbols():
    names = []
    for hdr in sorted(os.listdir(os.path.join(ROOT, "include"))):
        if not hdr.endswith(".h"):
            continue
        text = open(os.path.join(ROOT, "include", hdr)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names += re.findall(r"DET_API\s+[\w\s\*]+?\b(det_\w+)\s*\(", text)
    return names


def test_library_exports_every_declared_symbol(built_lib):
    names = declared_symbols()
    assert len(names) >= 16 and "det_linear_run" in names and "det_argmax_rows" in names
    lib = ctypes.CDLL(built_lib.LIB_PATH)
    for n in names:
        assert getattr(lib, n) is not None, n


def test_plan_params_rule_and_oracle_agree(built_lib):
    from oracle import oracle
    B = built_lib
    for M in (1, 2, 7, 32, 64, 65, 100, 128, 512, 2048, 5000):
        for N in (1, 7, 100, 1000, 1024, 4095, 4096, 6144, 28672, 128256):
            for K in (1, 7, 8, 255, 256, 257, 512, 1000, 3072, 4096, 14336):
                p = B.det_linear_plan_params(M, N, K)
                assert p.as_dict() == oracle.order_params(M, N, K), (M, N, K)
                assert p.workspace_bytes == (4 * p.S * M * N if p.S > 1 else 0)
                assert p.kernel == (0 if K % 8 else (1 if M <= 64 else 2))
    # decode parameters never read M (rule R4)
    ref = B.det_linear_plan_params(1, 1024, 512).as_dict()
    for M in range(1, 65):
        assert B.det_linear_plan_params(M, 1024, 512).as_dict() == ref


def test_bad_shapes_are_rejected_with_a_message(built_lib):
    B = built_lib
    for shp in [(0, 1, 1), (1, 0, 1), (1, 1, 0), (-3, 4, 8), (1, 1 << 31, 8), (1 << 21, 1 << 21, 8)]:
        with pytest.raises(B.DetLinearError) as ei:
            B.det_linear_plan_params(*shp)
        assert ei.value.status in (1, 2)
        assert B.det_last_error() != ""
    rc = B.lib().det_linear_plan_params(1, 1, 8, None)
    assert rc == 1
    assert B.det_order_version() == 1


def test_null_arguments_do_not_touch_the_device(built_lib):
    lib = built_lib.lib()
    assert lib.det_linear_run(None, None, None, None, None, None) == 1
    assert lib.det_linear_run_host(None, None, None, None, None, None) == 1
    assert lib.det_argmax_rows(None, 1, 1, None, None) == 1
    assert lib.det_linear_plan_check(None, None) == 1
    assert lib.det_linear_plan_describe(None, None, 0) == 1
    lib.det_linear_plan_destroy(None)


def test_bench_workload_definition():
    sys.path.insert(0, ROOT)
    import bench
    cases = bench.decode_cases()
    assert len(cases) == 20
    assert sum(2 * N * K for (_, N, K, _) in cases) == 5 * 2 * (6144 * 4096 + 4096 * 4096 + 28672 * 4096 + 4096 * 14336)
    assert bench.algorithmic_bytes(1, 2, 8) == 2 * 2 * 8 + 4 * 8 + 4 * 2 + 4 * 2
    assert abs(bench.fp32_peak_tflops(148) - 74.45) < 0.01


def test_bench_reference_arm_runs_on_cpu():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                          "--warmup", "0", "--ref-cols", "8"], capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert out.returncode == 0, out.stderr
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0


_GLOO_WORKER = r"""
import os, sys
sys.path.insert(0, {root!r})
import torch, torch.distributed as dist
import bench
world, rank, local = bench.dist_setup(2)
assert world == 2
bench.barrier(world)
m = bench.max_over_ranks(10.0 + rank, world)
assert m == 11.0, m
bench.barrier(world)
dist.destroy_process_group()
print("rank", rank, "ok")
"""


def test_bench_multi_process_plumbing_gloo(tmp_path):
    """world_size 2 on CPU (gloo): rendezvous, barrier and max-over-ranks timing reduction."""
    script = tmp_path / "worker.py"
    script.write_text(_GLOO_WORKER.format(root=ROOT))
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29531", WORLD_SIZE="2", CUDA_VISIBLE_DEVICES="")
    procs = [subprocess.Popen([sys.executable, str(script)], env=dict(env, RANK=str(r), LOCAL_RANK=str(r)),
                              stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True) for r in range(2)]
    for p in procs:
        out, err = p.communicate(timeout=300)
        assert p.returncode == 0, err
        assert "ok" in out
