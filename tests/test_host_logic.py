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
                assert p.workspace_bytes == (4 * p.S * M * N if (p.S > 1 and M > 64) else 0)   # decode folds in-kernel
                assert p.kernel == (0 if K % 8 else (1 if M <= 64 else 2))
    # decode parameters never read M (rule R4)
    ref = B.det_linear_plan_params(1, 1024, 512).as_dict()
    for M in range(1, 65):
        assert B.det_linear_plan_params(M, 1024, 512).as_dict() == ref


def test_attention_cluster_rule(built_lib):
    """The number of thread blocks that share one (batch, KV head) row of the decode attention is host arithmetic:
    one resident wave of two blocks per SM, never more blocks than 256-key segments, 16 only for few very long
    rows, more blocks when the scores of a block would not fit two to an SM."""
    B = built_lib
    sched = B.det_test_attention_schedule
    assert sched(32, 32, 8, 2048, 128)[0] == 1            # 256 rows fill 148 SMs twice over
    assert sched(16, 32, 8, 2048, 128)[0] == 2
    assert sched(8, 32, 8, 4096, 128)[0] == 4
    assert sched(4, 32, 8, 4096, 128)[0] == 8
    assert sched(1, 32, 8, 4096, 128)[0] == 8             # 16 segments, but 16-block clusters only from 64 segments on
    assert sched(1, 32, 8, 65536, 128)[0] == 16
    assert sched(2, 32, 8, 32768, 128)[0] == 8            # 16 rows: clusters of 8
    assert sched(1, 32, 8, 300, 128)[0] == 2              # two segments: at most two blocks
    assert sched(1, 8, 8, 1, 128)[0] == 1
    c, smem = sched(32, 32, 8, 8192, 128)                 # one block per row would need 164 KB: split in two
    assert c == 2 and smem <= 110 * 1024
    c, smem = sched(1, 4, 1, 131072, 128)
    assert c == 16 and smem <= 227 * 1024
    c, smem = sched(1, 4, 1, 200000, 128)                 # does not fit however it is split: the call is refused
    assert c == 16 and smem > 227 * 1024
    assert sched(8, 32, 8, 4096, 128, 74)[0] == 2         # half the SMs: half the blocks
    assert sched(0, 32, 8, 4096, 128)[0] == 0


def test_bad_shapes_are_rejected_with_a_message(built_lib):
    B = built_lib
    for shp in [(0, 1, 1), (1, 0, 1), (1, 1, 0), (-3, 4, 8), (1, 1 << 31, 8), (1 << 21, 1 << 21, 8)]:
        with pytest.raises(B.DetLinearError) as ei:
            B.det_linear_plan_params(*shp)
        assert ei.value.status in (1, 2)
        assert B.det_last_error() != ""
    rc = B.lib().det_linear_plan_params(1, 1, 8, None)
    assert rc == 1
    assert B.det_order_version() == 2


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


def test_bench_headline_is_the_short_last_line(tmp_path):
    """The last line of stdout must be a short, self-contained JSON headline (a reader that keeps only a
    few KB of the tail still gets value, roofline, cpu_baseline and e2e); the long tables go elsewhere."""
    import io
    sys.path.insert(0, ROOT)
    import bench
    line = {"metric": bench.METRIC, "value": 3000.12, "unit": bench.UNIT, "n_gpus": 1, "steps": 20, "warmup": 3,
            "ms_per_step": 0.7, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic", "config": {"workload": "w" * 200, "l2": "x" * 60, "multi_gpu": "replicas only"},
            "pct_of_hbm_peak": 45.0, "tflops_fp32": 34.0,
            "clocks": {"sm_mhz": 1965.0, "sm_max_mhz": 1965.0, "samples": 12, "reasons": [], "window": "y" * 50},
            "e2e": {"value": 2500.0, "unit": bench.UNIT, "h2d_bytes_per_step": 1, "d2h_bytes_per_step": 2},
            "gpu_launches": 400,
            "roofline": {"bound": "hbm", "achieved": 3000.0, "peak": 6543.1, "unit": "GB/s", "frac": 0.45, "traffic": 1,
                         "algorithmic_bytes_per_launch": 1, "frac_of_binding_roof": 0.7, "peak_source": "m", "kernel": "k" * 90},
            "cpu_baseline": {"value": 0.7, "unit": bench.UNIT, "cores": 16, "kind": "oracle", "sample": "s" * 90},
            "decode_pct_of_binding_roof": {f"M{m}": [80.0] * 4 for m in (1, 4, 8, 16, 32)},
            "prefill_pct_fp32_peak": [70.0] * 6, "lm_head_pct_of_binding_roof": [90.0] * 3, "stack_pct_hbm": [80.0, 60.0]}
    tables = {"per_case": [{"name": "n", "us": 1.0}] * 2000}          # far larger than any tail window
    out, err = io.StringIO(), io.StringIO()
    path = tmp_path / "sub" / "tables.json"
    bench.emit(line, tables, str(path), out=out, err=err)
    last = out.getvalue().strip().splitlines()[-1]
    assert len(last) < bench.HEADLINE_MAX_BYTES
    got = json.loads(last)
    for key in ("metric", "value", "unit", "n_gpus", "ms_per_step", "roofline", "cpu_baseline", "e2e", "clocks", "config"):
        assert key in got
    assert "per_case" not in got and len(out.getvalue()) < 2 * bench.HEADLINE_MAX_BYTES
    assert json.loads(path.read_text())["tables"]["per_case"][0]["name"] == "n"
    assert json.loads(err.getvalue())["headline"]["value"] == 3000.12
    # an over-long headline sheds its optional digests instead of growing past the limit
    line["config"]["workload"] = "w" * 700
    out2 = io.StringIO()
    bench.emit(line, {}, None, out=out2, err=io.StringIO())
    got2 = json.loads(out2.getvalue().strip().splitlines()[-1])
    assert len(out2.getvalue()) < bench.HEADLINE_MAX_BYTES + 2 and "roofline" in got2 and "stack_pct_hbm" not in got2


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
