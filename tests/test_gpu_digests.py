"""GPU side of tests/golden/digests.json: every benchmark case at full size, through the C ABI in the launch
configuration bench.py times, hashed at the file's sample positions and compared with the committed,
oracle-written digest (no oracle call here: the expected values are the file's)."""
import importlib.util
import json
import os

import numpy as np
import pytest
import torch

from paper_2609_25624_b200 import binding as B
from paper_2609_25624_b200 import inputs
from tests.gpu_util import run_gpu

pytestmark = pytest.mark.gpu

HERE = os.path.dirname(os.path.abspath(__file__))
_spec = importlib.util.spec_from_file_location("make_digests", os.path.join(HERE, "golden", "make_digests.py"))
make_digests = importlib.util.module_from_spec(_spec)
_spec.loader.exec_module(make_digests)

with open(os.path.join(HERE, "golden", "digests.json")) as _f:
    GOLDEN = json.load(_f)

LINEAR_KEYS = sorted(k for k in GOLDEN["cases"] if k.split(":")[0] in ("config1", "decode", "prefill"))


def test_order_version():
    assert GOLDEN["order_version"] == B.det_order_version()


@pytest.mark.parametrize("key", LINEAR_KEYS)
def test_linear_case_matches_the_golden_digest(key):
    kind, dims = key.split(":")
    M, N, K = (int(v) for v in dims.split("x"))
    entry = GOLDEN["cases"][key]
    x, W, b = inputs.make_case(M, N, K, seed=0 if kind == "config1" else None)
    plan = B.det_linear_plan(M, N, K)
    assert B.det_linear_plan_get_params(plan).as_dict() == entry["params"]
    plan.close()
    got = run_gpu(x, W, b)
    if kind == "config1":
        assert make_digests.digest(got) == entry["sha256"]
    else:
        ms, ns = make_digests.sample_points(M, N, inputs.shape_seed(M, N, K))
        assert len(ms) == entry["samples"]
        assert make_digests.digest(got[ms, ns]) == entry["sha256"]


def _logits_and_argmax(x, W):
    M, K = x.shape
    N = W.shape[0]
    y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    idx = torch.full((M,), -1, dtype=torch.int32, device="cuda")
    plan = B.det_linear_plan(M, N, K)
    B.det_linear_run(plan, x.cuda(), W.cuda(), None, y)
    B.det_argmax_rows(y, idx)
    B.det_linear_plan_check(plan)
    plan.close()
    return y.cpu().numpy(), idx.cpu().numpy()


@pytest.mark.parametrize("M", inputs.LM_HEAD_MS)
def test_lm_head_matches_the_golden_digest(M):
    name, K, N = inputs.LLAMA3_8B_LM_HEAD
    entry = GOLDEN["cases"][f"lm_head:{M}x{N}x{K}"]
    x, W = make_digests.lm_head_inputs(M)
    got, idx = _logits_and_argmax(x, W)
    ms, ns = make_digests.sample_points(M, N, inputs.shape_seed(M, N, K))
    assert make_digests.digest(got[ms, ns]) == entry["sha256"]
    if "argmax" in entry:
        assert idx.tolist() == entry["argmax"]


@pytest.mark.parametrize("n_positions", [16, 0])
def test_lm_head_tie_variants_match_the_golden_argmax(n_positions):
    """The near-tie / exact-tie weight matrices are rebuilt from the golden file's row numbers (no oracle):
    row r1 copied over row r2, then moved by one BF16 ulp in 16 seeded positions (or none)."""
    entry = GOLDEN["cases"][f"lm_head_tie:{n_positions}"]
    r1, r2 = entry["rows"]
    x, W = make_digests.lm_head_inputs(8)
    W2 = inputs.make_near_tie(W, r1, r2, n_positions=n_positions, seed=11)
    got, idx = _logits_and_argmax(x, W2)
    assert int(idx[0]) == entry["argmax_row0"]
    bits = [int(np.float32(got[0, r]).view(np.uint32)) for r in (r1, r2)]
    assert bits == entry["logits_r1_r2_bits"]
    if n_positions == 0:
        assert bits[0] == bits[1] and int(idx[0]) == min(r1, r2)
