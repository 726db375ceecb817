"""CPU check of tests/golden/digests.json (written by tests/golden/make_digests.py from the oracle alone):
the oracle of today must reproduce the committed digests and order parameters, and the CUDA library's
planner (a host function, no GPU needed) must derive the same parameters.  A change of the order's
constants -- split rules, bucket edge, V/L/P -- on either side, or on both at once, fails here."""
import importlib.util
import json
import os

import pytest

from oracle import oracle
from paper_2609_25624_b200 import inputs

HERE = os.path.dirname(os.path.abspath(__file__))
GOLDEN = os.path.join(HERE, "golden", "digests.json")
_spec = importlib.util.spec_from_file_location("make_digests", os.path.join(HERE, "golden", "make_digests.py"))
make_digests = importlib.util.module_from_spec(_spec)
_spec.loader.exec_module(make_digests)


def load():
    with open(GOLDEN) as f:
        return json.load(f)


def test_file_covers_every_benchmark_case():
    d = load()
    assert d["order_version"] == oracle.ORDER_VERSION
    keys = set(d["cases"])
    want = {"config1:1x1024x512", "lm_head_tie:16", "lm_head_tie:0"}
    want |= {f"decode:{M}x{N}x{K}" for M in inputs.DECODE_MS for (_, K, N) in inputs.LLAMA3_8B_LAYER}
    want |= {f"prefill:{M}x{N}x{K}" for M in inputs.PREFILL_MS for (_, K, N) in inputs.PREFILL_SHAPES}
    want |= {f"lm_head:{M}x128256x4096" for M in inputs.LM_HEAD_MS}
    assert keys == want


def test_order_parameters_match_oracle_and_planner():
    from paper_2609_25624_b200 import binding as B
    d = load()
    for key, entry in d["cases"].items():
        if "params" not in entry:
            continue
        M, N, K = (int(v) for v in key.split(":")[1].split("x"))
        assert oracle.order_params(M, N, K) == entry["params"], key
        assert B.det_linear_plan_params(M, N, K).as_dict() == entry["params"], key


def test_config1_digest():
    d = load()["cases"]["config1:1x1024x512"]
    x, W, b = inputs.make_case(1, 1024, 512, seed=0)
    y = oracle.linear(x.numpy(), inputs.bf16_bits(W), b.numpy())
    assert make_digests.digest(y) == d["sha256"]


@pytest.mark.parametrize("kind,M,name_k_n", [("decode", 1, inputs.LLAMA3_8B_LAYER[1]), ("decode", 8, inputs.LLAMA3_8B_LAYER[1]),
                                             ("decode", 32, inputs.LLAMA3_8B_LAYER[0]), ("prefill", 128, inputs.PREFILL_SHAPES[1])])
def test_sampled_digests_of_some_cases(kind, M, name_k_n):
    """A few of the smaller cases are recomputed here (the whole file takes about a minute to rebuild)."""
    _, K, N = name_k_n
    d = load()["cases"][f"{kind}:{M}x{N}x{K}"]
    got = make_digests.linear_case(kind, M, N, K)
    assert got == d


def test_digest_is_sensitive_to_the_split():
    """The same sampled outputs under another split factor hash differently: the file does pin S."""
    M, (_, K, N) = 8, inputs.LLAMA3_8B_LAYER[1]
    d = load()["cases"][f"decode:{M}x{N}x{K}"]
    x, W, b = inputs.make_case(M, N, K)
    ms, ns = make_digests.sample_points(M, N, inputs.shape_seed(M, N, K))
    prm = dict(d["params"])
    assert prm["S"] == 2
    other = dict(prm, seg_len=K, S=1)
    vals = oracle.linear_sampled(x.numpy(), inputs.bf16_bits(W), b.numpy(), ms, ns, params=other)
    assert make_digests.digest(vals) != d["sha256"]
    vals = oracle.linear_sampled(x.numpy(), inputs.bf16_bits(W), b.numpy(), ms, ns, params=prm)
    assert make_digests.digest(vals) == d["sha256"]
