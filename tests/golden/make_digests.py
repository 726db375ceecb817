#!/usr/bin/env python
"""Write tests/golden/digests.json: golden digests of the frozen reduction order on the benchmark's
configurations, computed by the CPU oracle ALONE (this script imports the oracle and the seeded input
generators, never the CUDA package).

    python tests/golden/make_digests.py

What is stored, per case: the order parameters the oracle derives from the shape (bucket, V, L, P,
seg_len, S, order version) and the SHA-256 of the float32 bytes of the outputs at a fixed, seeded sample
of (row, column) positions (config 1: the whole output).  For the LM head also the greedy argmax of
every batch row at M = 1, and for the near-tie and exact-tie variants the argmax of batch row 0.

The file pins the CONSTANTS of the order (split rules, bucket edge, V/L/P), which the paper does not
print: a change made to the rule on the oracle's side and on the planner's side at once still
changes these digests, and tests/test_golden_digests.py (CPU) and tests/test_gpu_digests.py (GPU)
then fail.
"""
import hashlib
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from oracle import oracle  # noqa: E402
from paper_2609_25624_b200 import inputs  # noqa: E402  (seeded generators only: no arithmetic of the method)

OUT = os.path.join(os.path.dirname(os.path.abspath(__file__)), "digests.json")
N_SAMPLES = 256


def sample_points(M, N, seed):
    """The fixed sample of output positions of a case: seeded, plus the four corners."""
    rng = np.random.default_rng(seed)
    ms = np.concatenate([rng.integers(0, M, size=N_SAMPLES), [0, 0, M - 1, M - 1]]).astype(np.int64)
    ns = np.concatenate([rng.integers(0, N, size=N_SAMPLES), [0, N - 1, 0, N - 1]]).astype(np.int64)
    return ms, ns


def digest(values):
    return hashlib.sha256(np.ascontiguousarray(values, dtype=np.float32).tobytes()).hexdigest()


def case_key(kind, M, N, K):
    return f"{kind}:{M}x{N}x{K}"


def linear_case(kind, M, N, K, seed=None):
    x, W, b = inputs.make_case(M, N, K, seed=seed)
    ms, ns = sample_points(M, N, inputs.shape_seed(M, N, K))
    vals = oracle.linear_sampled(x.numpy(), inputs.bf16_bits(W), b.numpy(), ms, ns)
    return {"params": oracle.order_params(M, N, K), "samples": int(len(ms)), "sha256": digest(vals)}


def lm_head_inputs(M):
    name, K, N = inputs.LLAMA3_8B_LM_HEAD
    W = inputs.make_weight(N, K, inputs.named_seed("lm_head"))
    import torch
    g = torch.Generator().manual_seed(inputs.shape_seed(M, N, K))
    x = torch.randn(M, K, generator=g)
    return x, W


def near_tie_weights(W, x_row0, n_positions):
    """The LM-head variant of the benchmark: the oracle's argmax row of batch row 0 copied over a seeded
    other row, then moved by one BF16 ulp in `n_positions` seeded positions (0 = exact tie)."""
    base = oracle.linear(x_row0, inputs.bf16_bits(W), None)
    r1 = int(oracle.argmax_rows(base)[0])
    r2 = int(np.random.default_rng(3).integers(0, W.shape[0]))
    if r2 == r1:
        r2 = (r1 + 1) % W.shape[0]
    return inputs.make_near_tie(W, r1, r2, n_positions=n_positions, seed=11), r1, r2


def build():
    out = {"order_version": oracle.ORDER_VERSION, "n_samples": N_SAMPLES, "cases": {}}
    cases = out["cases"]
    # config 1: the whole output
    x, W, b = inputs.make_case(1, 1024, 512, seed=0)
    y = oracle.linear(x.numpy(), inputs.bf16_bits(W), b.numpy())
    cases["config1:1x1024x512"] = {"params": oracle.order_params(1, 1024, 512), "samples": int(y.size), "sha256": digest(y)}
    # config 2: decode sweep
    for M in inputs.DECODE_MS:
        for (name, K, N) in inputs.LLAMA3_8B_LAYER:
            cases[case_key("decode", M, N, K)] = linear_case("decode", M, N, K)
            print("decode", M, name, flush=True)
    # config 4: prefill
    for M in inputs.PREFILL_MS:
        for (name, K, N) in inputs.PREFILL_SHAPES:
            cases[case_key("prefill", M, N, K)] = linear_case("prefill", M, N, K)
            print("prefill", M, name, flush=True)
    # config 3: LM head (no bias), sampled logits for every batch size, argmax at M = 1, tie variants
    name, K, N = inputs.LLAMA3_8B_LM_HEAD
    for M in inputs.LM_HEAD_MS:
        x, W = lm_head_inputs(M)
        ms, ns = sample_points(M, N, inputs.shape_seed(M, N, K))
        vals = oracle.linear_sampled(x.numpy(), inputs.bf16_bits(W), None, ms, ns)
        entry = {"params": oracle.order_params(M, N, K), "samples": int(len(ms)), "sha256": digest(vals)}
        if M == 1:
            entry["argmax"] = [int(v) for v in oracle.argmax_rows(oracle.linear(x.numpy(), inputs.bf16_bits(W), None))]
        cases[case_key("lm_head", M, N, K)] = entry
        print("lm_head", M, flush=True)
    x, W = lm_head_inputs(8)
    for n_positions in (16, 0):
        W2, r1, r2 = near_tie_weights(W, x[:1].numpy(), n_positions)
        row0 = oracle.linear(x[:1].numpy(), inputs.bf16_bits(W2), None)
        cases[f"lm_head_tie:{n_positions}"] = {"rows": [r1, r2], "argmax_row0": int(oracle.argmax_rows(row0)[0]),
                                              "logits_r1_r2_bits": [int(np.float32(row0[0, r]).view(np.uint32)) for r in (r1, r2)]}
        print("lm_head tie", n_positions, flush=True)
    return out


if __name__ == "__main__":
    data = build()
    with open(OUT, "w") as f:
        json.dump(data, f, indent=1, sort_keys=True)
        f.write("\n")
    print("wrote", OUT, len(data["cases"]), "cases")
