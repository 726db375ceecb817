"""Pins for the CPU oracle: the hand-traced order examples, the layout example, up(), the fused
single rounding, and agreement between the C oracle and the exact-rational micro-oracle."""
import random
import struct

import numpy as np
import pytest

from oracle import exact, oracle
from tests import golden_util as gu

EXAMPLES = gu.load_order_examples()


def _ids(e):
    return f"{e['name']}-V{e['V']}L{e['L']}P{e['P']}S{e['s_req']}"


@pytest.mark.parametrize("e", EXAMPLES, ids=_ids)
def test_hand_traced_examples_exact_micro_oracle(e):
    seg = gu.seg_len_for(len(e["x"]), e["s_req"], e["granule"])
    got = exact.output(e["x"], e["w"], e["b"], e["V"], e["L"], e["P"], seg)
    assert got == e["expected"]


@pytest.mark.parametrize("e", EXAMPLES, ids=_ids)
def test_hand_traced_examples_c_oracle(e):
    K = len(e["x"])
    seg = gu.seg_len_for(K, e["s_req"], e["granule"])
    x = np.array([e["x"]], dtype=np.float32)
    W = np.array([e["w"]], dtype=np.uint16)
    b = None if e["b"] is None else np.array([e["b"]], dtype=np.float32)
    y = oracle.linear(x, W, b, params=dict(V=e["V"], L=e["L"], P=e["P"], seg_len=seg))
    assert y.shape == (1, 1)
    assert float(y[0, 0]) == e["expected"]


def test_examples_cover_production_constants():
    """The fixture must exercise the constants the planner really uses."""
    dec = oracle.order_params(1, 4096, 4096)
    pre = oracle.order_params(128, 4096, 4096)
    seen = {(e["V"], e["L"], e["P"]) for e in EXAMPLES}
    assert (dec["V"], dec["L"], dec["P"]) in seen
    assert (pre["V"], pre["L"], pre["P"]) in seen


def test_layout_example_every_order():
    expected = np.array(gu.load_layout_example(), dtype=np.float32)
    M = N = 4
    K = 8
    x = np.array([[(m + 1) * (k + 1) for k in range(K)] for m in range(M)], dtype=np.float32)
    Wf = np.array([[n - k for k in range(K)] for n in range(N)], dtype=np.float32)
    W = (Wf.view(np.uint32) >> 16).astype(np.uint16)       # small integers are BF16-exact
    assert np.array_equal((W.astype(np.uint32) << 16).view(np.float32), Wf)
    b = np.array([n / 2 for n in range(N)], dtype=np.float32)
    for (V, L, P, seg) in [(1, 1, 1, 8), (1, 1, 1, 4), (2, 1, 2, 256), (4, 32, 2, 256), (2, 2, 2, 4),
                           (1, 4, 1, 4), (8, 32, 1, 256)]:
        y = oracle.linear(x, W, b, params=dict(V=V, L=L, P=P, seg_len=seg))
        assert np.array_equal(y, expected), (V, L, P, seg)
        ye = np.array(exact.linear(x.tolist(), W.tolist(), b.tolist(), V, L, P, seg), dtype=np.float32)
        assert np.array_equal(ye, expected)
    # production parameters chosen from the shape
    assert np.array_equal(oracle.linear(x, W, b), expected)
    # a transposed read of the weight buffer gives a different, known first row
    yT = oracle.linear(x, np.ascontiguousarray(W.reshape(-1).reshape(K, N).T), b)
    assert list(yT[0]) == [-6.0, -41.5, -77.0, -112.5]


def test_up_all_bit_patterns():
    """up(h) is the binary32 with bit pattern h << 16 (Eq. 2's register upcast): all 65 536 patterns
    against numpy bit operations and against torch's own bfloat16 -> float32 conversion."""
    import torch
    hs = np.arange(65536, dtype=np.uint32)
    want = (hs << 16).astype(np.uint32)
    got = np.array([struct.unpack("<I", struct.pack("<f", oracle.up(int(h))))[0]
                    if not np.isnan(oracle.up(int(h))) else None for h in hs], dtype=object)
    for h in range(65536):
        if got[h] is None:                     # NaN payloads may be quieted when returned by value
            assert np.isnan(np.uint32(want[h]).view(np.float32))
        else:
            assert got[h] == want[h], hex(h)
    t = torch.from_numpy(hs.astype(np.int16)).view(torch.bfloat16).to(torch.float32)
    tb = t.view(torch.int32).numpy().astype(np.uint32)
    finite = ~np.isnan(want.view(np.float32))
    assert np.array_equal(tb[finite], want[finite])
    for h in (0x0000, 0x8000, 0x3F80, 0x0001, 0x7F7F, 0xFF80):
        assert exact.bf16_bits_to_float(h) == oracle.up(h) or h == 0x8000
    assert np.signbit(oracle.up(0x8000)) and oracle.up(0x8000) == 0.0


def test_s_moves_the_bits():
    """Different split factors give different outputs on random data (supplement C on R3: an S sweep
    gives distinct outputs), so an oracle that ignored its segment length would be caught."""
    rng = np.random.default_rng(7)
    K = 2048
    x = rng.standard_normal((2, K)).astype(np.float32)
    W = (rng.standard_normal((64, K)).astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
    outs = []
    for seg in (2048, 1024, 512, 256):
        outs.append(oracle.linear(x, W, None, params=dict(V=4, L=32, P=1, seg_len=seg)).tobytes())
    assert len(set(outs)) == 4
    outs = []
    for prm in [(1, 1, 1), (2, 1, 2), (4, 32, 2), (8, 32, 1), (4, 32, 1)]:
        V, L, P = prm
        outs.append(oracle.linear(x, W, None, params=dict(V=V, L=L, P=P, seg_len=2048)).tobytes())
    assert len(set(outs)) == 5


def _rand_f32(rng):
    kind = rng.random()
    if kind < 0.1:
        return 0.0
    if kind < 0.2:                                      # subnormal or tiny
        return struct.unpack("<f", struct.pack("<I", rng.randrange(1, 1 << 23) | (rng.randrange(2) << 31)))[0]
    if kind < 0.3:
        return float(rng.choice([2.0 ** 24, -2.0 ** 24, 1.0, -1.0, 3.0]))
    v = np.float32(rng.gauss(0, 1) * 10 ** rng.randrange(-3, 4))
    return float(v)


def test_c_oracle_equals_exact_micro_oracle_on_tiny_random_cases():
    """Brute force on tiny inputs: the C oracle (libm fmaf) against exact rational arithmetic, over
    random order parameters, ragged K, subnormals, signed zeros and cancellations."""
    rng = random.Random(1234)
    for case in range(60):
        V = rng.choice([1, 2, 4, 8])
        L = rng.choice([1, 2, 4, 32])
        P = rng.choice([p for p in (1, 2, 4) if V % p == 0])
        C = V * L
        K = rng.choice([1, 2, 3, 7, 8, 9, 31, 64, 100, 257])
        gran = C if case % 2 else max(C, 8)
        gran = -(-gran // C) * C
        s_req = rng.choice([1, 2, 3, 4])
        seg = gu.seg_len_for(K, s_req, gran)
        M, N = rng.choice([1, 2]), rng.choice([1, 3])
        x = [[_rand_f32(rng) for _ in range(K)] for _ in range(M)]
        W = [[rng.choice([0x3F80, 0xBF80, 0x0000, 0x8000, 0x0001, 0x8001, rng.randrange(0x3000, 0x4800),
                          0x8000 | rng.randrange(0x3000, 0x4800)]) for _ in range(K)] for _ in range(N)]
        b = None if case % 3 == 0 else [_rand_f32(rng) for _ in range(N)]
        want = exact.linear(x, W, b, V, L, P, seg)
        got = oracle.linear(np.array(x, dtype=np.float32), np.array(W, dtype=np.uint16),
                            None if b is None else np.array(b, dtype=np.float32),
                            params=dict(V=V, L=L, P=P, seg_len=seg))
        want = np.array(want, dtype=np.float32)
        assert np.array_equal(got.view(np.uint32), want.view(np.uint32)), (case, V, L, P, K, seg)


def test_tail_elements_are_skipped_not_zero_filled():
    """A lane whose accumulator is -0.0 keeps it when later elements lie beyond K; a zero-filled
    fmaf(0, 0, -0.0) would turn it into +0.0."""
    tiny = struct.unpack("<f", struct.pack("<I", 0x80000001))[0]      # -min subnormal
    x = np.array([[tiny, 0, 0]], dtype=np.float32)                      # K = 3, ragged
    W = np.array([[0x0001, 0, 0]], dtype=np.uint16)                     # +min BF16 subnormal
    y = oracle.linear(x, W, None, params=dict(V=1, L=1, P=1, seg_len=256))
    # product underflows to -0.0; the two real zeros keep it (-0 + +0*+0 = +0 actually adds +0):
    ye = exact.linear(x.tolist(), W.tolist(), None, 1, 1, 1, 256)
    assert np.array_equal(y.view(np.uint32), np.array(ye, dtype=np.float32).view(np.uint32))
    x1 = np.array([[tiny]], dtype=np.float32)
    W1 = np.array([[0x0001]], dtype=np.uint16)
    y1 = oracle.linear(x1, W1, None, params=dict(V=4, L=1, P=1, seg_len=256))   # 3 skipped elements
    assert y1.view(np.uint32)[0, 0] == 0x80000000


def test_up_fp16_all_bit_patterns():
    """Binary16 -> binary32 widening of the oracle: all 65 536 patterns against numpy's own
    float16 -> float32 conversion (NaNs compared as NaNs)."""
    hs = np.arange(65536, dtype=np.uint16)
    want = hs.view(np.float16).astype(np.float32)
    got = np.array([oracle.up_fp16(int(h)) for h in hs], dtype=np.float32)
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan].view(np.uint32), want[~nan].view(np.uint32))
    for h in (0x0001, 0x03FF, 0x0400, 0x7BFF, 0x8001, 0xFBFF, 0x3C00):
        assert exact.fp16_bits_to_float(h) == oracle.up_fp16(h)


@pytest.mark.parametrize("wfmt", ["fp16", "fp32"])
def test_other_weight_formats_follow_the_same_order(wfmt):
    """FP16 and FP32 weights go through the same reduction order: hand-traced examples with all
    weights = 1 give the same values, the C oracle equals the exact micro-oracle on random tiny
    cases, and values exactly representable in BF16 give bit-identical results in every format."""
    one = {"fp16": 0x3C00, "fp32": 1.0}[wfmt]
    for e in EXAMPLES:
        if any(w != gu.ONE_BF16 for w in e["w"]):
            continue
        K = len(e["x"])
        seg = gu.seg_len_for(K, e["s_req"], e["granule"])
        x = np.array([e["x"]], dtype=np.float32)
        W = np.full((1, K), one, dtype=np.float32 if wfmt == "fp32" else np.uint16)
        b = None if e["b"] is None else np.array([e["b"]], dtype=np.float32)
        y = oracle.linear(x, W, b, params=dict(V=e["V"], L=e["L"], P=e["P"], seg_len=seg), wfmt=wfmt)
        assert float(y[0, 0]) == e["expected"], e["name"]
    rng = random.Random(77)
    for case in range(25):
        V, L, P = rng.choice([(1, 1, 1), (4, 32, 1), (2, 2, 2), (8, 32, 1)])
        K = rng.choice([3, 8, 31, 100, 257])
        seg = gu.seg_len_for(K, rng.choice([1, 2, 3]), max(V * L, 8) // (V * L) * (V * L) if V * L <= 8 else V * L)
        x = [[_rand_f32(rng) for _ in range(K)] for _ in range(2)]
        if wfmt == "fp16":
            W = [[rng.choice([0x3C00, 0xBC00, 0x0000, 0x8000, 0x0001, 0x83FF, rng.randrange(0x2000, 0x5000),
                              0x8000 | rng.randrange(0x2000, 0x5000)]) for _ in range(K)] for _ in range(3)]
            Wa = np.array(W, dtype=np.uint16)
        else:
            W = [[_rand_f32(rng) for _ in range(K)] for _ in range(3)]
            Wa = np.array(W, dtype=np.float32)
        want = np.array(exact.linear(x, W, None, V, L, P, seg, wfmt), dtype=np.float32)
        got = oracle.linear(np.array(x, dtype=np.float32), Wa, None, params=dict(V=V, L=L, P=P, seg_len=seg), wfmt=wfmt)
        assert np.array_equal(got.view(np.uint32), want.view(np.uint32)), (case, V, L, P, K)
    # BF16-exact values: identical bits whatever the storage format
    g = np.random.default_rng(5)
    Wb = (g.standard_normal((7, 640)).astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
    Wf = (Wb.astype(np.uint32) << 16).view(np.float32)
    x = g.standard_normal((3, 640)).astype(np.float32)
    ref = oracle.linear(x, Wb, None)
    assert np.array_equal(oracle.linear(x, Wf, None, wfmt="fp32").view(np.uint32), ref.view(np.uint32))
