"""Python face of the CPU oracle (ctypes over liboracle.so) and the oracle's own copy of the
shape -> order-parameter rule.

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the benchmark's CPU-baseline
leg; never by the product path, and it imports nothing from the CUDA package.

The rule below restates, independently of the CUDA library's planner, how the reduction order is
chosen from the problem shape alone (design rule R2: configuration is a pure function of (M, N, K);
R3: the split is shape-pure; R4: inside the decode bucket nothing depends on M).  The tests assert
that both sides arrive at the same parameters.
"""
import ctypes
import os

import numpy as np

from . import build_oracle

ORDER_VERSION = 2

#: segment boundaries fall on multiples of this many k elements in both buckets
SEGMENT_GRANULE = 256
#: decode bucket edge (R2/R4: batches of up to 64 rows are decode-shaped)
DECODE_MAX_M = 64
#: decode bucket: weight matrices with at least this many rows are not split (they fill the machine)
DECODE_NO_SPLIT_ROWS = 16384


def _ceil_div(a: int, b: int) -> int:
    return -(-a // b)


def _segments_for(K: int, s_req: int):
    """Segment layout for a requested split: boundaries on multiples of the granule, every segment
    non-empty.  Returns (seg_len, S)."""
    n_gran = _ceil_div(K, SEGMENT_GRANULE)
    gran_per_seg = _ceil_div(n_gran, min(s_req, n_gran))
    return SEGMENT_GRANULE * gran_per_seg, _ceil_div(n_gran, gran_per_seg)


def split_request(M: int, N: int, K: int) -> int:
    """Requested number of K segments before clamping to what K allows.

    Decode (never reads M, rule R4): 1 when N >= 16384 (enough weight rows to keep every SM busy on its
    own; the paper's lm_head likewise takes no split), otherwise 2.
    Prefill: the request in 1..16 that minimises rounds * (seg_len + overhead) * occupancy_factor,
    with tiles = number of 128x128 output tiles, units = tiles * S, rounds = ceil(units / 148),
    overhead = 8 k-steps per work unit plus 32 when partials are written and combined,
    occupancy_factor = 9 if units <= 148 else 8; ties go to the larger request.  The constants are
    frozen parts of the order definition (tuned once on a 148-SM part, never read from the device)."""
    if M <= DECODE_MAX_M:
        return 1 if N >= DECODE_NO_SPLIT_ROWS else 2
    tiles = _ceil_div(M, 128) * _ceil_div(N, 128)
    best, best_cost = 1, None
    for s_req in range(1, 17):
        seg_len, S = _segments_for(K, s_req)
        units = tiles * S
        rounds = _ceil_div(units, 148)
        cost = rounds * (seg_len + (40 if S > 1 else 8)) * (9 if units <= 148 else 8)
        if best_cost is None or cost <= best_cost:
            best, best_cost = s_req, cost
    return best


def order_params(M: int, N: int, K: int) -> dict:
    """Order parameters for a problem shape: bucket, (V, L, P), seg_len and the segment count S."""
    if min(M, N, K) < 1:
        raise ValueError("M, N, K must be >= 1")
    if M <= DECODE_MAX_M:
        bucket, V, L, P = "decode", 4, 32, 1
    else:
        bucket, V, L, P = "prefill", 1, 1, 1
    seg_len, S = _segments_for(K, split_request(M, N, K))
    return {"bucket": bucket, "V": V, "L": L, "P": P, "seg_len": seg_len, "S": S,
            "order_version": ORDER_VERSION}


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        path = build_oracle.build()
        L = ctypes.CDLL(path)
        i64, i32, p = ctypes.c_int64, ctypes.c_int, ctypes.c_void_p
        L.det_oracle_linear.argtypes = [p, p, p, p, i64, i64, i64, i32, i32, i32, i64, i32]
        L.det_oracle_linear.restype = i32
        L.det_oracle_linear_sampled.argtypes = [p, p, p, p, p, i64, p, i64, i64, i64,
                                                i32, i32, i32, i64, i32]
        L.det_oracle_linear_sampled.restype = i32
        L.det_oracle_linear_w.argtypes = [p, p, i32, p, p, i64, i64, i64, i32, i32, i32, i64, i32]
        L.det_oracle_linear_w.restype = i32
        L.det_oracle_linear_sampled_w.argtypes = [p, p, i32, p, p, p, i64, p, i64, i64, i64,
                                                  i32, i32, i32, i64, i32]
        L.det_oracle_linear_sampled_w.restype = i32
        L.det_oracle_up_fp16.argtypes = [ctypes.c_uint16]
        L.det_oracle_up_fp16.restype = ctypes.c_float
        L.det_oracle_argmax_rows.argtypes = [p, i64, i64, p]
        L.det_oracle_argmax_rows.restype = i32
        L.det_oracle_up.argtypes = [ctypes.c_uint16]
        L.det_oracle_up.restype = ctypes.c_float
        L.det_oracle_threads.restype = i32
        L.det_oracle_sum_squares.argtypes = [p, i64]
        L.det_oracle_sum_squares.restype = ctypes.c_float
        L.det_oracle_rmsnorm.argtypes = [p, p, ctypes.c_float, i64, i64, p]
        L.det_oracle_rmsnorm.restype = i32
        L.det_oracle_exp.argtypes = [ctypes.c_float]
        L.det_oracle_exp.restype = ctypes.c_float
        L.det_oracle_attention_decode.argtypes = [p, p, p, ctypes.c_float, i64, i64, i64, i64, i64, p, p]
        L.det_oracle_attention_decode.restype = i32
        L.det_oracle_lane_dot.argtypes = [p, p, i64]
        L.det_oracle_lane_dot.restype = ctypes.c_float
        L.det_oracle_lane_sum.argtypes = [p, i64]
        L.det_oracle_lane_sum.restype = ctypes.c_float
        _lib = L
    return _lib


def _f32(a, shape):
    a = np.ascontiguousarray(a, dtype=np.float32)
    assert a.shape == shape, (a.shape, shape)
    return a


#: weight formats: 16-bit formats are passed as bit patterns (uint16), FP32 weights as float32
WEIGHT_FORMATS = {"bf16": 0, "fp16": 1, "fp32": 2}


def _weights(W, shape, wfmt):
    W = np.ascontiguousarray(W)
    if wfmt == "fp32":
        assert W.dtype == np.float32, "FP32 weights must be a float32 array"
    else:
        assert W.dtype == np.uint16, "16-bit weights must be given as bit patterns (uint16)"
    assert W.shape == shape, (W.shape, shape)
    return W


def _resolve(M, N, K, params):
    prm = order_params(M, N, K) if params is None else params
    return int(prm["V"]), int(prm["L"]), int(prm["P"]), int(prm["seg_len"])


def linear(x, W_bits, b=None, params=None, threads=0, wfmt="bf16"):
    """y = x . up(W)^T (+ b) in the frozen order.  x [M,K] float32, W_bits [N,K] uint16 (BF16 or FP16
    bit patterns) or float32 (wfmt="fp32"), b [N] float32 or None.  `params` overrides the
    shape-derived order (for the scaled-down hand examples)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    M, K = x.shape
    N = W_bits.shape[0]
    W_bits = _weights(W_bits, (N, K), wfmt)
    V, L, P, seg_len = _resolve(M, N, K, params)
    y = np.empty((M, N), dtype=np.float32)
    bp = None
    if b is not None:
        b = _f32(b, (N,))
        bp = b.ctypes.data
    rc = lib().det_oracle_linear_w(x.ctypes.data, W_bits.ctypes.data, WEIGHT_FORMATS[wfmt], bp, y.ctypes.data,
                                   M, N, K, V, L, P, seg_len, threads)
    if rc != 0:
        raise ValueError("det_oracle_linear_w rejected its arguments")
    return y


def linear_sampled(x, W_bits, b, ms, ns, params=None, threads=0, wfmt="bf16"):
    """Selected outputs y[ms[i], ns[i]] of the same computation."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    M, K = x.shape
    N = W_bits.shape[0]
    W_bits = _weights(W_bits, (N, K), wfmt)
    V, L, P, seg_len = _resolve(M, N, K, params)
    ms = np.ascontiguousarray(ms, dtype=np.int64)
    ns = np.ascontiguousarray(ns, dtype=np.int64)
    out = np.empty(ms.shape[0], dtype=np.float32)
    bp = None
    if b is not None:
        b = _f32(b, (N,))
        bp = b.ctypes.data
    rc = lib().det_oracle_linear_sampled_w(x.ctypes.data, W_bits.ctypes.data, WEIGHT_FORMATS[wfmt], bp,
                                           ms.ctypes.data, ns.ctypes.data, ms.shape[0], out.ctypes.data,
                                           M, N, K, V, L, P, seg_len, threads)
    if rc != 0:
        raise ValueError("det_oracle_linear_sampled_w rejected its arguments")
    return out


def argmax_rows(y):
    """Index of the row maximum, lowest index on ties."""
    y = np.ascontiguousarray(y, dtype=np.float32)
    M, N = y.shape
    idx = np.empty(M, dtype=np.int32)
    rc = lib().det_oracle_argmax_rows(y.ctypes.data, M, N, idx.ctypes.data)
    if rc != 0:
        raise ValueError("det_oracle_argmax_rows rejected its arguments")
    return idx


def sum_squares(x) -> float:
    """Fixed-order sum of squares of one row (the reduction inside rmsnorm)."""
    x = np.ascontiguousarray(x, dtype=np.float32).reshape(-1)
    return float(lib().det_oracle_sum_squares(x.ctypes.data, x.size))


def rmsnorm(x, g, eps: float):
    """Fixed-order RMSNorm per row: y = (x * r) * g, r = 1 / sqrt(sum_squares(x) / H + eps), every
    step one binary32 operation.  x [M,H] float32, g [H] float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    M, H = x.shape
    g = _f32(g, (H,))
    y = np.empty((M, H), dtype=np.float32)
    rc = lib().det_oracle_rmsnorm(x.ctypes.data, g.ctypes.data, float(np.float32(eps)), M, H, y.ctypes.data)
    if rc != 0:
        raise ValueError("det_oracle_rmsnorm rejected its arguments")
    return y


def exp_det(x: float) -> float:
    """The fixed-sequence exponential of the attention (defined for x <= 0)."""
    return float(lib().det_oracle_exp(float(np.float32(x))))


def lane_dot(a, b) -> float:
    """Dot product in the decode lane order (the attention's q . k_j before the scale)."""
    a = np.ascontiguousarray(a, dtype=np.float32).reshape(-1)
    b = np.ascontiguousarray(b, dtype=np.float32).reshape(-1)
    assert a.size == b.size
    return float(lib().det_oracle_lane_dot(a.ctypes.data, b.ctypes.data, a.size))


def lane_sum(e) -> float:
    """Sum in the lane order over the keys (the attention's softmax denominator)."""
    e = np.ascontiguousarray(e, dtype=np.float32).reshape(-1)
    return float(lib().det_oracle_lane_sum(e.ctypes.data, e.size))


def attention_decode(q, k, v, scale: float):
    """Fixed-order decode attention: q [B,Hq,D], k and v [B,Hkv,T,D] float32 -> o [B,Hq,D]; one query row
    per (batch, head) against T cached keys and values, grouped-query heads when Hq > Hkv."""
    q = np.ascontiguousarray(q, dtype=np.float32)
    k = np.ascontiguousarray(k, dtype=np.float32)
    v = np.ascontiguousarray(v, dtype=np.float32)
    B, Hq, D = q.shape
    Bk, Hkv, T, Dk = k.shape
    assert (Bk, Dk) == (B, D) and v.shape == k.shape and Hq % Hkv == 0
    o = np.empty((B, Hq, D), dtype=np.float32)
    scratch = np.empty(T * max(1, int(lib().det_oracle_threads())), dtype=np.float32)
    rc = lib().det_oracle_attention_decode(q.ctypes.data, k.ctypes.data, v.ctypes.data, float(np.float32(scale)),
                                           B, Hq, Hkv, T, D, o.ctypes.data, scratch.ctypes.data)
    if rc != 0:
        raise ValueError("det_oracle_attention_decode rejected its arguments")
    return o


def up(h: int) -> float:
    return float(lib().det_oracle_up(int(h) & 0xFFFF))


def up_fp16(h: int) -> float:
    return float(lib().det_oracle_up_fp16(int(h) & 0xFFFF))


def threads() -> int:
    """Threads the oracle uses by default (bounded by the process's CPU affinity)."""
    return min(int(lib().det_oracle_threads()), len(os.sched_getaffinity(0)))
