"""Thin Python binding of libdet_linear.so (ctypes): argument marshalling only.

Every function has the name of the C entry point it calls (include/det_linear.h) minus nothing:
`det_linear_plan`, `det_linear_run`, ...  Tensors are torch CUDA tensors; only their data pointers,
shapes and the current stream cross the boundary.  There is no CPU fallback: if the shared library
is missing or cannot be loaded, importing symbols from here raises.
"""
import ctypes
import json
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdet_linear.so")

DET_OK = 0
STATUS_NAMES = {0: "DET_OK", 1: "DET_ERR_INVALID_ARG", 2: "DET_ERR_UNSUPPORTED_SHAPE", 3: "DET_ERR_ALIGNMENT",
                4: "DET_ERR_ALLOC", 5: "DET_ERR_CUDA", 6: "DET_ERR_DEVICE_TIMEOUT", 7: "DET_ERR_ARCH"}


class DetLinearError(RuntimeError):
    def __init__(self, status, message):
        super().__init__(f"{STATUS_NAMES.get(status, status)}: {message}")
        self.status = status


class Params(ctypes.Structure):
    """Mirror of det_linear_params_t."""
    _fields_ = [("M", ctypes.c_int64), ("N", ctypes.c_int64), ("K", ctypes.c_int64),
                ("bucket", ctypes.c_int32), ("V", ctypes.c_int32), ("L", ctypes.c_int32), ("P", ctypes.c_int32),
                ("seg_len", ctypes.c_int64), ("S", ctypes.c_int32), ("order_version", ctypes.c_int32),
                ("kernel", ctypes.c_int32), ("weight_format", ctypes.c_int32), ("workspace_bytes", ctypes.c_uint64)]

    def as_dict(self):
        return {"bucket": "decode" if self.bucket == 0 else "prefill", "V": self.V, "L": self.L, "P": self.P,
                "seg_len": self.seg_len, "S": self.S, "order_version": self.order_version}


_lib = None


def lib() -> ctypes.CDLL:
    """Load libdet_linear.so (once).  Raises if it has not been built: there is no fallback."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(f"{LIB_PATH} is missing: build it with `python -m paper_2609_25624_b200.build`")
        L = ctypes.CDLL(LIB_PATH)
        p, i64, i32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int
        L.det_linear_plan_params.argtypes = [i64, i64, i64, ctypes.POINTER(Params)]
        L.det_linear_plan_params.restype = i32
        L.det_linear_plan.argtypes = [i64, i64, i64]
        L.det_linear_plan.restype = p
        L.det_linear_plan_w.argtypes = [i64, i64, i64, ctypes.c_int32]
        L.det_linear_plan_w.restype = p
        L.det_linear_plan_shard.argtypes = [i64, i64, i64, i64, i64, i64, ctypes.c_int32]
        L.det_linear_plan_shard.restype = p
        L.det_linear_run.argtypes = [p, p, p, p, p, p]
        L.det_linear_run.restype = i32
        L.det_linear_run_w.argtypes = [p, p, p, p, p, p]
        L.det_linear_run_w.restype = i32
        L.det_linear_run_host.argtypes = [p, p, p, p, p, p]
        L.det_linear_run_host.restype = i32
        L.det_linear_run_host_async.argtypes = [p, p, p, p, p, p]
        L.det_linear_run_host_async.restype = i32
        L.det_linear_plan_tune.argtypes = [p, p, p, p, p, p, ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_float)]
        L.det_linear_plan_tune.restype = i32
        L.det_linear_plan_check.argtypes = [p, p]
        L.det_linear_plan_check.restype = i32
        L.det_linear_plan_get_params.argtypes = [p, ctypes.POINTER(Params)]
        L.det_linear_plan_get_params.restype = i32
        L.det_linear_plan_describe.argtypes = [p, ctypes.c_char_p, ctypes.c_size_t]
        L.det_linear_plan_describe.restype = i32
        L.det_linear_plan_destroy.argtypes = [p]
        L.det_linear_plan_destroy.restype = None
        L.det_argmax_rows.argtypes = [p, i64, i64, p, p]
        L.det_argmax_rows.restype = i32
        L.det_rmsnorm.argtypes = [p, p, ctypes.c_float, i64, i64, p, p]
        L.det_rmsnorm.restype = i32
        L.det_attention_decode.argtypes = [p, p, p, ctypes.c_float, i64, i64, i64, i64, i64, p, p]
        L.det_attention_decode.restype = i32
        L.det_last_error.restype = ctypes.c_char_p
        L.det_order_version.restype = i32
        L.det_last_status.restype = i32
        L.det_test_attention_schedule.argtypes = [i64, i64, i64, i64, i64, i32, ctypes.POINTER(ctypes.c_uint64)]
        L.det_test_attention_schedule.restype = i32
        L.det_test_attention_set_split.argtypes = [i32]
        L.det_test_attention_set_split.restype = None
        L.det_test_fail_next_alloc.argtypes = [i32]
        L.det_test_fail_next_alloc.restype = None
        L.det_test_plan_set_wait.argtypes = [p, ctypes.c_uint64, i32]
        L.det_test_plan_set_wait.restype = i32
        L.det_test_plan_force_kernel.argtypes = [p, i32]
        L.det_test_plan_force_kernel.restype = i32
        L.det_test_plan_set_max_blocks.argtypes = [p, i32]
        L.det_test_plan_set_max_blocks.restype = i32
        L.det_test_plan_set_variant.argtypes = [p, i32]
        L.det_test_plan_set_variant.restype = i32
        L.det_test_green_stream_create.argtypes = [i32, ctypes.POINTER(p), ctypes.POINTER(p), ctypes.POINTER(i32)]
        L.det_test_green_stream_create.restype = i32
        L.det_test_green_stream_destroy.argtypes = [p]
        L.det_test_green_stream_destroy.restype = None
        L.det_linear_run_noalloc.argtypes = [i64, i64, i64, p, p, p, p, p]
        L.det_linear_run_noalloc.restype = i32
        L.det_test_linear_atomic_splitk.argtypes = [i64, i64, i64, ctypes.c_int32, p, p, p, p, p]
        L.det_test_linear_atomic_splitk.restype = i32
        L.det_test_scale_cols.argtypes = [p, i64, p, i64, i64, ctypes.c_float, p]
        L.det_test_scale_cols.restype = i32
        L.det_test_measure_fma_peak.argtypes = [i32, ctypes.POINTER(ctypes.c_double)]
        L.det_test_measure_fma_peak.restype = i32
        L.det_test_measure_read_bandwidth.argtypes = [p, ctypes.c_size_t, ctypes.POINTER(ctypes.c_double)]
        L.det_test_measure_read_bandwidth.restype = i32
        _lib = L
    return _lib


def _check(status):
    if status != DET_OK:
        raise DetLinearError(status, det_last_error())


def det_last_error() -> str:
    return lib().det_last_error().decode()


def det_order_version() -> int:
    return int(lib().det_order_version())


def det_last_status() -> int:
    """Status behind the last det_linear_plan* call of this thread (DET_OK if it returned a plan)."""
    return int(lib().det_last_status())


def det_linear_plan_params(M: int, N: int, K: int) -> Params:
    out = Params()
    _check(lib().det_linear_plan_params(M, N, K, ctypes.byref(out)))
    return out


def _stream_ptr(stream):
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


# det_weight_format_t and the torch dtype that carries each format
DET_WEIGHT_BF16, DET_WEIGHT_FP16, DET_WEIGHT_FP32 = 0, 1, 2
WEIGHT_DTYPES = {DET_WEIGHT_BF16: torch.bfloat16, DET_WEIGHT_FP16: torch.float16, DET_WEIGHT_FP32: torch.float32}
WEIGHT_FORMATS = {"bf16": DET_WEIGHT_BF16, "fp16": DET_WEIGHT_FP16, "fp32": DET_WEIGHT_FP32}


class Plan:
    """Owner of a det_linear_plan_t*."""

    def __init__(self, M: int, N: int, K: int, wfmt: int = DET_WEIGHT_BF16, shard=None):
        """shard = (n_begin, n_count, ldy) makes a column-shard plan (det_linear_plan_shard)."""
        self.M, self.N, self.K = int(M), int(N), int(K)
        self.wfmt = WEIGHT_FORMATS.get(wfmt, wfmt) if isinstance(wfmt, str) else int(wfmt)
        self.w_dtype = WEIGHT_DTYPES.get(self.wfmt, torch.bfloat16)
        self.shard = None if shard is None else tuple(int(v) for v in shard)
        if self.shard is not None:
            self._h = lib().det_linear_plan_shard(self.M, self.N, self.K, *self.shard, self.wfmt)
        elif self.wfmt == DET_WEIGHT_BF16:
            self._h = lib().det_linear_plan(self.M, self.N, self.K)
        else:
            self._h = lib().det_linear_plan_w(self.M, self.N, self.K, self.wfmt)
        if not self._h:
            raise DetLinearError(det_last_status(), det_last_error())

    def close(self):
        if getattr(self, "_h", None):
            lib().det_linear_plan_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def handle(self):
        return self._h


def det_linear_plan(M: int, N: int, K: int) -> Plan:
    return Plan(M, N, K)


def det_linear_plan_w(M: int, N: int, K: int, wfmt) -> Plan:
    """Plan for weights stored as "bf16" / "fp16" / "fp32" (or the det_weight_format_t value)."""
    return Plan(M, N, K, wfmt)


def det_linear_plan_shard(M: int, N: int, K: int, n_begin: int, n_count: int, ldy: int, wfmt="bf16") -> Plan:
    """Plan for the column shard [n_begin, n_begin + n_count) of the layer (M, N, K); the order is the
    whole layer's, so the shard's outputs have the bits of the same columns of det_linear_plan(M, N, K)."""
    return Plan(M, N, K, wfmt, shard=(n_begin, n_count, ldy))


def det_linear_run_shard(plan: Plan, x, W_shard, b_shard, y_cols, stream=None) -> None:
    """Run a shard plan.  W_shard [n_count, K] (the shard's weight rows), b_shard [n_count] or None,
    y_cols: a [M, n_count] float32 CUDA view whose row stride is the plan's ldy and column stride 1
    (e.g. y_full[:, n_begin:n_begin + n_count] for ldy = N)."""
    n_begin, n_count, ldy = plan.shard
    _expect(x, torch.float32, (plan.M, plan.K), "x")
    _expect(W_shard, plan.w_dtype, (n_count, plan.K), "W_shard")
    if b_shard is not None:
        _expect(b_shard, torch.float32, (n_count,), "b_shard")
    if (not y_cols.is_cuda or y_cols.dtype != torch.float32 or tuple(y_cols.shape) != (plan.M, n_count)
            or y_cols.stride(1) != 1 or (plan.M > 1 and y_cols.stride(0) != ldy)):
        raise ValueError(f"y_cols: need a float32 CUDA view of shape {(plan.M, n_count)} with strides ({ldy}, 1), "
                         f"got {tuple(y_cols.shape)} strides {y_cols.stride()}")
    _check(lib().det_linear_run_w(plan.handle, x.data_ptr(), W_shard.data_ptr(),
                                  b_shard.data_ptr() if b_shard is not None else None, y_cols.data_ptr(),
                                  _stream_ptr(stream)))


def det_linear_plan_destroy(plan: Plan) -> None:
    plan.close()


def det_linear_plan_get_params(plan: Plan) -> Params:
    out = Params()
    _check(lib().det_linear_plan_get_params(plan.handle, ctypes.byref(out)))
    return out


def det_linear_plan_describe(plan: Plan) -> dict:
    buf = ctypes.create_string_buffer(1024)
    _check(lib().det_linear_plan_describe(plan.handle, buf, 1024))
    return json.loads(buf.value.decode())


def _expect(t, dtype, shape, name):
    if not t.is_cuda or t.dtype != dtype or tuple(t.shape) != tuple(shape) or not t.is_contiguous():
        raise ValueError(f"{name}: need a contiguous CUDA tensor of dtype {dtype} and shape {tuple(shape)}, "
                         f"got {t.dtype} {tuple(t.shape)} cuda={t.is_cuda}")


def det_linear_run(plan: Plan, x, W, b, y, stream=None) -> None:
    """Enqueue y = x . up(W)^T (+ b) on `stream` (default: torch's current stream)."""
    _expect(x, torch.float32, (plan.M, plan.K), "x")
    _expect(W, plan.w_dtype, (plan.N, plan.K), "W")
    _expect(y, torch.float32, (plan.M, plan.N), "y")
    if b is not None:
        _expect(b, torch.float32, (plan.N,), "b")
    fn = lib().det_linear_run if plan.wfmt == DET_WEIGHT_BF16 else lib().det_linear_run_w
    _check(fn(plan.handle, x.data_ptr(), W.data_ptr(), b.data_ptr() if b is not None else None,
              y.data_ptr(), _stream_ptr(stream)))


def det_linear_run_w(plan: Plan, x, W, b, y, stream=None) -> None:
    """det_linear_run for a plan of any weight format (always through the det_linear_run_w entry)."""
    _expect(x, torch.float32, (plan.M, plan.K), "x")
    _expect(W, plan.w_dtype, (plan.N, plan.K), "W")
    _expect(y, torch.float32, (plan.M, plan.N), "y")
    if b is not None:
        _expect(b, torch.float32, (plan.N,), "b")
    _check(lib().det_linear_run_w(plan.handle, x.data_ptr(), W.data_ptr(), b.data_ptr() if b is not None else None,
                                  y.data_ptr(), _stream_ptr(stream)))


def det_linear_run_host(plan: Plan, x_host, W, b, y_host, stream=None, sync: bool = True) -> None:
    """x_host / y_host are (pinned) CPU tensors; W, b are CUDA tensors.  Synchronises the stream
    unless sync=False (then it calls det_linear_run_host_async and the caller synchronises)."""
    for t, shape, name in ((x_host, (plan.M, plan.K), "x_host"), (y_host, (plan.M, plan.N), "y_host")):
        if t.is_cuda or t.dtype != torch.float32 or tuple(t.shape) != shape or not t.is_contiguous():
            raise ValueError(f"{name}: need a contiguous CPU float32 tensor of shape {shape}")
    _expect(W, plan.w_dtype, (plan.N, plan.K), "W")
    if b is not None:
        _expect(b, torch.float32, (plan.N,), "b")
    fn = lib().det_linear_run_host if sync else lib().det_linear_run_host_async
    _check(fn(plan.handle, x_host.data_ptr(), W.data_ptr(), b.data_ptr() if b is not None else None,
              y_host.data_ptr(), _stream_ptr(stream)))


def det_linear_run_host_async(plan: Plan, x_host, W, b, y_host, stream=None) -> None:
    det_linear_run_host(plan, x_host, W, b, y_host, stream=stream, sync=False)


def det_linear_run_noalloc(x, W, b, y, stream=None) -> None:
    """The same linear layer without any allocation (no plan; split-K partials in the library's
    built-in 4 MiB scratch).  For callers that must not allocate: hosts that own all device memory
    through their own pool, plugins after initialisation, latency-critical loops.  Calls whose GPU
    work overlaps race on the shared scratch."""
    M, K = x.shape
    N = W.shape[0]
    _expect(x, torch.float32, (M, K), "x")
    _expect(W, torch.bfloat16, (N, K), "W")
    _expect(y, torch.float32, (M, N), "y")
    if b is not None:
        _expect(b, torch.float32, (N,), "b")
    _check(lib().det_linear_run_noalloc(M, N, K, x.data_ptr(), W.data_ptr(), b.data_ptr() if b is not None else None,
                                        y.data_ptr(), _stream_ptr(stream)))


def det_linear_plan_tune(plan: Plan, x, W, b, y, stream=None):
    """Time the plan's candidate tilings on these buffers and pin the fastest (schedule only: every
    candidate gives the same bits).  Returns (variant, microseconds); (0, -1.0) when there is nothing
    to choose.  Synchronises the stream."""
    n_count = plan.N if plan.shard is None else plan.shard[1]
    _expect(x, torch.float32, (plan.M, plan.K), "x")
    _expect(W, plan.w_dtype, (n_count, plan.K), "W")
    if b is not None:
        _expect(b, torch.float32, (n_count,), "b")
    variant, us = ctypes.c_int32(0), ctypes.c_float(0.0)
    _check(lib().det_linear_plan_tune(plan.handle, x.data_ptr(), W.data_ptr(), b.data_ptr() if b is not None else None,
                                      y.data_ptr(), _stream_ptr(stream), ctypes.byref(variant), ctypes.byref(us)))
    return int(variant.value), float(us.value)


def det_linear_plan_check(plan: Plan, stream=None) -> None:
    _check(lib().det_linear_plan_check(plan.handle, _stream_ptr(stream)))


def det_rmsnorm(x, g, eps: float, y, stream=None) -> None:
    """Fixed-order RMSNorm of the rows of x [M,H] with gain g [H] into y [M,H] (a different buffer)."""
    M, H = x.shape
    _expect(x, torch.float32, (M, H), "x")
    _expect(g, torch.float32, (H,), "g")
    _expect(y, torch.float32, (M, H), "y")
    _check(lib().det_rmsnorm(x.data_ptr(), g.data_ptr(), float(eps), M, H, y.data_ptr(), _stream_ptr(stream)))


def det_attention_decode(q, k, v, scale: float, o, stream=None) -> None:
    """Fixed-order decode attention: q [B,Hq,D], k and v [B,Hkv,T,D], o [B,Hq,D], float32 CUDA tensors."""
    B_, Hq, D = q.shape
    Bk, Hkv, T, Dk = k.shape
    _expect(q, torch.float32, (B_, Hq, D), "q")
    _expect(k, torch.float32, (B_, Hkv, T, D), "k")
    _expect(v, torch.float32, (B_, Hkv, T, D), "v")
    _expect(o, torch.float32, (B_, Hq, D), "o")
    _check(lib().det_attention_decode(q.data_ptr(), k.data_ptr(), v.data_ptr(), float(scale), B_, Hq, Hkv, T, D,
                                      o.data_ptr(), _stream_ptr(stream)))


def det_argmax_rows(y, idx, stream=None) -> None:
    M, N = y.shape
    _expect(y, torch.float32, (M, N), "y")
    _expect(idx, torch.int32, (M,), "idx")
    _check(lib().det_argmax_rows(y.data_ptr(), M, N, idx.data_ptr(), _stream_ptr(stream)))


# ---- test-only exports (include/det_linear_test.h) ------------------------------------------
def det_test_plan_force_kernel(plan: Plan, kernel: int) -> None:
    _check(lib().det_test_plan_force_kernel(plan.handle, kernel))


def det_test_plan_set_max_blocks(plan: Plan, max_blocks: int) -> None:
    _check(lib().det_test_plan_set_max_blocks(plan.handle, max_blocks))


def det_test_plan_set_variant(plan: Plan, variant: int) -> None:
    _check(lib().det_test_plan_set_variant(plan.handle, variant))


def det_test_attention_schedule(B_: int, Hq: int, Hkv: int, T: int, D: int, sm_count: int = 148):
    """(cluster size, shared-memory bytes per block) det_attention_decode would use; host arithmetic only."""
    smem = ctypes.c_uint64(0)
    c = lib().det_test_attention_schedule(B_, Hq, Hkv, T, D, sm_count, ctypes.byref(smem))
    return c, smem.value


def det_test_attention_set_split(blocks_per_row: int) -> None:
    """Force the cluster size of det_attention_decode (1, 2, 4, 8, 16; 0 = automatic).  Same bits for every value."""
    lib().det_test_attention_set_split(blocks_per_row)


def det_test_fail_next_alloc(nth: int = 1) -> None:
    """Host-side fault injection: the nth device allocation from now on fails once (0 = off)."""
    lib().det_test_fail_next_alloc(int(nth))


def det_test_plan_set_wait(plan: Plan, wait_limit_ns: int, withhold_first_copy: bool = False, two_pass_combine: bool = False) -> None:
    """Bound of one device-side wait for this plan's kernels; optionally stall one wait on purpose; optionally make a
    prefill plan fold its K segments with the second launch instead of inside the kernel (same bits)."""
    flags = (1 if withhold_first_copy else 0) | (2 if two_pass_combine else 0)
    _check(lib().det_test_plan_set_wait(plan.handle, int(wait_limit_ns), flags))


def det_test_green_stream_create(sm_count: int):
    """Returns (stream_ptr:int, handle, sm_granted)."""
    st, h, g = ctypes.c_void_p(), ctypes.c_void_p(), ctypes.c_int(0)
    _check(lib().det_test_green_stream_create(sm_count, ctypes.byref(st), ctypes.byref(h), ctypes.byref(g)))
    return st.value, h, g.value


def det_test_green_stream_destroy(handle) -> None:
    lib().det_test_green_stream_destroy(handle)


def det_test_measure_fma_peak(packed) -> float:
    """Measured FP32 FMA issue peak of the CUDA cores in TFLOP/s: False/0 scalar, True/1 packed FP32x2,
    2 the prefill multiply loop alone on resident shared-memory tiles."""
    out = ctypes.c_double(0.0)
    _check(lib().det_test_measure_fma_peak(int(packed), ctypes.byref(out)))
    return out.value


def det_test_measure_read_bandwidth(buf) -> float:
    """Read-only streaming bandwidth in GB/s over a CUDA tensor (use one much larger than L2)."""
    out = ctypes.c_double(0.0)
    _check(lib().det_test_measure_read_bandwidth(buf.data_ptr(), buf.numel() * buf.element_size(), ctypes.byref(out)))
    return out.value


def det_test_linear_atomic_splitk(x, W, b, y, S_req: int, stream=None) -> None:
    """Negative control for rule R3: split-K partials combined with atomicAdd in arrival order."""
    M, K = x.shape
    N = W.shape[0]
    _expect(x, torch.float32, (M, K), "x")
    _expect(W, torch.bfloat16, (N, K), "W")
    _expect(y, torch.float32, (M, N), "y")
    if b is not None:
        _expect(b, torch.float32, (N,), "b")
    _check(lib().det_test_linear_atomic_splitk(M, N, K, int(S_req), x.data_ptr(), W.data_ptr(),
                                               b.data_ptr() if b is not None else None, y.data_ptr(), _stream_ptr(stream)))


def det_test_scale_cols(src, cols: int, c: float, stream=None):
    """Harness glue: returns a new contiguous [M, cols] tensor = src[:, :cols] * c (one rounding each)."""
    M, ld = src.shape
    _expect(src, torch.float32, (M, ld), "src")
    dst = torch.empty((M, cols), dtype=torch.float32, device=src.device)
    _check(lib().det_test_scale_cols(src.data_ptr(), ld, dst.data_ptr(), M, cols, float(c), _stream_ptr(stream)))
    return dst
