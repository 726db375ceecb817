"""Seeded synthetic inputs for the fused-upcast linear layer.

This module holds none of the method's arithmetic: it only draws numbers.  Every tensor is drawn
from a CPU generator with a fixed seed and copied to the device afterwards, so every run and
every device sees identical input bits (the paper's seeded-probe methodology: inputs are seeded
on the CPU so every GPU sees identical bits).

Value recipe (stands in for real checkpoints and prompts, which are not available offline):
W = round-to-nearest-even BF16 of N(0, 0.02^2) drawn in FP32, x ~ N(0, 1) FP32,
b ~ N(0, 0.01^2) FP32; drawn in the order W, x, b from one generator.
"""
import zlib

import numpy as np
import torch

#: Llama-3-8B-architecture projection shapes as (name, K, N)
LLAMA3_8B_LAYER = (("qkv", 4096, 6144), ("o", 4096, 4096), ("gate_up", 4096, 28672),
                   ("down", 14336, 4096))
LLAMA3_8B_LM_HEAD = ("lm_head", 4096, 128256)
DECODE_MS = (1, 4, 8, 16, 32)
LM_HEAD_MS = (1, 8, 32)
PREFILL_MS = (128, 512, 2048)
PREFILL_SHAPES = (("gate_up", 4096, 28672), ("down", 14336, 4096))


def shape_seed(M: int, N: int, K: int) -> int:
    """Seed per problem shape."""
    return zlib.crc32(f"{M},{N},{K}".encode())


def named_seed(name: str) -> int:
    return zlib.crc32(name.encode())


def make_case(M: int, N: int, K: int, seed=None, bias: bool = True):
    """Return (x [M,K] float32, W [N,K] bfloat16, b [N] float32 or None) as CPU tensors."""
    g = torch.Generator(device="cpu")
    g.manual_seed(shape_seed(M, N, K) if seed is None else int(seed))
    W = (0.02 * torch.randn(N, K, dtype=torch.float32, generator=g)).to(torch.bfloat16)
    x = torch.randn(M, K, dtype=torch.float32, generator=g)
    b = 0.01 * torch.randn(N, dtype=torch.float32, generator=g) if bias else None
    return x, W, b


#: torch dtype that carries each weight format
WEIGHT_DTYPES = {"bf16": torch.bfloat16, "fp16": torch.float16, "fp32": torch.float32}


def make_case_w(M: int, N: int, K: int, wfmt: str, seed=None, bias: bool = True):
    """make_case with the weights stored as "bf16", "fp16" or "fp32": the same FP32 draws, rounded to
    nearest even into the 16-bit formats (about 0.2 % of the FP16 weights are then subnormal) or
    kept as drawn for FP32."""
    g = torch.Generator(device="cpu")
    g.manual_seed(shape_seed(M, N, K) if seed is None else int(seed))
    W = (0.02 * torch.randn(N, K, dtype=torch.float32, generator=g)).to(WEIGHT_DTYPES[wfmt])
    x = torch.randn(M, K, dtype=torch.float32, generator=g)
    b = 0.01 * torch.randn(N, dtype=torch.float32, generator=g) if bias else None
    return x, W, b


def weight_format_of(W: torch.Tensor) -> str:
    for name, dt in WEIGHT_DTYPES.items():
        if W.dtype == dt:
            return name
    raise ValueError(f"no weight format for dtype {W.dtype}")


def weight_bits(W: torch.Tensor) -> np.ndarray:
    """Weight tensor -> numpy array of its stored elements: uint16 bit patterns for the 16-bit
    formats, float32 for FP32 (same memory layout)."""
    if W.dtype == torch.float32:
        return W.contiguous().numpy()
    assert W.dtype in (torch.bfloat16, torch.float16)
    return W.contiguous().view(torch.int16).numpy().view(np.uint16)


def make_weight(N: int, K: int, seed: int):
    """One BF16 weight matrix [N,K] ~ N(0, 0.02^2) (for the multi-layer stack)."""
    g = torch.Generator(device="cpu")
    g.manual_seed(int(seed))
    return (0.02 * torch.randn(N, K, dtype=torch.float32, generator=g)).to(torch.bfloat16)


def make_int_case(M: int, N: int, K: int, seed: int = 0, bias: bool = True, lo: int = -8, hi: int = 8):
    """Integer-valued inputs in [lo, hi]: every value is exact in BF16 and FP32 and, for
    K * max|x| * max|w| < 2^24, every partial sum in any order is exact."""
    g = torch.Generator(device="cpu")
    g.manual_seed(int(seed))
    W = torch.randint(lo, hi + 1, (N, K), generator=g).to(torch.float32).to(torch.bfloat16)
    x = torch.randint(lo, hi + 1, (M, K), generator=g).to(torch.float32)
    b = torch.randint(lo, hi + 1, (N,), generator=g).to(torch.float32) if bias else None
    return x, W, b


def bf16_bits(W: torch.Tensor) -> np.ndarray:
    """BF16 tensor -> numpy uint16 bit patterns (same memory layout)."""
    assert W.dtype == torch.bfloat16
    return W.contiguous().view(torch.int16).numpy().view(np.uint16)


def bits_to_bf16(bits: np.ndarray) -> torch.Tensor:
    """numpy uint16 bit patterns -> BF16 CPU tensor."""
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16)


def make_near_tie(W: torch.Tensor, r1: int, r2: int, n_positions: int = 16, seed: int = 0):
    """Copy row r1 of W over row r2, then move `n_positions` seeded entries of row r2 to the
    adjacent BF16 value (bit pattern +-1, seeded sign).  With n_positions = 0 the two rows are
    identical (an exact tie).  Returns a new tensor."""
    bits = bf16_bits(W).copy()
    bits[r2] = bits[r1]
    rng = np.random.default_rng(seed)
    K = bits.shape[1]
    if n_positions:
        pos = rng.choice(K, size=n_positions, replace=False)
        sign = rng.integers(0, 2, size=n_positions) * 2 - 1
        for k, s in zip(pos, sign):
            v = int(bits[r2, k])
            mag = v & 0x7FFF
            if mag == 0 and s < 0:            # stay finite and keep the pattern valid
                s = 1
            bits[r2, k] = np.uint16((v & 0x8000) | ((mag + int(s)) & 0x7FFF))
    return bits_to_bf16(bits)
