"""Exact-rational micro-oracle: the same reduction order, with every binary32 rounding carried out
on Python `fractions.Fraction` values instead of by the CPU's FMA unit.

TEST INFRASTRUCTURE ONLY.  It exists to check the C oracle's arithmetic (is fmaf really a single
rounding? is the tree adjacent-first? are tails skipped?) with an implementation that shares
neither language nor floating-point hardware with it.  Pure Python loops: tiny shapes only.

Values are Python floats that are exactly representable in binary32 (a Python float can hold any
binary32 value, including signed zeros and infinities).
"""
import math
import struct
from fractions import Fraction

_MIN_EXP = -126          # exponent of the smallest normal binary32
_MANT = 23               # explicit significand bits
_MAX_FINITE = Fraction(2 ** 24 - 1, 1) * Fraction(2) ** (127 - 23)


def bf16_bits_to_float(h: int) -> float:
    """up(): the binary32 value whose bit pattern is h << 16 (Eq. 2's register upcast)."""
    return struct.unpack("<f", struct.pack("<I", (h & 0xFFFF) << 16))[0]


def fp16_bits_to_float(h: int) -> float:
    """up() for IEEE binary16 bit patterns (exact: every binary16 value is a binary32 value)."""
    return struct.unpack("<e", struct.pack("<H", h & 0xFFFF))[0]


def round_to_binary32(q: Fraction) -> float:
    """Round an exact rational to the nearest binary32, ties to even, gradual underflow,
    overflow to infinity (IEEE-754 roundTiesToEven)."""
    if q == 0:
        return 0.0
    sign = -1.0 if q < 0 else 1.0
    a = -q if q < 0 else q
    # e = floor(log2(a)), found exactly
    e = a.numerator.bit_length() - a.denominator.bit_length()
    if Fraction(2) ** e > a:
        e -= 1
    elif Fraction(2) ** (e + 1) <= a:
        e += 1
    quantum = Fraction(2) ** (max(e, _MIN_EXP) - _MANT)
    n = a / quantum
    lo = n.numerator // n.denominator
    rem = n - lo
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and (lo & 1)):
        lo += 1
    r = lo * quantum
    # IEEE overflow rule: a value that rounds (with unbounded exponent) beyond the largest finite
    # number becomes infinity
    if r > _MAX_FINITE:
        return sign * math.inf
    return sign * float(r)       # exact: r has at most 24 significant bits; -0.0 when r == 0


def _is_neg(v: float) -> bool:
    return math.copysign(1.0, v) < 0


def fma32(x: float, w: float, a: float) -> float:
    """fusedMultiplyAdd in binary32: x*w + a with one rounding (rule R1)."""
    if not (math.isfinite(x) and math.isfinite(w) and math.isfinite(a)):
        raise ValueError("exact micro-oracle handles finite operands only")
    q = Fraction(x) * Fraction(w) + Fraction(a)
    if q != 0:
        return round_to_binary32(q)        # a nonzero value that underflows keeps its own sign
    # exact zero: -0 only when a zero product of negative sign meets a = -0; a cancellation of
    # nonzero terms gives +0 under roundTiesToEven
    prod_is_zero = (x == 0 or w == 0)
    prod_neg = _is_neg(x) != _is_neg(w)
    return -0.0 if (prod_is_zero and prod_neg and _is_neg(a)) else 0.0


def add32(a: float, b: float) -> float:
    """binary32 addition, one rounding."""
    if not (math.isfinite(a) and math.isfinite(b)):
        raise ValueError("exact micro-oracle handles finite operands only")
    q = Fraction(a) + Fraction(b)
    if q == 0:
        zneg = (a == 0 and b == 0 and _is_neg(a) and _is_neg(b))
        return -0.0 if zneg else 0.0
    return round_to_binary32(q)


def output(xrow, wrow, bias, V, L, P, seg_len, wfmt="bf16"):
    """One output element.  xrow: binary32-representable floats; wrow: BF16 or FP16 bit patterns
    (ints) or, for wfmt="fp32", binary32-representable floats; bias: float or None.  Follows the order family (V, L, P, seg_len): chunks of V*L elements
    ascending, lane l owns V consecutive elements, element j feeds sub-chain j mod P, leaves are
    tree-summed adjacent-first, segments are summed ascending, bias is added last."""
    K = len(xrow)
    assert len(wrow) == K
    decode = {"bf16": bf16_bits_to_float, "fp16": fp16_bits_to_float, "fp32": float}[wfmt]
    nleaf = L * P
    assert nleaf & (nleaf - 1) == 0
    C = V * L
    t = None
    k_lo = 0
    while k_lo < K:
        k_hi = min(K, k_lo + seg_len)
        a = [0.0] * nleaf
        c = k_lo
        while c < k_hi:
            for l in range(L):
                for j in range(V):
                    k = c + l * V + j
                    if k < k_hi:
                        leaf = l * P + (j % P)
                        a[leaf] = fma32(xrow[k], decode(wrow[k]), a[leaf])
            c += C
        w = nleaf
        while w > 1:
            a = [add32(a[2 * i], a[2 * i + 1]) for i in range(w // 2)]
            w //= 2
        t = a[0] if t is None else add32(t, a[0])
        k_lo += seg_len
    return add32(t, bias) if bias is not None else t


def linear(x, W_bits, b, V, L, P, seg_len, wfmt="bf16"):
    """Whole (tiny) problem as nested lists: y[m][n]."""
    conv = float if wfmt == "fp32" else int
    return [[output(list(map(float, xr)), list(map(conv, wr)), None if b is None else float(b[n]),
                    V, L, P, seg_len, wfmt)
             for n, wr in enumerate(W_bits)] for xr in x]


# ---- fixed-order RMSNorm, exact-rational version --------------------------------------------------

def mul32(a: float, b: float) -> float:
    """binary32 multiplication, one rounding (finite, nonzero-sign handling as for add32)."""
    q = Fraction(a) * Fraction(b)
    if q == 0:
        return -0.0 if (_is_neg(a) != _is_neg(b)) else 0.0
    return round_to_binary32(q)


def div32(a: float, b: float) -> float:
    """binary32 division a / b, one rounding; b != 0."""
    q = Fraction(a) / Fraction(b)
    if q == 0:
        return -0.0 if (_is_neg(a) != _is_neg(b)) else 0.0
    return round_to_binary32(q)


def sqrt32(t: float) -> float:
    """Correctly rounded binary32 square root of t >= 0.  The root is bracketed to 2^-160 with an
    integer square root; a binary32 rounding boundary (a 25-bit number) can only be hit exactly by
    a perfect square, which is detected, so a point strictly inside the bracket rounds correctly."""
    if t == 0:
        return t
    q = Fraction(t)
    k = 160
    scaled = q * Fraction(4) ** k                    # t * 2^(2k)
    num = scaled.numerator // scaled.denominator
    exact_int = scaled.denominator == 1
    n = math.isqrt(num)
    if exact_int and n * n == num:
        return round_to_binary32(Fraction(n, 2 ** k))
    return round_to_binary32(Fraction(2 * n + 1, 2 ** (k + 1)))


def sum_squares(xrow) -> float:
    """Decode-order sum of squares: chunks of 128 ascending, lane l owns 4 consecutive elements,
    fma(x, x, acc) from +0, tails skipped, adjacent-first tree over the 32 lanes."""
    H = len(xrow)
    lanes = [0.0] * 32
    for c in range(0, H, 128):
        for l in range(32):
            for j in range(4):
                k = c + 4 * l + j
                if k < H:
                    lanes[l] = fma32(xrow[k], xrow[k], lanes[l])
    w = 32
    while w > 1:
        lanes = [add32(lanes[2 * i], lanes[2 * i + 1]) for i in range(w // 2)]
        w //= 2
    return lanes[0]


def rmsnorm_row(xrow, g, eps: float):
    H = len(xrow)
    ss = sum_squares(xrow)
    mean = div32(ss, round_to_binary32(Fraction(H)))
    t = add32(mean, eps)
    r = div32(1.0, sqrt32(t))
    return [mul32(mul32(xv, r), gv) for xv, gv in zip(xrow, g)]


# ---- fixed-order decode attention (same definition as the C oracle, on exact rationals) ----------
def _f32(bits: int) -> float:
    return struct.unpack("<f", struct.pack("<I", bits))[0]


def rint32(t: float) -> float:
    """Round to the nearest integer, ties to even (what rintf does in the default rounding mode)."""
    q = Fraction(t)
    lo = q.numerator // q.denominator
    rem = q - lo
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and (lo & 1)):
        lo += 1
    if lo == 0:
        return -0.0 if _is_neg(t) else 0.0
    return float(lo)


def exp_det(x: float) -> float:
    """The attention's exponential for x <= 0: range reduction by ln 2 in two pieces, a degree-7 Taylor
    polynomial evaluated by Horner's rule with fused multiply-adds, scaling by 2^n (through 2^(n+64) and
    2^-64 below the normal range); every step one binary32 operation."""
    if x > 0:
        raise ValueError("exp_det is defined for x <= 0")
    if x < -104.0:
        return 0.0
    t = mul32(x, _f32(0x3FB8AA3B))
    n = rint32(t)
    f = fma32(n, -_f32(0x3F317200), x)
    f = fma32(n, -_f32(0x35BFBE8E), f)
    p = _f32(0x39500D01)
    for c in (_f32(0x3AB60B61), _f32(0x3C088889), _f32(0x3D2AAAAB), _f32(0x3E2AAAAB), 0.5, 1.0, 1.0):
        p = fma32(p, f, c)
    ni = int(n)
    if ni >= -126:
        return mul32(p, math.ldexp(1.0, ni))
    return mul32(mul32(p, math.ldexp(1.0, ni + 64)), math.ldexp(1.0, -64))


def _lane_tree(acc):
    w = len(acc)
    while w > 1:
        acc = [add32(acc[2 * i], acc[2 * i + 1]) for i in range(w // 2)]
        w //= 2
    return acc[0]


def lane_dot(a, b) -> float:
    acc = [0.0] * 32
    D = len(a)
    for c in range(0, D, 128):
        for l in range(32):
            for j in range(4):
                k = c + 4 * l + j
                if k < D:
                    acc[l] = fma32(a[k], b[k], acc[l])
    return _lane_tree(acc)


def lane_sum(e) -> float:
    acc = [0.0] * 32
    T = len(e)
    for c in range(0, T, 128):
        for l in range(32):
            for j in range(4):
                k = c + 4 * l + j
                if k < T:
                    acc[l] = add32(acc[l], e[k])
    return _lane_tree(acc)


def attention_row(q, keys, values, scale: float):
    """One (batch, head): q [D], keys and values [T][D] (lists of binary32-representable floats)."""
    T, D = len(keys), len(q)
    s = [mul32(lane_dot(q, keys[j]), scale) for j in range(T)]
    m = max(s)
    e = [exp_det(add32(s[j], -m)) for j in range(T)]
    l = lane_sum(e)
    out = []
    for d in range(D):
        t = None
        for j0 in range(0, T, 256):
            a = 0.0
            for j in range(j0, min(T, j0 + 256)):
                a = fma32(e[j], values[j][d], a)
            t = a if t is None else add32(t, a)
        out.append(div32(t, l))
    return out
