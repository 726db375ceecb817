"""Parser for tests/golden/order_examples.txt (hand-traced reduction-order examples)."""
import os
import struct

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
T = float(2 ** 24)
ONE_BF16 = 0x3F80


def _f32_from_bits(b):
    return struct.unpack("<f", struct.pack("<I", b))[0]


def _parse_x(field):
    field = field.strip()
    if field[:1] in ("K", "Z") and ":" in field and field[1:field.index(":")].isdigit():
        # "K<n>: i=v, ..." = a row of n ones with the listed overrides; "Z<n>: ..." = a row of n zeros
        n = int(field[1:field.index(":")])
        x = [1.0 if field[0] == "K" else 0.0] * n
        for item in field[field.index(":") + 1:].split(","):
            i, v = item.split("=")
            x[int(i)] = _parse_val(v.strip())
        return x
    if field.startswith("xbits"):
        return [_f32_from_bits(int(t, 16)) if t.lower().startswith("0x") else float(t)
                for t in field.split()[1:]]
    return [_parse_val(t) for t in field.split()]


def _parse_val(t):
    if t == "T":
        return T
    if t == "-T":
        return -T
    return float(t)


def load_order_examples():
    """Yield dicts: name, x (floats), w (BF16 bit patterns), b (float or None), V, L, P, s_req,
    granule, expected."""
    out = []
    with open(os.path.join(GOLDEN, "order_examples.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            parts = [p.strip() for p in line.split(";")]
            name, xf, vlp, s_req, gran, exp = parts[:6]
            x = _parse_x(xf)
            w = [ONE_BF16] * len(x)
            b = None
            for extra in parts[6:]:
                toks = extra.split()
                if toks[0] == "w":
                    w = [int(t, 16) if t.lower().startswith("0x") else int(t) for t in toks[1:]]
                elif toks[0] == "b":
                    b = float(toks[1])
            V, L, P = (int(t) for t in vlp.split())
            out.append(dict(name=name, x=x, w=w, b=b, V=V, L=L, P=P, s_req=int(s_req),
                            granule=int(gran), expected=float(exp)))
    return out


def seg_len_for(K, s_req, granule):
    """Segment length rule: boundaries on multiples of `granule`, every segment non-empty."""
    n_g = -(-K // granule)
    per = -(-n_g // min(s_req, n_g))
    return granule * per


def load_layout_example():
    rows = []
    with open(os.path.join(GOLDEN, "layout_example.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            rows.append([float(t) for t in line.split()])
    return rows
