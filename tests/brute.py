"""Per-element Python loops over the definitions (Eq. 1-2, Eq. 6, Eq. 10-11).

Deliberately scalar: math.exp / math.cos on Python floats, one element at a
time, nothing vectorised.  Used only to pin the numpy oracle on tiny inputs.
"""
import math


def bf16_to_float(bits: int) -> float:
    import struct
    return struct.unpack("<f", struct.pack("<I", (int(bits) & 0xFFFF) << 16))[0]


def float_to_bf16_bits(x: float) -> int:
    """Round a Python float to bf16, ties to even, by exact rational comparison of neighbours."""
    import struct
    from fractions import Fraction
    if x == 0.0:
        return 0x8000 if math.copysign(1.0, x) < 0 else 0
    f32 = struct.unpack("<f", struct.pack("<f", x))[0]            # nearby fp32 only to find the neighbourhood
    u = struct.unpack("<I", struct.pack("<f", f32))[0]
    lo = u & 0xFFFF0000
    cands = []
    for delta in (-0x10000, 0, 0x10000):
        c = lo + delta
        if 0 <= (c & 0x7FFFFFFF) < 0x7F800000:
            cands.append(c >> 16)
    fx = Fraction(x)
    best = None
    for c in cands:
        val = Fraction(bf16_to_float(c))
        err = abs(val - fx)
        key = (err, c & 1)                                         # tie -> even mantissa
        if best is None or key < best[0]:
            best = (key, c)
    return best[1]


def rope_scalar(vec, p, theta):
    d = len(vec)
    h = d // 2
    out = [0.0] * d
    for t in range(h):
        phi = p * theta ** (-2.0 * t / d)
        c, s = math.cos(phi), math.sin(phi)
        out[t] = vec[t] * c - vec[t + h] * s
        out[t + h] = vec[t + h] * c + vec[t] * s
    return out


def rope_round_token(bits_vec, p, theta):
    rot = rope_scalar([bf16_to_float(b) for b in bits_vec], p, theta)
    return [bf16_to_float(float_to_bf16_bits(x)) for x in rot]


def causal_attention_loops(q_bits, k_bits, v_bits, c, h, theta, scale):
    """Returns (A rows as list of lists, O rows, LSE list) for chunk c, q-head h; everything by loops."""
    L, Hq, d = len(q_bits[c]), len(q_bits[c][0]), len(q_bits[c][0][0])
    Hkv = len(k_bits[c][0])
    hk = h // (Hq // Hkv)
    qr = [rope_round_token(q_bits[c][i][h], i, theta) for i in range(L)]
    kr = [rope_round_token(k_bits[c][j][hk], j, theta) for j in range(L)]
    vv = [[bf16_to_float(b) for b in v_bits[c][j][hk]] for j in range(L)]
    A, O, LSE = [], [], []
    for i in range(L):
        logits = []
        for j in range(i + 1):
            acc = 0.0
            for t in range(d):
                acc += qr[i][t] * kr[j][t]
            logits.append(acc * scale)
        mx = max(logits)
        ex = [math.exp(x - mx) for x in logits]
        z = sum(ex)
        row = [e / z for e in ex] + [0.0] * (L - i - 1)
        A.append(row)
        O.append([sum(row[j] * vv[j][t] for j in range(i + 1)) for t in range(d)])
        LSE.append(mx + math.log(z))
    return A, O, LSE
