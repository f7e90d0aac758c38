"""A second, deliberately different restatement of the paper's integer rules in pure Python,
used only to cross-check the C oracle on tiny inputs (two independent transcriptions agreeing
catches slips in either).  Rounding works on bit *strings*; sums use Python ints."""
import numpy as np


def bit_length_of_max(values):
    return max((abs(int(v)) for v in values), default=0).bit_length()


def psr_bits(x, bp, mbits=7):
    """Algorithm 3 on the binary expansion of |x| written as a string."""
    x = int(x)
    s = bin(abs(x))[2:].zfill(bp + 1)
    int_part, frac = s[:len(s) - bp], s[len(s) - bp:] if bp else ""
    q = int(int_part, 2)
    if len(frac) % 2 == 1:
        frac = frac[:-1]                     # drop the least significant fraction bit
    half = len(frac) // 2
    top, bot = frac[:half], frac[half:]
    if half and int(top, 2) > int(bot, 2):
        q += 1
    q = min(q, 2 ** mbits - 1)
    return -q if x < 0 else q


def nearest_bits(x, bp, mbits=7):
    x = int(x)
    m = abs(x)
    q = (m + (1 << (bp - 1))) >> bp if bp else m
    q = min(q, 2 ** mbits - 1)
    return -q if x < 0 else q


def shift_round(acc, mbits=7, rounder=psr_bits):
    flat = [int(v) for v in np.asarray(acc).reshape(-1)]
    b = bit_length_of_max(flat)
    bp = max(0, b - mbits)
    q = np.array([rounder(v, bp, mbits) for v in flat], dtype=np.int64).reshape(np.shape(acc))
    return q, b, bp


def conv_fwd_padded(x, w, pad):
    """Zero-pads x explicitly and slides the window: x [B,H,W,Ci], w [Co,R,S,Ci]."""
    x = np.asarray(x, dtype=object)
    B, H, W, Ci = x.shape
    Co, R, S, _ = w.shape
    xp = np.zeros((B, H + 2 * pad, W + 2 * pad, Ci), dtype=object)
    xp[:, pad:pad + H, pad:pad + W, :] = x
    Ho, Wo = H + 2 * pad - R + 1, W + 2 * pad - S + 1
    y = np.zeros((B, Ho, Wo, Co), dtype=object)
    for b in range(B):
        for i in range(Ho):
            for j in range(Wo):
                win = xp[b, i:i + R, j:j + S, :]
                for co in range(Co):
                    y[b, i, j, co] = int((win * w[co].astype(object)).sum())
    return y.astype(np.int64)


def xent_row(a_row, s_a, label):
    """Section 3.5 for one sample with Python ints; returns the unrounded e32 row."""
    a_row = [int(v) for v in a_row]
    if s_a <= -7:
        T = [2 ** (1 - 2 * s_a) + a * 2 ** (1 - s_a) + a * a for a in a_row]
    else:
        xh = []
        for a in a_row:
            P = 47274 * a
            sh = 15 - s_a
            xh.append(P // (2 ** sh) if sh >= 0 else P * 2 ** (-sh))   # floor division
        mx = max(xh)
        p = min(v for v in xh if v > mx - 10)
        T = [2 ** max(0, v - p) for v in xh]
    Csum = sum(T)
    return [t - (Csum if i == label else 0) for i, t in enumerate(T)]
