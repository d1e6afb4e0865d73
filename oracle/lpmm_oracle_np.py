"""Second, independent writing of the oracle in NumPy (TEST INFRASTRUCTURE ONLY).

It restates the same definitions as oracle/lpmm_oracle.c with array operations instead of loops
and shares no code with it; the two are compared bit for bit in the CPU test-suite, so a slip in
either one shows up without any GPU. Every float operation is a separate NumPy float32 ufunc call
(NumPy never fuses a multiply with an add), so the rounding sequence equals the C oracle's.
"""
from __future__ import annotations

from fractions import Fraction

import numpy as np

F32 = np.float32
FLT_MIN = np.finfo(np.float32).tiny  # smallest normal binary32


# ----------------------------------------------------------------------------- mappings

def linear_map(bits: int = 4) -> np.ndarray:
    """App. E.2: T(i) = (i+1)/2^b; zero is excluded (Sec. 4.1)."""
    return np.array([Fraction(i + 1, 2 ** bits) for i in range(2 ** bits)], dtype=np.float64).astype(F32)


def de_fraction(F: int, k: int) -> Fraction:
    """App. E.2: midpoint of the k-th of 2^F equal cells of [0.1, 1]."""
    p = lambda j: Fraction(9, 10) * Fraction(j, 2 ** F) + Fraction(1, 10)
    return (p(k) + p(k + 1)) / 2


def _de_value(bitstring: str) -> Fraction:
    E = len(bitstring) - len(bitstring.lstrip("0"))       # leading zeros
    frac_bits = bitstring[E + 1:]                          # after the indicator bit
    k = int(frac_bits, 2) if frac_bits else 0
    return Fraction(1, 10 ** E) * de_fraction(len(frac_bits), k)


def de_map(bits: int = 4, signed: bool = True, drop_zero: bool = False) -> np.ndarray:
    """App. E.2: dynamic-exponent table from the bit patterns, sorted increasingly."""
    vals = []
    for p in range(2 ** bits):
        s = format(p, f"0{bits}b")
        if not signed:
            if p == 0:
                v = Fraction(0)
            elif p == 1:
                v = Fraction(1)
            else:
                v = _de_value(s)
        else:
            sign, rest = s[0], s[1:]
            if int(rest, 2) == 0:
                v = Fraction(1) if sign == "1" else Fraction(0)
            else:
                v = _de_value(rest) * (-1 if sign == "1" else 1)
        if drop_zero and v == 0:
            continue
        vals.append(v)
    vals.sort()
    # Fraction -> float is correctly rounded to binary64; the binary32 cast then rounds again, which
    # could only differ from direct rounding at an exact binary32 midpoint (none of these is one).
    return np.array([float(v) for v in vals], dtype=np.float64).astype(F32)


def nearest(T: np.ndarray, n: np.ndarray) -> np.ndarray:
    """Sec. 2.2: argmin_i |n - T(i)|, exact (binary64 differences), first minimiser on ties."""
    n = np.asarray(n, dtype=F32)
    out = np.empty(n.size, np.uint8)
    flat = n.ravel().astype(np.float64)
    T64 = T.astype(np.float64)
    step = 1 << 18
    for lo in range(0, flat.size, step):
        d = np.abs(flat[lo:lo + step, None] - T64[None, :])
        out[lo:lo + step] = np.argmin(d, axis=1)
    return out.reshape(n.shape)


def rcp(s: np.ndarray) -> np.ndarray:
    s = np.asarray(s, dtype=F32)
    safe = np.where(s >= FLT_MIN, s, F32(1.0))
    return np.where(s >= FLT_MIN, F32(1.0) / safe, F32(0.0)).astype(F32)


# ----------------------------------------------------------------------------- normalizers

def block_scales(x: np.ndarray, B: int) -> np.ndarray:
    a = np.abs(np.asarray(x, F32).ravel())
    nb = -(-a.size // B)
    pad = np.zeros(nb * B, F32)
    pad[:a.size] = a
    return pad.reshape(nb, B).max(axis=1)


def rank1_stats(x: np.ndarray) -> list[np.ndarray]:
    """Alg. 4 first loop: per-axis maxima of |x|."""
    a = np.abs(np.asarray(x, F32))
    return [a.max(axis=tuple(ax for ax in range(a.ndim) if ax != r)) for r in range(a.ndim)]


def rank1_scale_field(shape, stats) -> np.ndarray:
    """Alg. 4 second loop: element-wise minimum over the axes' statistics."""
    M = None
    for r, mu in enumerate(stats):
        view = [1] * len(shape)
        view[r] = shape[r]
        b = np.broadcast_to(mu.reshape(view), shape)
        M = b if M is None else np.minimum(M, b)
    return np.ascontiguousarray(M, dtype=F32)


def quantize_block(x, B, T, scale=None, true_division=False):
    x = np.asarray(x, F32).ravel()
    if scale is None:
        scale = block_scales(x, B)
    s_elem = np.repeat(scale, B)[:x.size]
    if true_division:
        ok = s_elem >= FLT_MIN
        n = np.where(ok, x / np.where(ok, s_elem, F32(1)), F32(0)).astype(F32)
    else:
        n = x * rcp(s_elem)
    return nearest(T, n), scale


def quantize_rank1(x, T, r=None, c=None, true_division=False):
    a = np.abs(np.asarray(x, F32))
    if r is None:
        r, c = a.max(axis=1), a.max(axis=0)
    if true_division:
        s = np.minimum(r[:, None], c[None, :])
        ok = s >= FLT_MIN
        n = np.where(ok, a / np.where(ok, s, F32(1)), F32(0)).astype(F32)
    else:
        n = a * np.maximum(rcp(r)[:, None], rcp(c)[None, :])
    return nearest(T, n), r, c


def dequantize_block(codes, B, T, scale):
    codes = np.asarray(codes).ravel()
    return T[codes] * np.repeat(scale, B)[:codes.size]


def dequantize_rank1(codes, T, r, c):
    return T[np.asarray(codes)] * np.minimum(r[:, None], c[None, :])


def pack4(codes):
    q = np.asarray(codes, np.uint8).ravel()
    if q.size % 2:
        q = np.concatenate([q, np.zeros(1, np.uint8)])
    return (q[0::2] | (q[1::2] << 4)).astype(np.uint8)


def unpack4(packed, numel):
    p = np.asarray(packed, np.uint8).ravel()
    q = np.empty(p.size * 2, np.uint8)
    q[0::2] = p & 0x0F
    q[1::2] = p >> 4
    return q[:numel]


# ----------------------------------------------------------------------------- the step

def adamw4_step(w, g, state: dict, *, lr, beta1, beta2, eps, weight_decay, step, true_division=False):
    """Alg. 3 (compressed Adam) with Eq. 1 and decoupled weight decay on one tensor.

    state: {"kind": "fp32"|"block"|"rank1", "rows", "cols", "m_block", "v_block", and either
    "m32","v32" or "m_codes","m_scale","v_codes","v_s0"[, "v_s1"]} with packed uint8 codes.
    Returns the new w (float32, flat) and updates `state` in place.
    """
    rows, cols = state["rows"], state["cols"]
    numel = rows * cols
    w = np.asarray(w, F32).ravel()
    g = np.asarray(g, F32).ravel()
    lr, beta1, beta2, eps, wd = F32(lr), F32(beta1), F32(beta2), F32(eps), F32(weight_decay)
    Tde, Tlin = de_map(4, True), linear_map(4)
    kind = state["kind"]

    if kind == "fp32":
        m, v = state["m32"], state["v32"]
    else:
        m = dequantize_block(unpack4(state["m_codes"], numel), state["m_block"], Tde, state["m_scale"])
        qv = unpack4(state["v_codes"], numel)
        if kind == "block":
            v = dequantize_block(qv, state["v_block"], Tlin, state["v_s0"])
        else:
            v = dequantize_rank1(qv.reshape(rows, cols), Tlin, state["v_s0"], state["v_s1"]).ravel()

    omb1 = F32(1.0) - beta1
    omb2 = F32(1.0) - beta2
    bc1 = F32(1.0 - float(beta1) ** step)
    bc2 = F32(1.0 - float(beta2) ** step)
    mt = beta1 * m + omb1 * g
    vt = beta2 * v + omb2 * (g * g)
    mhat = mt / bc1
    vhat = vt / bc2
    upd = lr * (mhat / (np.sqrt(vhat) + eps))
    w_new = w * (F32(1.0) - lr * wd) - upd

    if kind == "fp32":
        state["m32"], state["v32"] = mt, vt
    else:
        qm, state["m_scale"] = quantize_block(mt, state["m_block"], Tde, true_division=true_division)
        state["m_codes"] = pack4(qm)
        if kind == "block":
            qv, state["v_s0"] = quantize_block(vt, state["v_block"], Tlin, true_division=true_division)
        else:
            qv, state["v_s0"], state["v_s1"] = quantize_rank1(vt.reshape(rows, cols), Tlin,
                                                              true_division=true_division)
        state["v_codes"] = pack4(qv)
    return w_new.astype(F32)


def adamw4_step_nd(w, g, state: dict, *, lr, beta1, beta2, eps, weight_decay, step):
    """Alg. 3 on a tensor of any rank with Alg. 4's normalization for the second moment.

    state: {"dims", "m_block", "m_codes", "m_scale", "v_codes", "mu": [per-axis maxima]}; returns the new w (flat).
    """
    dims = tuple(int(d) for d in state["dims"])
    numel = int(np.prod(dims))
    w = np.asarray(w, F32).ravel()
    g = np.asarray(g, F32).ravel()
    lr, beta1, beta2, eps, wd = F32(lr), F32(beta1), F32(beta2), F32(eps), F32(weight_decay)
    Tde, Tlin = de_map(4, True), linear_map(4)
    m = dequantize_block(unpack4(state["m_codes"], numel), state["m_block"], Tde, state["m_scale"])
    v = (Tlin[unpack4(state["v_codes"], numel)] * rank1_scale_field(dims, state["mu"]).ravel()).astype(F32)
    omb1, omb2 = F32(1.0) - beta1, F32(1.0) - beta2
    bc1 = F32(1.0 - float(beta1) ** step)
    bc2 = F32(1.0 - float(beta2) ** step)
    mt = beta1 * m + omb1 * g
    vt = beta2 * v + omb2 * (g * g)
    upd = lr * ((mt / bc1) / (np.sqrt(vt / bc2) + eps))
    w_new = w * (F32(1.0) - lr * wd) - upd
    qm, state["m_scale"] = quantize_block(mt, state["m_block"], Tde)
    state["m_codes"] = pack4(qm)
    state["mu"] = rank1_stats(vt.reshape(dims))
    M = rank1_scale_field(dims, state["mu"]).ravel()
    state["v_codes"] = pack4(nearest(Tlin, vt * rcp(M)))
    return w_new.astype(F32)


def sgdm4_step(w, g, state: dict, *, lr, beta, true_division=False):
    """Alg. 2 (compressed SGDM) on one tensor: m = beta m + g ; w = w - lr m ; compress m (B/DE)."""
    numel = state["rows"] * state["cols"]
    w = np.asarray(w, F32).ravel()
    g = np.asarray(g, F32).ravel()
    lr, beta = F32(lr), F32(beta)
    Tde = de_map(4, True)
    if state["kind"] == "fp32":
        m = state["m32"]
    else:
        m = dequantize_block(unpack4(state["m_codes"], numel), state["m_block"], Tde, state["m_scale"])
    mt = beta * m + g
    w_new = w - lr * mt
    if state["kind"] == "fp32":
        state["m32"] = mt
    else:
        qm, state["m_scale"] = quantize_block(mt, state["m_block"], Tde, true_division=true_division)
        state["m_codes"] = pack4(qm)
    return w_new.astype(F32)


def adamw4_factor_step(w, g, state: dict, *, lr, beta1, beta2, eps, weight_decay, step):
    """Factorized second moment (Sec. 4.3, Adafactor's rank-1 reconstruction) with a 4-bit first moment.

    state: {"rows", "cols", "m_block", "m_codes", "m_scale", "R", "C"}; returns the new w (flat float32).
    """
    rows, cols = state["rows"], state["cols"]
    numel = rows * cols
    w = np.asarray(w, F32).ravel()
    g = np.asarray(g, F32).reshape(rows, cols)
    lr, beta1, beta2, eps, wd = F32(lr), F32(beta1), F32(beta2), F32(eps), F32(weight_decay)
    Tde = de_map(4, True)
    m = dequantize_block(unpack4(state["m_codes"], numel), state["m_block"], Tde, state["m_scale"])
    omb1, omb2 = F32(1.0) - beta1, F32(1.0) - beta2
    bc1 = F32(1.0 - float(beta1) ** step)
    bc2 = F32(1.0 - float(beta2) ** step)
    gg = (g * g).astype(np.float64)
    rs = gg.sum(axis=1).astype(F32)
    cs = gg.sum(axis=0).astype(F32)
    R = beta2 * state["R"] + omb2 * rs
    Cc = beta2 * state["C"] + omb2 * cs
    total = F32(R.astype(np.float64).sum())
    rS = rcp(np.array([total], F32))[0]
    vt = ((R * rS)[:, None] * Cc[None, :]).astype(F32).ravel()
    mt = beta1 * m + omb1 * g.ravel()
    upd = lr * ((mt / bc1) / (np.sqrt(vt / bc2) + eps))
    w_new = w * (F32(1.0) - lr * wd) - upd
    qm, state["m_scale"] = quantize_block(mt, state["m_block"], Tde)
    state["m_codes"] = pack4(qm)
    state["R"], state["C"] = R.astype(F32), Cc.astype(F32)
    return w_new.astype(F32)
