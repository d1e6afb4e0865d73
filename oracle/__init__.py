"""ctypes front-end of the C oracle (oracle/lpmm_oracle.c).

TEST INFRASTRUCTURE ONLY: the test-suite, the smoke check and the benchmark's CPU-baseline leg
may import this package; the CUDA library and its Python binding never do.

All arrays are NumPy, C-contiguous; floats are float32, codes are uint8.
"""
from __future__ import annotations

import ctypes as C
from dataclasses import dataclass, field

import numpy as np

from . import build as _build

FP32, BLOCK, RANK1 = 0, 1, 2

_lib = None


class _Hyper(C.Structure):
    _fields_ = [("lr", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float),
                ("weight_decay", C.c_float), ("step", C.c_int64), ("true_division", C.c_int32)]


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(_build.build())
        _lib.lpmm_oracle_de_fraction.restype = C.c_double
        _lib.lpmm_oracle_de_fraction.argtypes = [C.c_int, C.c_int]
        _lib.lpmm_oracle_rcp.restype = C.c_float
        _lib.lpmm_oracle_rcp.argtypes = [C.c_float]
        _lib.lpmm_oracle_nearest.argtypes = [C.c_void_p, C.c_int, C.c_float]
        _lib.lpmm_oracle_kind.argtypes = [C.c_int64, C.c_int64, C.c_int, C.c_int64, C.c_int]
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def _u8(a):
    return np.ascontiguousarray(a, dtype=np.uint8)


def threads() -> int:
    return int(lib().lpmm_oracle_threads())


def set_threads(n: int) -> None:
    lib().lpmm_oracle_set_threads(C.c_int(int(n)))


def linear_map(bits: int = 4) -> np.ndarray:
    T = np.zeros(1 << bits, np.float32)
    lib().lpmm_oracle_linear_map(C.c_int(bits), _p(T))
    return T


def de_map(bits: int = 4, signed: bool = True, drop_zero: bool = False) -> np.ndarray:
    T = np.zeros(1 << bits, np.float32)
    n = lib().lpmm_oracle_de_map(C.c_int(bits), C.c_int(int(signed)), C.c_int(int(drop_zero)), _p(T))
    return T[:n].copy()


def de_fraction(F: int, k: int) -> float:
    return float(lib().lpmm_oracle_de_fraction(F, k))


def nearest(T: np.ndarray, n: float) -> int:
    T = _f32(T)
    return int(lib().lpmm_oracle_nearest(_p(T), len(T), C.c_float(float(n))))


def rcp(s: float) -> float:
    return float(lib().lpmm_oracle_rcp(C.c_float(float(s))))


def block_scales(x: np.ndarray, B: int) -> np.ndarray:
    x = _f32(x).ravel()
    out = np.zeros((x.size + B - 1) // B, np.float32)
    lib().lpmm_oracle_block_scales(_p(x), C.c_int64(x.size), C.c_int64(B), _p(out))
    return out


def rank1_stats(x: np.ndarray) -> list[np.ndarray]:
    x = _f32(x)
    dims = np.asarray(x.shape, np.int64)
    mu = np.zeros(int(dims.sum()), np.float32)
    lib().lpmm_oracle_rank1_stats(_p(x), C.c_int(x.ndim), _p(dims), _p(mu))
    out, off = [], 0
    for d in x.shape:
        out.append(mu[off:off + d].copy())
        off += d
    return out


def rank1_scale_field(shape, stats: list[np.ndarray]) -> np.ndarray:
    dims = np.asarray(shape, np.int64)
    mu = _f32(np.concatenate(stats))
    M = np.zeros(int(np.prod(dims)), np.float32)
    lib().lpmm_oracle_rank1_scale_field(C.c_int(len(shape)), _p(dims), _p(mu), _p(M))
    return M.reshape(shape)


def map_codes(x, scale_of_elem, T, true_division=False) -> np.ndarray:
    x, s, T = _f32(x), _f32(scale_of_elem), _f32(T)
    codes = np.zeros(x.size, np.uint8)
    lib().lpmm_oracle_map_codes(_p(x), _p(s), C.c_int64(x.size), _p(T), C.c_int(len(T)),
                                C.c_int(int(true_division)), _p(codes))
    return codes.reshape(x.shape)


def quantize_block(x, B, T, scale=None, true_division=False):
    x, T = _f32(x).ravel(), _f32(T)
    given = scale is not None
    scale = _f32(scale).copy() if given else np.zeros((x.size + B - 1) // B, np.float32)
    codes = np.zeros(x.size, np.uint8)
    lib().lpmm_oracle_quantize_block(_p(x), C.c_int64(x.size), C.c_int64(B), _p(T), C.c_int(len(T)),
                                     C.c_int(int(given)), C.c_int(int(true_division)), _p(scale), _p(codes))
    return codes, scale


def quantize_rank1(x, T, r=None, c=None, true_division=False):
    x, T = _f32(x), _f32(T)
    rows, cols = x.shape
    given = r is not None
    r = _f32(r).copy() if given else np.zeros(rows, np.float32)
    c = _f32(c).copy() if given else np.zeros(cols, np.float32)
    codes = np.zeros(x.size, np.uint8)
    lib().lpmm_oracle_quantize_rank1(_p(x), C.c_int64(rows), C.c_int64(cols), _p(T), C.c_int(len(T)),
                                     C.c_int(int(given)), C.c_int(int(true_division)), _p(r), _p(c), _p(codes))
    return codes.reshape(rows, cols), r, c


def dequantize_block(codes, B, T, scale) -> np.ndarray:
    codes, T, scale = _u8(codes).ravel(), _f32(T), _f32(scale)
    out = np.zeros(codes.size, np.float32)
    lib().lpmm_oracle_dequantize_block(_p(codes), C.c_int64(codes.size), C.c_int64(B), _p(T), _p(scale), _p(out))
    return out


def dequantize_rank1(codes, T, r, c) -> np.ndarray:
    codes, T, r, c = _u8(codes), _f32(T), _f32(r), _f32(c)
    rows, cols = codes.shape
    out = np.zeros(codes.size, np.float32)
    lib().lpmm_oracle_dequantize_rank1(_p(codes), C.c_int64(rows), C.c_int64(cols), _p(T), _p(r), _p(c), _p(out))
    return out.reshape(rows, cols)


def pack4(codes) -> np.ndarray:
    codes = _u8(codes).ravel()
    out = np.zeros((codes.size + 1) // 2, np.uint8)
    lib().lpmm_oracle_pack4(_p(codes), C.c_int64(codes.size), _p(out))
    return out


def unpack4(packed, numel: int) -> np.ndarray:
    packed = _u8(packed).ravel()
    out = np.zeros(numel, np.uint8)
    lib().lpmm_oracle_unpack4(_p(packed), C.c_int64(numel), _p(out))
    return out


def bf16_bits_to_f32(bits) -> np.ndarray:
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    out = np.zeros(bits.size, np.float32)
    lib().lpmm_oracle_bf16_to_f32(_p(bits), C.c_int64(bits.size), _p(out))
    return out.reshape(bits.shape)


def f32_to_bf16_bits(x) -> np.ndarray:
    x = _f32(x)
    out = np.zeros(x.size, np.uint16)
    lib().lpmm_oracle_f32_to_bf16(_p(x), C.c_int64(x.size), _p(out))
    return out.reshape(x.shape)


def kind_of(rows: int, cols: int, ndim: int, min_quant_numel: int = 4096, force: int = 0) -> int:
    return int(lib().lpmm_oracle_kind(rows, cols, ndim, min_quant_numel, force))


@dataclass
class TensorState:
    """Compressed (or fp32) optimizer state of one tensor, in the packed layout."""
    rows: int
    cols: int
    kind: int
    m_block: int = 128
    v_block: int = 128
    m_codes: np.ndarray = field(default=None)
    m_scale: np.ndarray = field(default=None)
    v_codes: np.ndarray = field(default=None)
    v_s0: np.ndarray = field(default=None)
    v_s1: np.ndarray = field(default=None)
    m32: np.ndarray = field(default=None)
    v32: np.ndarray = field(default=None)

    @property
    def numel(self) -> int:
        return self.rows * self.cols


def state_init(rows: int, cols: int, kind: int, m_block: int = 128, v_block: int = 128) -> TensorState:
    numel = rows * cols
    st = TensorState(rows, cols, kind, m_block, v_block)
    if kind == FP32:
        st.m32 = np.empty(numel, np.float32)
        st.v32 = np.empty(numel, np.float32)
    else:
        nbytes = (numel + 1) // 2
        st.m_codes = np.empty(nbytes, np.uint8)
        st.v_codes = np.empty(nbytes, np.uint8)
        st.m_scale = np.empty((numel + m_block - 1) // m_block, np.float32)
        if kind == BLOCK:
            st.v_s0 = np.empty((numel + v_block - 1) // v_block, np.float32)
        else:
            st.v_s0 = np.empty(rows, np.float32)
            st.v_s1 = np.empty(cols, np.float32)
    lib().lpmm_oracle_state_init(C.c_int64(rows), C.c_int64(cols), C.c_int(kind), C.c_int64(m_block),
                                 C.c_int64(v_block), _p(st.m_codes), _p(st.m_scale), _p(st.v_codes),
                                 _p(st.v_s0), _p(st.v_s1), _p(st.m32), _p(st.v32))
    return st


def adamw4_step(w: np.ndarray, g: np.ndarray, st: TensorState, *, lr, beta1, beta2, eps, weight_decay,
                step: int, true_division: bool = False) -> None:
    """One compressed AdamW step on one tensor; w and the state are updated in place."""
    assert w.dtype == np.float32 and w.flags.c_contiguous and w.size == st.numel
    g = _f32(g)
    assert g.size == st.numel
    h = _Hyper(lr, beta1, beta2, eps, weight_decay, step, int(true_division))
    rc = lib().lpmm_oracle_adamw4_step(_p(w), _p(g), C.c_int64(st.rows), C.c_int64(st.cols), C.c_int(st.kind),
                                       C.c_int64(st.m_block), C.c_int64(st.v_block),
                                       _p(st.m_codes), _p(st.m_scale), _p(st.v_codes), _p(st.v_s0), _p(st.v_s1),
                                       _p(st.m32), _p(st.v32), C.byref(h))
    if rc != 0:
        raise ValueError("lpmm_oracle_adamw4_step rejected its arguments")


def adamw4_step_nd(w: np.ndarray, g: np.ndarray, dims, m_block: int, m_codes: np.ndarray, m_scale: np.ndarray,
                   v_codes: np.ndarray, mu_flat: np.ndarray, *, lr, beta1, beta2, eps, weight_decay, step: int,
                   true_division: bool = False) -> None:
    """One compressed AdamW step on a tensor of any rank with the general rank-1 normalization of Alg. 4;
    w, the codes, m_scale and mu_flat (per-axis maxima, concatenated) are updated in place."""
    dims = np.asarray(dims, np.int64)
    numel = int(np.prod(dims))
    assert w.dtype == np.float32 and w.flags.c_contiguous and w.size == numel
    assert m_codes.dtype == np.uint8 and v_codes.dtype == np.uint8 and m_codes.size == (numel + 1) // 2 == v_codes.size
    assert m_scale.dtype == np.float32 and m_scale.size == (numel + m_block - 1) // m_block
    assert mu_flat.dtype == np.float32 and mu_flat.size == int(dims.sum())
    g = _f32(g)
    assert g.size == numel
    h = _Hyper(lr, beta1, beta2, eps, weight_decay, step, int(true_division))
    rc = lib().lpmm_oracle_adamw4_step_nd(_p(w), _p(g), C.c_int(len(dims)), _p(dims), C.c_int64(m_block), _p(m_codes),
                                          _p(m_scale), _p(v_codes), _p(mu_flat), C.byref(h))
    if rc != 0:
        raise ValueError("lpmm_oracle_adamw4_step_nd rejected its arguments")


def sgdm4_step(w: np.ndarray, g: np.ndarray, st: TensorState, *, lr, beta, true_division: bool = False) -> None:
    """One compressed SGDM step (Alg. 2) on one tensor; only the first-moment part of `st` is used."""
    assert w.dtype == np.float32 and w.flags.c_contiguous and w.size == st.numel
    g = _f32(g)
    rc = lib().lpmm_oracle_sgdm4_step(_p(w), _p(g), C.c_int64(st.numel), C.c_int(int(st.kind != FP32)),
                                      C.c_int64(st.m_block), _p(st.m_codes), _p(st.m_scale), _p(st.m32),
                                      C.c_float(lr), C.c_float(beta), C.c_int(int(true_division)))
    if rc != 0:
        raise ValueError("lpmm_oracle_sgdm4_step rejected its arguments")


def adamw4_factor_step(w: np.ndarray, g: np.ndarray, st: TensorState, R: np.ndarray, C_: np.ndarray, *, lr, beta1,
                       beta2, eps, weight_decay, step: int) -> None:
    """One step of the factorized-second-moment variant on a matrix; w, the m part of `st`, R and C_ change in place."""
    assert w.dtype == np.float32 and w.size == st.numel and R.dtype == np.float32 and C_.dtype == np.float32
    assert R.size == st.rows and C_.size == st.cols
    g = _f32(g)
    h = _Hyper(lr, beta1, beta2, eps, weight_decay, step, 0)
    rc = lib().lpmm_oracle_adamw4_factor_step(_p(w), _p(g), C.c_int64(st.rows), C.c_int64(st.cols), C.c_int64(st.m_block),
                                              _p(st.m_codes), _p(st.m_scale), _p(R), _p(C_), C.byref(h))
    if rc != 0:
        raise ValueError("lpmm_oracle_adamw4_factor_step rejected its arguments")
