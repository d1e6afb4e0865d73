"""Thin ctypes binding of include/lpmm.h (argument marshalling only; all arithmetic runs in the CUDA library).

PyTorch is used for device memory and streams. There is no CPU fallback: if liblpmm.so is missing
or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "liblpmm.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_ALIGNMENT, ERR_ARENA_TOO_SMALL, ERR_CUDA = 0, -1, -2, -3, -4, -5
ERR_TOO_LARGE = -6
NOALLOC_MAX_SCALES = 262144
F32, BF16 = 0, 1
NORM_BLOCK, NORM_RANK1 = 0, 1
MAP_DE_SIGNED, MAP_LINEAR_NOZERO = 0, 1
V_RANK1, V_BLOCK, V_FACTORED = 0, 1, 2
UPDATE_FAST, UPDATE_IEEE = 0, 1
SCHEDULE_AUTO, SCHEDULE_TWO_PASS, SCHEDULE_FUSED, SCHEDULE_OVERLAP = 0, 1, 2, 3
FORCE_QUANT, FORCE_FP32 = 1, 2
Q_GIVEN_SCALES = 1
KIND_FP32, KIND_BLOCK, KIND_RANK1, KIND_FACTORED = 0, 1, 2, 3

EXPORTS = ("lpmm_state_bytes", "lpmm_state_init", "lpmm_state_attach", "lpmm_adamw4_step", "lpmm_adamw4_step_bf16w",
           "lpmm_adamw4_step_host", "lpmm_stage_bytes", "lpmm_quantize", "lpmm_dequantize",
           "lpmm_quantize_rank1_noalloc", "lpmm_sgdm4_step",
           "lpmm_state_view", "lpmm_state_view_axis", "lpmm_state_phase", "lpmm_state_last_launches", "lpmm_state_destroy",
           "lpmm_state_profile", "lpmm_state_profile_read", "lpmm_state_device_status", "lpmm_state_selftest_wait",
           "lpmm_state_schedule", "lpmm_state_wait_stats", "lpmm_build_is_checking", "lpmm_state_check_guards",
           "lpmm_state_selftest_check",
           "lpmm_status_string", "lpmm_last_cuda_error")


MAX_NDIM = 4


class Shape(C.Structure):
    _fields_ = [("rows", C.c_int64), ("cols", C.c_int64), ("ndim", C.c_int32), ("flags", C.c_uint32),
                ("dims", C.c_int64 * MAX_NDIM)]


def nd_shape(dims, flags: int = 0) -> Shape:
    """Shape of a tensor with three or more axes (row-major extents): rows is the product of the leading ones."""
    dims = [int(d) for d in dims]
    rows = 1
    for d in dims[:-1]:
        rows *= d
    arr = (C.c_int64 * MAX_NDIM)(*(dims + [0] * (MAX_NDIM - len(dims)))) if len(dims) <= MAX_NDIM else (C.c_int64 * MAX_NDIM)()
    return Shape(rows, dims[-1], len(dims), flags, arr)


class Config(C.Structure):
    _fields_ = [("bits", C.c_int32), ("m_block", C.c_int32), ("v_block", C.c_int32), ("v_mode", C.c_int32),
                ("min_quant_numel", C.c_int64), ("update_math", C.c_int32), ("schedule", C.c_int32),
                ("tile_elems", C.c_int32), ("tile_elems_maxima", C.c_int32), ("l2_keep_mbytes", C.c_int32),
                ("lead_melems", C.c_int32), ("gap_items", C.c_int32), ("no_l2_hints", C.c_int32), ("overlap_groups", C.c_int32)]


def default_config(v_mode: int = V_RANK1, min_quant_numel: int = 4096, update_math: int = 0, m_block: int = 128,
                   schedule: int = 0, tile_elems: int = 0, tile_elems_maxima: int = 0, l2_keep_mbytes: int = 0,
                   lead_melems: int = 0, gap_items: int = 0, no_l2_hints: int = 0, overlap_groups: int = 0) -> Config:
    return Config(4, m_block, 128, v_mode, min_quant_numel, update_math, schedule, tile_elems, tile_elems_maxima,
                  l2_keep_mbytes, lead_melems, gap_items, no_l2_hints, overlap_groups)


class LpmmError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().lpmm_status_string(status).decode()
        if status == ERR_CUDA:
            msg += f" (cudaError {lib().lpmm_last_cuda_error()})"
        super().__init__(f"{where}: {msg} [{status}]")


_lib = None


def use_library(path: str) -> None:
    """Binds this module to another build of the library (e.g. the checking build liblpmm_debug.so). Call it before
    anything else in the process: states made by one build must not be handed to another."""
    global _lib, LIB_PATH
    LIB_PATH = path
    _lib = None


def lib():
    """Loads liblpmm.so; fails loudly if it has not been built (python -m paper_2309_01507_b200.build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python paper_2309_01507_b200/build.py`; "
                               "there is no CPU fallback")
        L = C.CDLL(LIB_PATH)
        vp, i32, i64, f32, u32 = C.c_void_p, C.c_int32, C.c_int64, C.c_float, C.c_uint32
        L.lpmm_state_bytes.argtypes = [C.POINTER(Config), C.POINTER(Shape), i32, C.POINTER(C.c_size_t)]
        L.lpmm_state_init.argtypes = [C.POINTER(Config), C.POINTER(Shape), i32, vp, C.c_size_t, C.POINTER(vp), vp]
        L.lpmm_state_attach.argtypes = [C.POINTER(Config), C.POINTER(Shape), i32, vp, C.c_size_t, i32, C.POINTER(vp), vp]
        L.lpmm_adamw4_step.argtypes = [vp, C.POINTER(vp), C.POINTER(vp), i32, f32, f32, f32, f32, f32, i64, vp]
        L.lpmm_adamw4_step_bf16w.argtypes = [vp, C.POINTER(vp), C.POINTER(vp), C.POINTER(vp), i32, f32, f32, f32, f32, f32, i64, vp]
        L.lpmm_adamw4_step_host.argtypes = [vp, C.POINTER(vp), C.POINTER(vp), i32, f32, f32, f32, f32, f32, i64,
                                            vp, vp, C.c_size_t, vp]
        L.lpmm_sgdm4_step.argtypes = [vp, C.POINTER(vp), C.POINTER(vp), i32, f32, f32, vp]
        L.lpmm_stage_bytes.argtypes = [vp, C.POINTER(C.c_size_t)]
        L.lpmm_quantize.argtypes = [vp, i64, i64, i32, i32, i32, u32, vp, vp, vp, vp]
        L.lpmm_dequantize.argtypes = [vp, vp, vp, i64, i64, i32, i32, i32, vp, vp]
        L.lpmm_quantize_rank1_noalloc.argtypes = [vp, i64, i64, vp, vp, vp, vp]
        L.lpmm_state_view.argtypes = [vp, i32, C.POINTER(i32)] + [C.POINTER(vp)] * 7
        L.lpmm_state_view_axis.argtypes = [vp, i32, i32, C.POINTER(vp), C.POINTER(i64)]
        L.lpmm_state_profile.argtypes = [vp, i32]
        L.lpmm_state_profile_read.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(C.c_double), C.POINTER(C.c_double),
                                              C.POINTER(i32)]
        L.lpmm_state_device_status.argtypes = [vp, C.POINTER(i32), vp]
        L.lpmm_state_selftest_wait.argtypes = [vp, C.POINTER(i32), C.POINTER(i32), vp]
        L.lpmm_state_schedule.argtypes = [vp]
        L.lpmm_state_wait_stats.argtypes = [vp, C.POINTER(i64), C.POINTER(i64), vp]
        L.lpmm_build_is_checking.argtypes = []
        L.lpmm_state_check_guards.argtypes = [vp, C.POINTER(i64), C.POINTER(i64), vp]
        L.lpmm_state_selftest_check.argtypes = [vp, C.POINTER(i32), vp]
        L.lpmm_state_phase.argtypes = [vp]
        L.lpmm_state_last_launches.argtypes = [vp]
        L.lpmm_state_destroy.argtypes = [vp]
        L.lpmm_state_destroy.restype = None
        L.lpmm_status_string.argtypes = [i32]
        L.lpmm_status_string.restype = C.c_char_p
        for name in EXPORTS:
            if name not in ("lpmm_state_destroy", "lpmm_status_string"):
                getattr(L, name).restype = i32
        _lib = L
    return _lib


def _check(status: int, where: str) -> None:
    if status != OK:
        raise LpmmError(status, where)


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream


def make_shapes(shapes) -> C.Array:
    """shapes: iterable of (rows, cols, ndim, flags) tuples or objects with those attributes."""
    items = []
    for s in shapes:
        if isinstance(s, Shape):
            items.append(s)
        elif isinstance(s, (tuple, list)):
            rows, cols, ndim = s[0], s[1], s[2]
            flags = s[3] if len(s) > 3 else 0
            items.append(Shape(rows, cols, ndim, flags))
        else:
            flags = FORCE_QUANT if getattr(s, "force_quant", False) else 0
            dims = getattr(s, "dims", None)
            if dims is not None and len(dims) >= 3:
                items.append(nd_shape(dims, flags))
            else:
                items.append(Shape(s.rows, s.cols, s.ndim, flags))
    return (Shape * len(items))(*items)


def state_bytes(config: Config, shapes) -> int:
    arr = make_shapes(shapes)
    out = C.c_size_t(0)
    _check(lib().lpmm_state_bytes(C.byref(config), arr, len(arr), C.byref(out)), "lpmm_state_bytes")
    return out.value


@dataclass
class State:
    handle: C.c_void_p
    arena: torch.Tensor
    shapes: C.Array
    config: Config
    n: int

    def __del__(self):
        try:
            if self.handle:
                lib().lpmm_state_destroy(self.handle)
                self.handle = None
        except Exception:
            pass

    @property
    def phase(self) -> int:
        return lib().lpmm_state_phase(self.handle)

    @property
    def last_launches(self) -> int:
        return lib().lpmm_state_last_launches(self.handle)

    @property
    def schedule(self) -> int:
        return lib().lpmm_state_schedule(self.handle)


def state_init(config: Config, shapes, device="cuda", stream=None) -> State:
    arr = make_shapes(shapes)
    nbytes = state_bytes(config, arr)
    arena = torch.empty(nbytes, dtype=torch.uint8, device=device)
    h = C.c_void_p()
    with torch.cuda.device(arena.device):
        _check(lib().lpmm_state_init(C.byref(config), arr, len(arr), arena.data_ptr(), nbytes, C.byref(h),
                                     _stream_ptr(stream)), "lpmm_state_init")
    return State(h, arena, arr, config, len(arr))


def state_attach(config: Config, shapes, arena: torch.Tensor, phase: int, stream=None) -> State:
    arr = make_shapes(shapes)
    h = C.c_void_p()
    with torch.cuda.device(arena.device):
        _check(lib().lpmm_state_attach(C.byref(config), arr, len(arr), arena.data_ptr(), arena.numel(), phase,
                                       C.byref(h), _stream_ptr(stream)), "lpmm_state_attach")
    return State(h, arena, arr, config, len(arr))


def _ptr_array(tensors):
    return (C.c_void_p * len(tensors))(*[t.data_ptr() for t in tensors])


def _grad_dtype(grads) -> int:
    dt = grads[0].dtype
    if any(g.dtype != dt for g in grads):
        raise ValueError("all gradients must share one dtype")
    if dt == torch.float32:
        return F32
    if dt == torch.bfloat16:
        return BF16
    raise ValueError(f"unsupported gradient dtype {dt}")


def adamw4_step(state: State, params, grads, *, lr, beta1, beta2, eps, weight_decay, step, stream=None,
                ptr_cache=None, params_bf16=None) -> None:
    """lpmm_adamw4_step: params (fp32, updated in place) and grads are lists of contiguous CUDA tensors.
    params_bf16 (optional list of bfloat16 tensors of the same sizes) receives a rounded copy of the new parameters
    (lpmm_adamw4_step_bf16w)."""
    if len(params) != state.n or len(grads) != state.n:
        raise ValueError("params/grads must have one tensor per state entry")
    if ptr_cache is None:
        for p in params:
            if p.dtype != torch.float32 or not p.is_contiguous() or not p.is_cuda:
                raise ValueError("parameters must be contiguous fp32 CUDA tensors")
        for g in grads:
            if not g.is_contiguous() or not g.is_cuda:
                raise ValueError("gradients must be contiguous CUDA tensors")
        pp, gp, gd = _ptr_array(params), _ptr_array(grads), _grad_dtype(grads)
    else:
        pp, gp, gd = ptr_cache
    with torch.cuda.device(state.arena.device):
        if params_bf16 is not None:
            if len(params_bf16) != state.n:
                raise ValueError("params_bf16 must have one tensor per state entry")
            for p, c in zip(params, params_bf16):
                if c.dtype != torch.bfloat16 or not c.is_contiguous() or not c.is_cuda or c.numel() != p.numel():
                    raise ValueError("bfloat16 copies must be contiguous CUDA tensors of the parameters' sizes")
            _check(lib().lpmm_adamw4_step_bf16w(state.handle, pp, _ptr_array(params_bf16), gp, gd, lr, beta1, beta2, eps,
                                                weight_decay, step, _stream_ptr(stream)), "lpmm_adamw4_step_bf16w")
            return
        _check(lib().lpmm_adamw4_step(state.handle, pp, gp, gd, lr, beta1, beta2, eps, weight_decay, step,
                                      _stream_ptr(stream)), "lpmm_adamw4_step")


def sgdm4_step(state: State, params, grads, *, lr, beta, stream=None) -> None:
    """lpmm_sgdm4_step: compressed SGDM (Alg. 2) on lists of contiguous CUDA tensors."""
    if len(params) != state.n or len(grads) != state.n:
        raise ValueError("params/grads must have one tensor per state entry")
    with torch.cuda.device(state.arena.device):
        _check(lib().lpmm_sgdm4_step(state.handle, _ptr_array(params), _ptr_array(grads), _grad_dtype(grads), lr, beta,
                                     _stream_ptr(stream)), "lpmm_sgdm4_step")


def make_ptr_cache(params, grads):
    """Pre-marshalled pointer arrays for repeated steps on the same buffers (skips per-call Python work)."""
    return _ptr_array(params), _ptr_array(grads), _grad_dtype(grads)


def profile(state: State, enable: bool) -> None:
    _check(lib().lpmm_state_profile(state.handle, int(enable)), "lpmm_state_profile")


def profile_read(state: State) -> dict:
    """Summed kernel durations (ms) over the steps recorded since the last read."""
    p1, rc, p2, n = C.c_double(), C.c_double(), C.c_double(), C.c_int32()
    _check(lib().lpmm_state_profile_read(state.handle, C.byref(p1), C.byref(rc), C.byref(p2), C.byref(n)),
           "lpmm_state_profile_read")
    return {"pass1_ms": p1.value, "rcp_ms": rc.value, "pass2_ms": p2.value, "steps": n.value}


def device_status(state: State, stream=None) -> int:
    """Device-side error word of the state (0 = ok); synchronizes the stream."""
    out = C.c_int32()
    _check(lib().lpmm_state_device_status(state.handle, C.byref(out), _stream_ptr(stream)), "lpmm_state_device_status")
    return out.value


def selftest_wait(state: State, stream=None):
    """lpmm_state_selftest_wait: (CTAs that gave up, status word they left)."""
    n, w = C.c_int32(), C.c_int32()
    with torch.cuda.device(state.arena.device):
        _check(lib().lpmm_state_selftest_wait(state.handle, C.byref(n), C.byref(w), _stream_ptr(stream)),
               "lpmm_state_selftest_wait")
    return n.value, w.value


def wait_stats(state: State, stream=None):
    """lpmm_state_wait_stats: (waits that had to poll, their summed nanoseconds) since the last call."""
    n, ns = C.c_int64(), C.c_int64()
    with torch.cuda.device(state.arena.device):
        _check(lib().lpmm_state_wait_stats(state.handle, C.byref(n), C.byref(ns), _stream_ptr(stream)), "lpmm_state_wait_stats")
    return n.value, ns.value


def check_guards(state: State, stream=None):
    """lpmm_state_check_guards (checking build only): (guard zones, damaged bytes)."""
    z, b = C.c_int64(), C.c_int64()
    with torch.cuda.device(state.arena.device):
        _check(lib().lpmm_state_check_guards(state.handle, C.byref(z), C.byref(b), _stream_ptr(stream)), "lpmm_state_check_guards")
    return z.value, b.value


def selftest_check(state: State, stream=None) -> int:
    """lpmm_state_selftest_check (checking build only): the status word a failing index check leaves."""
    w = C.c_int32()
    with torch.cuda.device(state.arena.device):
        _check(lib().lpmm_state_selftest_check(state.handle, C.byref(w), _stream_ptr(stream)), "lpmm_state_selftest_check")
    return w.value


def stage_bytes(state: State) -> int:
    out = C.c_size_t(0)
    _check(lib().lpmm_stage_bytes(state.handle, C.byref(out)), "lpmm_stage_bytes")
    return out.value


def adamw4_step_host(state: State, h_params, h_grads, d_param_stage, d_grad_stage, *, lr, beta1, beta2, eps,
                     weight_decay, step, stream=None) -> None:
    """lpmm_adamw4_step_host: params/grads are HOST tensors (pinned for asynchronous copies)."""
    gd = _grad_dtype(h_grads)
    torch.cuda.set_device(state.arena.device)
    _check(lib().lpmm_adamw4_step_host(state.handle, _ptr_array(h_params), _ptr_array(h_grads), gd, lr, beta1,
                                       beta2, eps, weight_decay, step, d_param_stage.data_ptr(),
                                       d_grad_stage.data_ptr(), min(d_param_stage.numel() * d_param_stage.element_size(),
                                                                    d_grad_stage.numel() * d_grad_stage.element_size()),
                                       _stream_ptr(stream)), "lpmm_adamw4_step_host")


def quantize(x: torch.Tensor, norm: int, map_: int, block: int = 128, scales=None, stream=None):
    """lpmm_quantize on a contiguous fp32 CUDA tensor (1-D or 2-D). Returns (codes, scale0, scale1)."""
    if x.dtype != torch.float32 or not x.is_contiguous() or not x.is_cuda or x.dim() not in (1, 2):
        raise ValueError("x must be a contiguous fp32 CUDA tensor with 1 or 2 dimensions")
    rows, cols = (x.shape[0], 1) if x.dim() == 1 else x.shape
    numel = rows * cols
    codes = torch.empty((numel + 1) // 2, dtype=torch.uint8, device=x.device)
    flags = 0
    if scales is not None:
        s0, s1 = scales
        flags = Q_GIVEN_SCALES
    elif norm == NORM_RANK1:
        s0 = torch.empty(rows, dtype=torch.float32, device=x.device)
        s1 = torch.empty(cols, dtype=torch.float32, device=x.device)
    else:
        s0 = torch.empty((numel + block - 1) // max(block, 1), dtype=torch.float32, device=x.device)
        s1 = None
    with torch.cuda.device(x.device):
        _check(lib().lpmm_quantize(x.data_ptr(), rows, cols, norm, map_, block, flags, codes.data_ptr(),
                                   s0.data_ptr(), None if s1 is None else s1.data_ptr(), _stream_ptr(stream)),
               "lpmm_quantize")
    return codes, s0, s1


def quantize_rank1_noalloc(x: torch.Tensor, codes: torch.Tensor, r: torch.Tensor, c: torch.Tensor, stream=None) -> None:
    """lpmm_quantize_rank1_noalloc: the caller supplies the input and all three outputs; nothing is allocated.

    The C entry point only sees raw pointers, so the buffers are checked here: x a contiguous 2-D fp32 CUDA tensor,
    codes uint8 with at least ceil(rows*cols/2) bytes, r and c contiguous fp32 with at least rows / cols elements, all
    on x's device. Anything else raises ValueError before the library is called."""
    if x.dim() != 2 or x.dtype != torch.float32 or not x.is_cuda or not x.is_contiguous():
        raise ValueError("x must be a contiguous 2-D fp32 CUDA tensor")
    rows, cols = x.shape
    if rows <= 0 or cols <= 0:
        raise ValueError("x must not be empty")
    for name, t, dtype, need in (("codes", codes, torch.uint8, (rows * cols + 1) // 2), ("r", r, torch.float32, rows),
                                 ("c", c, torch.float32, cols)):
        if t.dtype != dtype or not t.is_cuda or not t.is_contiguous() or t.device != x.device:
            raise ValueError(f"{name} must be a contiguous {dtype} CUDA tensor on x's device")
        if t.numel() < need:
            raise ValueError(f"{name} holds {t.numel()} elements, {need} are needed")
    with torch.cuda.device(x.device):
        _check(lib().lpmm_quantize_rank1_noalloc(x.data_ptr(), rows, cols, codes.data_ptr(), r.data_ptr(),
                                                 c.data_ptr(), _stream_ptr(stream)), "lpmm_quantize_rank1_noalloc")


def dequantize(codes: torch.Tensor, s0: torch.Tensor, s1, rows: int, cols: int, norm: int, map_: int,
               block: int = 128, stream=None) -> torch.Tensor:
    out = torch.empty(rows * cols, dtype=torch.float32, device=codes.device)
    with torch.cuda.device(codes.device):
        _check(lib().lpmm_dequantize(codes.data_ptr(), s0.data_ptr(), None if s1 is None else s1.data_ptr(),
                                     rows, cols, norm, map_, block, out.data_ptr(), _stream_ptr(stream)),
               "lpmm_dequantize")
    return out.reshape(rows, cols) if cols > 1 else out


def state_view(state: State, i: int) -> dict:
    """Current state of tensor i as torch views into the arena (no copies)."""
    kind = C.c_int32()
    ptrs = [C.c_void_p() for _ in range(7)]
    _check(lib().lpmm_state_view(state.handle, i, C.byref(kind), *[C.byref(p) for p in ptrs]), "lpmm_state_view")
    sh = state.shapes[i]
    numel = sh.rows * sh.cols
    base = state.arena.data_ptr()

    def view(p, nbytes, dtype):
        if not p.value:
            return None
        off = p.value - base
        return state.arena[off:off + nbytes].view(dtype)

    nblk_m = (numel + state.config.m_block - 1) // state.config.m_block
    nblk_v = (numel + state.config.v_block - 1) // state.config.v_block
    k = kind.value
    return {
        "kind": k,
        "m_codes": view(ptrs[0], (numel + 1) // 2, torch.uint8),
        "m_scale": view(ptrs[1], 4 * nblk_m, torch.float32),
        "v_codes": view(ptrs[2], (numel + 1) // 2, torch.uint8),
        # rank-1: the first axis' maxima (a matrix: r; three or more axes: see state_view_axis for the others)
        "v_s0": view(ptrs[3], 4 * ((sh.dims[0] if sh.ndim >= 3 else sh.rows) if k in (KIND_RANK1, KIND_FACTORED) else nblk_v),
                     torch.float32),
        "v_s1": view(ptrs[4], 4 * sh.cols, torch.float32),
        "m32": view(ptrs[5], 4 * numel, torch.float32),
        "v32": view(ptrs[6], 4 * numel, torch.float32),
    }


def state_view_axis(state: State, tensor: int, axis: int) -> torch.Tensor:
    """Per-axis maxima of a rank-1 tensor's second moment (Alg. 4), as a view into the arena."""
    p = C.c_void_p()
    n = C.c_int64()
    _check(lib().lpmm_state_view_axis(state.handle, tensor, axis, C.byref(p), C.byref(n)), "lpmm_state_view_axis")
    off = p.value - state.arena.data_ptr()
    return state.arena[off:off + 4 * n.value].view(torch.float32)
