"""Host-only checks of the C-ABI library: it loads without a GPU, exports every declared symbol,
sizes the arena, and rejects bad arguments before touching CUDA."""
import ctypes as C
import os
import re

import pytest

from paper_2309_01507_b200 import build as lib_build
from paper_2309_01507_b200 import lpmm, workloads

lib_build.build()      # nvcc cross-compiles without a GPU; a no-op when the library is newer than its sources

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "lpmm.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(lpmm_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    declared = _declared_symbols()
    assert set(declared) == set(lpmm.EXPORTS)
    L = lpmm.lib()
    for name in declared:
        assert hasattr(L, name), name


def test_status_strings():
    L = lpmm.lib()
    for code in (0, -1, -2, -3, -4, -5):
        assert L.lpmm_status_string(code)
    assert L.lpmm_status_string(0) == b"ok"


def test_state_bytes_accounts_for_every_buffer():
    cfg = lpmm.default_config()
    for wl in (workloads.single_matrix(), workloads.transformer_base(), workloads.roberta_large(), workloads.llama_7b()):
        nbytes = lpmm.state_bytes(cfg, wl.tensors)
        need = 0
        for t in wl.tensors:
            quant = t.force_quant or t.numel > 4096
            if not quant:
                need += 8 * t.numel
            else:
                need += 2 * ((t.numel + 1) // 2) + 4 * ((t.numel + 127) // 128)
                if t.ndim == 1 or t.rows == 1 or t.cols == 1:
                    need += 4 * ((t.numel + 127) // 128)
                else:
                    need += 3 * 4 * (t.rows + t.cols)       # two rank-1 scale buffers + their reciprocals
        assert nbytes >= need
        assert nbytes <= need * 1.02 + 600 * 1024            # alignment padding and tables only
    # 4-bit states take about 1/8 of fp32 states (two moments): 1 byte + scales vs 8 bytes per element
    wl = workloads.llama_7b()
    assert lpmm.state_bytes(cfg, wl.tensors) < 0.14 * 8 * wl.numel


def test_bad_configurations_are_rejected_on_the_host():
    L = lpmm.lib()
    out = C.c_size_t()
    shapes = lpmm.make_shapes([(64, 128, 2, 0)])
    cfg = lpmm.default_config()
    assert L.lpmm_state_bytes(None, shapes, 1, C.byref(out)) == lpmm.ERR_INVALID_ARG
    assert L.lpmm_state_bytes(C.byref(cfg), shapes, 0, C.byref(out)) == lpmm.ERR_INVALID_ARG
    assert L.lpmm_state_bytes(C.byref(cfg), shapes, 1, None) == lpmm.ERR_INVALID_ARG
    for field, value, want in (("bits", 8, lpmm.ERR_UNSUPPORTED), ("m_block", 64, lpmm.ERR_UNSUPPORTED), ("v_block", 2048, lpmm.ERR_UNSUPPORTED),
                               ("v_mode", 7, lpmm.ERR_INVALID_ARG), ("min_quant_numel", -1, lpmm.ERR_INVALID_ARG)):
        bad = lpmm.default_config()
        setattr(bad, field, value)
        assert L.lpmm_state_bytes(C.byref(bad), shapes, 1, C.byref(out)) == want
    for shp, want in (((0, 4, 2, 0), lpmm.ERR_INVALID_ARG), ((4, 4, 3, 0), lpmm.ERR_INVALID_ARG),   # ndim 3 without extents
                      ((4, 4, 5, 0), lpmm.ERR_UNSUPPORTED),
                      ((4, 4, 1, 0), lpmm.ERR_INVALID_ARG), ((4, 4, 2, 3), lpmm.ERR_INVALID_ARG),
                      ((1 << 39, 1 << 39, 2, 0), lpmm.ERR_INVALID_ARG)):
        assert L.lpmm_state_bytes(C.byref(cfg), lpmm.make_shapes([shp]), 1, C.byref(out)) == want
    # three and four axes (Alg. 4 in general form): extents must restate rows and cols
    nd = lpmm.nd_shape((6, 10, 200))
    assert L.lpmm_state_bytes(C.byref(cfg), lpmm.make_shapes([nd]), 1, C.byref(out)) == lpmm.OK
    assert out.value >= 2 * (12000 // 2) + 4 * (12000 // 128) + 3 * 4 * (6 + 10 + 200)
    bad = lpmm.nd_shape((6, 10, 200))
    bad.rows = 61
    assert L.lpmm_state_bytes(C.byref(cfg), lpmm.make_shapes([bad]), 1, C.byref(out)) == lpmm.ERR_INVALID_ARG
    fact = lpmm.default_config(v_mode=lpmm.V_FACTORED)
    assert L.lpmm_state_bytes(C.byref(fact), lpmm.make_shapes([nd]), 1, C.byref(out)) == lpmm.ERR_UNSUPPORTED
    assert L.lpmm_state_view_axis(None, 0, 0, None, None) == lpmm.ERR_INVALID_ARG
    h = C.c_void_p()
    assert L.lpmm_state_init(C.byref(cfg), shapes, 1, None, 1 << 20, C.byref(h), None) == lpmm.ERR_INVALID_ARG
    assert L.lpmm_state_init(C.byref(cfg), shapes, 1, 0x1010, 1 << 20, C.byref(h), None) == lpmm.ERR_ALIGNMENT
    assert L.lpmm_state_init(C.byref(cfg), shapes, 1, 0x1000, 16, C.byref(h), None) == lpmm.ERR_ARENA_TOO_SMALL
    assert L.lpmm_adamw4_step(None, None, None, 0, 1e-3, 0.9, 0.999, 1e-8, 0.0, 1, None) == lpmm.ERR_INVALID_ARG
    assert L.lpmm_quantize(None, 4, 4, 0, 0, 128, 0, None, None, None, None) == lpmm.ERR_INVALID_ARG
    assert L.lpmm_quantize(0x1000, 4, 4, 0, 0, 64, 0, 0x1000, 0x1000, None, None) == lpmm.ERR_UNSUPPORTED
    assert L.lpmm_quantize(0x1000, 4, 4, 1, 0, 128, 0, 0x1000, 0x1000, 0x1000, None) == lpmm.ERR_UNSUPPORTED
    assert L.lpmm_dequantize(0x1000, 0x1000, None, 4, 4, 1, 1, 128, 0x1000, None) == lpmm.ERR_INVALID_ARG
    L.lpmm_state_destroy(None)


def test_schedule_and_tuning_fields_are_validated_and_sized_on_the_host():
    L = lpmm.lib()
    out = C.c_size_t()
    shapes = lpmm.make_shapes([(1024, 4096, 2, 0), (4096, 1, 1, 1)])
    for field, value, want in (("schedule", 9, lpmm.ERR_INVALID_ARG), ("tile_elems", 3000, lpmm.ERR_INVALID_ARG),
                               ("tile_elems", 1024, lpmm.ERR_INVALID_ARG), ("tile_elems_maxima", 1 << 23, lpmm.ERR_INVALID_ARG),
                               ("l2_keep_mbytes", -1, lpmm.ERR_INVALID_ARG), ("lead_melems", -1, lpmm.ERR_INVALID_ARG),
                               ("gap_items", -5, lpmm.ERR_INVALID_ARG), ("no_l2_hints", 2, lpmm.ERR_INVALID_ARG),
                               ("overlap_groups", -1, lpmm.ERR_INVALID_ARG)):
        bad = lpmm.default_config()
        setattr(bad, field, value)
        assert L.lpmm_state_bytes(C.byref(bad), shapes, 2, C.byref(out)) == want, field
    # the fused schedule needs the default quantizers
    for kw in (dict(v_mode=lpmm.V_BLOCK), dict(v_mode=lpmm.V_FACTORED), dict(m_block=2048)):
        cfg = lpmm.default_config(schedule=lpmm.SCHEDULE_FUSED, **kw)
        assert L.lpmm_state_bytes(C.byref(cfg), shapes, 2, C.byref(out)) == lpmm.ERR_UNSUPPORTED
    # its work list lies behind the states: a fused arena is a two-pass arena plus 8 bytes per tile
    two = lpmm.state_bytes(lpmm.default_config(schedule=lpmm.SCHEDULE_TWO_PASS), shapes)
    fused = lpmm.state_bytes(lpmm.default_config(schedule=lpmm.SCHEDULE_FUSED), shapes)
    auto = lpmm.state_bytes(lpmm.default_config(), shapes)
    assert two < fused <= two + 8 * 2 * (1024 * 4096 // 2048 + 8) + 512 and auto == fused      # 4.2 M elements: AUTO = fused
    big = workloads.llama_7b().tensors
    assert lpmm.state_bytes(lpmm.default_config(), big) == lpmm.state_bytes(lpmm.default_config(schedule=lpmm.SCHEDULE_TWO_PASS), big)
    # smaller tiles, longer list
    assert lpmm.state_bytes(lpmm.default_config(schedule=lpmm.SCHEDULE_FUSED, tile_elems=32768, tile_elems_maxima=65536), big) > \
        lpmm.state_bytes(lpmm.default_config(schedule=lpmm.SCHEDULE_FUSED), big)
    assert L.lpmm_state_selftest_wait(None, None, None, None) == lpmm.ERR_INVALID_ARG
    assert L.lpmm_state_wait_stats(None, None, None, None) == lpmm.ERR_INVALID_ARG
    assert L.lpmm_state_check_guards(None, None, None, None) == lpmm.ERR_INVALID_ARG
    assert L.lpmm_build_is_checking() == 0
    assert L.lpmm_state_schedule(None) == -1


def test_workload_shapes_match_the_named_architectures():
    assert len(workloads.transformer_base().tensors) == 181
    assert len(workloads.roberta_large().tensors) == 394
    assert len(workloads.llama_7b().tensors) == 291
    assert abs(workloads.transformer_base().numel - 60.5e6) < 0.3e6
    assert abs(workloads.roberta_large().numel - 355.4e6) < 0.3e6
    assert abs(workloads.llama_7b().numel - 6.738e9) < 0.005e9


def test_gradient_generator_is_seeded_and_structured():
    import torch
    spec = workloads.TensorSpec("t", 64, 256, 2)
    a = workloads.make_grad(spec, 0, 0, 1)
    b = workloads.make_grad(spec, 0, 0, 1)
    c = workloads.make_grad(spec, 0, 0, 2)
    assert torch.equal(a, b) and not torch.equal(a, c)
    ratio = (c.abs() > 0).float().mean()
    assert ratio > 0.99
    sp = workloads.TensorSpec("e", 1000, 64, 2, sparse_rows=0.9)
    g = workloads.make_grad(sp, 0, 1, 1)
    zero_rows = (g.abs().sum(dim=1) == 0).float().mean().item()
    assert 0.85 < zero_rows < 0.95
    assert workloads.make_grad(spec, 0, 0, 1, dtype=torch.bfloat16).dtype == torch.bfloat16
