"""Runs the shape zoo through the checking build of the library (liblpmm_debug.so) in a process of its own.

Started by tests/test_gpu_checking_build.py; prints one line 'OK ...' on success. The checking build stands in for a
memory checker: after every step the device status word must be 0 (no index check failed) and every guard zone behind
the arena's sub-buffers must still hold its pattern (no stray write crossed a sub-buffer's end)."""
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import torch

from paper_2309_01507_b200 import build as lib_build
from paper_2309_01507_b200 import lpmm, workloads
from paper_2309_01507_b200.workloads import TensorSpec


def mat(r, c, **kw):
    return TensorSpec(f"m{r}x{c}", r, c, 2, **kw)


def vec(n, **kw):
    return TensorSpec(f"v{n}", n, 1, 1, **kw)


def nd(*dims):
    rows = 1
    for d in dims[:-1]:
        rows *= d
    return TensorSpec("t" + "x".join(map(str, dims)), rows, dims[-1], len(dims), dims=tuple(dims))


def main():
    lpmm.use_library(lib_build.build(debug=True))
    assert lpmm.lib().lpmm_build_is_checking() == 1
    zoo = [mat(96, 256), mat(33, 77), mat(5, 1000), mat(130, 384), mat(64, 1024), mat(8, 2048), mat(1, 8192), mat(8192, 1),
           mat(300, 640), mat(257, 129), mat(70, 128), vec(50265), vec(4097), vec(4096), vec(4096, force_quant=True), vec(1),
           vec(300), mat(16, 16), mat(65, 64), vec(12345), nd(6, 10, 200), nd(3, 5, 7, 64), vec(196608), mat(1030, 4096)]
    tiled_only = [mat(96, 256), mat(64, 2048), mat(24, 4096), vec(50265), vec(300), mat(1030, 4096)]
    hyper = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01)
    cases = [("two_pass", lpmm.default_config(schedule=lpmm.SCHEDULE_TWO_PASS), zoo, torch.float32),
             ("fused", lpmm.default_config(schedule=lpmm.SCHEDULE_FUSED), zoo, torch.bfloat16),
             ("overlap", lpmm.default_config(schedule=lpmm.SCHEDULE_OVERLAP, overlap_groups=3), zoo, torch.float32),
             ("b2048", lpmm.default_config(m_block=2048), zoo, torch.bfloat16),
             ("block_v", lpmm.default_config(v_mode=lpmm.V_BLOCK), zoo[:20] + zoo[22:], torch.float32),
             ("block_v_b2048", lpmm.default_config(v_mode=lpmm.V_BLOCK, m_block=2048), tiled_only, torch.bfloat16),
             ("factored", lpmm.default_config(v_mode=lpmm.V_FACTORED), tiled_only, torch.float32)]
    zones_total = 0
    for name, cfg, specs, gdt in cases:
        params = [workloads.make_param(s, 21, i, device="cuda") for i, s in enumerate(specs)]
        state = lpmm.state_init(cfg, specs)
        for t in (1, 2, 3):
            grads = [workloads.make_grad(s, 21, i, t, device="cuda", dtype=gdt) for i, s in enumerate(specs)]
            lpmm.adamw4_step(state, params, grads, step=t, **hyper)
            if name in ("two_pass", "b2048") and t == 3:
                copies = [torch.empty(s.numel, dtype=torch.bfloat16, device="cuda") for s in specs]
                lpmm.adamw4_step(state, params, grads, step=4, params_bf16=copies, **hyper)
            assert lpmm.device_status(state) == 0, (name, t, hex(lpmm.device_status(state)))
            zones, damaged = lpmm.check_guards(state)
            assert zones > len(specs) and damaged == 0, (name, t, zones, damaged)
        if name in ("two_pass", "b2048"):        # the SGDM kernel on a state of its own
            st2 = lpmm.state_init(cfg, specs)
            lpmm.sgdm4_step(st2, params, grads, lr=0.01, beta=0.9)
            assert lpmm.device_status(st2) == 0 and lpmm.check_guards(st2)[1] == 0, name
        for p in params:
            assert torch.isfinite(p).all(), name
        zones_total += zones
    # the checkers themselves: a guard byte damaged from the host is found; a check that fails on purpose is reported
    state = lpmm.state_init(lpmm.default_config(), [mat(96, 256), vec(5000)])
    torch.cuda.synchronize()
    view = lpmm.state_view(state, 0)
    m_codes = view["m_codes"]
    off = m_codes.data_ptr() - state.arena.data_ptr() + ((m_codes.numel() + 255) // 256) * 256     # first byte behind the sub-buffer
    assert int(state.arena[off]) == 0xC5
    state.arena[off + 3] = 0
    assert lpmm.check_guards(state)[1] == 1
    state.arena[off + 3] = 0xC5
    assert lpmm.check_guards(state)[1] == 0
    assert lpmm.selftest_check(state) == 0x17f
    assert lpmm.device_status(state) == 0
    print(f"OK {len(cases)} configurations, {zones_total} guard zones checked after every step")


if __name__ == "__main__":
    main()
