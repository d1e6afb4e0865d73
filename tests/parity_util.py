"""Helpers shared by the GPU parity tests: drive the CUDA library and the CPU oracle side by side."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2309_01507_b200 import lpmm, workloads

ORACLE_KIND = {lpmm.KIND_FP32: oracle.FP32, lpmm.KIND_BLOCK: oracle.BLOCK, lpmm.KIND_RANK1: oracle.RANK1}


def hyper_of(wl) -> dict:
    return dict(lr=wl.lr, beta1=wl.beta1, beta2=wl.beta2, eps=wl.eps, weight_decay=wl.weight_decay)


def param_tol(w_ref: np.ndarray, lr: float, tol: float) -> np.ndarray:
    """Allowed |difference| per element: tol * max(|w_ref|, lr) (relative error with a floor at the step size)."""
    return tol * np.maximum(np.abs(w_ref), lr)


class Pair:
    """The same tensors held by the CUDA library (device) and by the oracle (host)."""

    def __init__(self, specs, hyper, *, config=None, device="cuda", grad_dtype=torch.float32, workload_index=9,
                 schedule=None):
        self.specs = list(specs)
        self.hyper = dict(hyper)
        self.config = config or lpmm.default_config()
        if schedule is not None:
            self.config.schedule = schedule
            if schedule == lpmm.SCHEDULE_OVERLAP:
                self.config.overlap_groups = 3
        self.grad_dtype = grad_dtype
        self.widx = workload_index
        self.params = [workloads.make_param(s, self.widx, i, device=device) for i, s in enumerate(self.specs)]
        self.state = lpmm.state_init(self.config, self.specs, device=device)
        self.w_ref = [p.detach().cpu().numpy().ravel().copy() for p in self.params]
        self.ostate = []
        for i, s in enumerate(self.specs):
            k = ORACLE_KIND[lpmm.state_view(self.state, i)["kind"]]
            forced = 1 if s.force_quant else 0
            want = oracle.kind_of(s.rows, s.cols, s.ndim, self.config.min_quant_numel, forced)
            if self.config.v_mode == lpmm.V_BLOCK and want == oracle.RANK1:
                want = oracle.BLOCK
            assert k == want, (s, k, want)
            self.ostate.append(oracle.state_init(s.rows, s.cols, k, m_block=self.config.m_block))

    def grads_for(self, step, outlier_p=1e-3, device="cuda"):
        return [workloads.make_grad(s, self.widx, i, step, device=device, dtype=self.grad_dtype, outlier_p=outlier_p)
                for i, s in enumerate(self.specs)]

    def step(self, step, grads, true_division=False):
        lpmm.adamw4_step(self.state, self.params, grads, step=step, **self.hyper)
        for i, g in enumerate(grads):
            g32 = g.detach().float().cpu().numpy().ravel()
            oracle.adamw4_step(self.w_ref[i], g32, self.ostate[i], step=step, true_division=true_division,
                               **self.hyper)
        torch.cuda.synchronize()

    def compare(self, tol=1e-6, share_params=True, exact_params=False):
        """Codes and scales bit for bit; parameters within tol. Returns the worst normalised parameter error."""
        worst = 0.0
        assert lpmm.device_status(self.state) == 0, "a step kernel reported an expired wait"
        for i, s in enumerate(self.specs):
            view = lpmm.state_view(self.state, i)
            o = self.ostate[i]
            for name, ref in (("m_codes", o.m_codes), ("m_scale", o.m_scale), ("v_codes", o.v_codes),
                              ("v_s0", o.v_s0), ("v_s1", o.v_s1), ("m32", o.m32), ("v32", o.v32)):
                got = view[name]
                if ref is None:
                    continue
                assert got is not None, (s.name, name)
                got = got.cpu().numpy()
                if not np.array_equal(got.view(np.uint8), ref.view(np.uint8)):
                    bad = np.flatnonzero(got != ref)
                    raise AssertionError(f"{s.name}: {name} differs at {bad.size} of {ref.size} entries; first "
                                         f"{bad[:5]} gpu={got[bad[:5]]} oracle={ref[bad[:5]]}")
            w_gpu = self.params[i].detach().cpu().numpy().ravel()
            err = np.abs(w_gpu - self.w_ref[i]) / np.maximum(np.abs(self.w_ref[i]), self.hyper["lr"])
            e = float(err.max()) if err.size else 0.0
            worst = max(worst, e)
            assert e <= tol, f"{s.name}: parameter error {e:.3e} > {tol:.1e}"
            if exact_params:
                assert np.array_equal(w_gpu, self.w_ref[i]), s.name
            if share_params:
                self.w_ref[i][:] = w_gpu     # next step starts from a shared state
        return worst
