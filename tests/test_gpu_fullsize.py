"""Full-size parity: the LLaMA-7B-shaped workload exactly as bench.py launches it (all 291 tensors, bf16
gradients, one multi-tensor launch per pass), checked on sampled tensors the oracle can compute one by one:
one tensor of every distinct shape. Codes and scales bit for bit, parameters within 1e-6 * max(|w|, lr)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2309_01507_b200 import lpmm, workloads
from parity_util import ORACLE_KIND, hyper_of

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("schedule", [lpmm.SCHEDULE_AUTO, lpmm.SCHEDULE_FUSED], ids=["auto", "fused"])
def test_llama_7b_full_size_sampled_tensors(schedule):
    free, _ = torch.cuda.mem_get_info()
    if free < 60 * 2 ** 30:
        pytest.skip("needs about 50 GB of free device memory")
    wl = workloads.llama_7b()
    hyper = hyper_of(wl)
    dev = "cuda"
    params = [workloads.make_param(t, wl.index, i, device=dev) for i, t in enumerate(wl.tensors)]
    state = lpmm.state_init(lpmm.default_config(schedule=schedule), wl.tensors, device=dev)
    names = {t.name: i for i, t in enumerate(wl.tensors)}
    sample = [names[n] for n in ("embed", "l0.q", "l17.gate", "l31.down", "l5.norm1", "lm_head")]
    w_ref = {i: params[i].detach().cpu().numpy().ravel().copy() for i in sample}
    ostate = {}
    for i in sample:
        t = wl.tensors[i]
        ostate[i] = oracle.state_init(t.rows, t.cols, ORACLE_KIND[lpmm.state_view(state, i)["kind"]])
    steps = 2
    for step in range(1, steps + 1):
        grads = [workloads.make_grad(t, wl.index, i, step, device=dev, dtype=torch.bfloat16)
                 for i, t in enumerate(wl.tensors)]
        lpmm.adamw4_step(state, params, grads, step=step, **hyper)
        torch.cuda.synchronize()
        for i in sample:
            oracle.adamw4_step(w_ref[i], grads[i].float().cpu().numpy().ravel(), ostate[i], step=step, **hyper)
        del grads
    assert state.last_launches == (1 if schedule == lpmm.SCHEDULE_FUSED else 3)
    for i in sample:
        t = wl.tensors[i]
        view = lpmm.state_view(state, i)
        o = ostate[i]
        for name, ref in (("m_codes", o.m_codes), ("m_scale", o.m_scale), ("v_codes", o.v_codes),
                          ("v_s0", o.v_s0), ("v_s1", o.v_s1), ("m32", o.m32), ("v32", o.v32)):
            if ref is None:
                continue
            got = view[name].cpu().numpy()
            assert np.array_equal(got.view(np.uint8), ref.view(np.uint8)), (t.name, name)
        w = params[i].detach().cpu().numpy().ravel()
        err = np.abs(w - w_ref[i]) / np.maximum(np.abs(w_ref[i]), hyper["lr"])
        assert float(err.max()) <= 1e-6, (t.name, float(err.max()))
    # every parameter tensor moved and stayed finite (cheap whole-workload property)
    for i in (1, 100, 200, 289):
        assert torch.isfinite(params[i]).all()
