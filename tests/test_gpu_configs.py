"""The benchmark's workloads as specified, against the oracle: the Transformer-base list over its 100 steps with the
oracle keeping its own fp32 trajectory, the whole RoBERTa-large list in one multi-tensor step, and the flattened
LLaMA-7B list at full size. Tolerances: codes and scales bit for bit after a step from a shared state, parameters
within 1e-6 * max(|w|, lr); over the 100-step trajectory parameters within 1e-4 and at most 1e-6 of the codes off by
one adjacent code."""
import numpy as np
import pytest
import torch

import oracle
from paper_2309_01507_b200 import lpmm, workloads
from parity_util import ORACLE_KIND, hyper_of

pytestmark = pytest.mark.gpu

STATE_FIELDS = ("m_codes", "m_scale", "v_codes", "v_s0", "v_s1", "m32", "v32")


def _oracle_states(state, wl, sample):
    out = {}
    for i in sample:
        t = wl.tensors[i]
        out[i] = oracle.state_init(t.rows, t.cols, ORACLE_KIND[lpmm.state_view(state, i)["kind"]])
    return out


def _assert_states_equal(state, wl, ostate, i):
    view = lpmm.state_view(state, i)
    for name in STATE_FIELDS:
        ref = getattr(ostate[i], name)
        if ref is None:
            continue
        got = view[name].cpu().numpy()
        assert np.array_equal(got.view(np.uint8), ref.view(np.uint8)), (wl.tensors[i].name, name)


def test_transformer_base_100_step_trajectory():
    # Config as specified: 181 tensors, fresh gradients every step, 100 steps, every tensor in each launch. The oracle
    # runs its own trajectory from the same initial parameters (nothing is shared after step 0).
    wl = workloads.transformer_base()
    hyper = hyper_of(wl)
    n = len(wl.tensors)
    params = [workloads.make_param(t, wl.index, i, device="cuda") for i, t in enumerate(wl.tensors)]
    state = lpmm.state_init(lpmm.default_config(), wl.tensors)
    w_ref = [p.cpu().numpy().ravel().copy() for p in params]
    ostate = _oracle_states(state, wl, range(n))
    for step in range(1, wl.steps + 1):
        grads = [workloads.make_grad(t, wl.index, i, step, device="cuda") for i, t in enumerate(wl.tensors)]
        lpmm.adamw4_step(state, params, grads, step=step, **hyper)
        for i in range(n):
            oracle.adamw4_step(w_ref[i], grads[i].cpu().numpy().ravel(), ostate[i], step=step, **hyper)
    torch.cuda.synchronize()
    assert lpmm.device_status(state) == 0
    total_codes = off_codes = 0
    worst = 0.0
    for i, t in enumerate(wl.tensors):
        view = lpmm.state_view(state, i)
        o = ostate[i]
        for name in ("m_codes", "v_codes"):
            ref = getattr(o, name)
            if ref is None:
                continue
            a = oracle.unpack4(view[name].cpu().numpy(), t.numel).astype(np.int32)
            b = oracle.unpack4(ref, t.numel).astype(np.int32)
            diff = np.abs(a - b)
            assert diff.max(initial=0) <= 1, (t.name, name)
            total_codes += t.numel
            off_codes += int(np.count_nonzero(diff))
        w = params[i].cpu().numpy().ravel()
        err = np.abs(w - w_ref[i]) / np.maximum(np.abs(w_ref[i]), hyper["lr"])
        worst = max(worst, float(err.max()))
    assert off_codes <= 1e-6 * total_codes, (off_codes, total_codes)
    assert worst <= 1e-4, worst
    # the state path never reads the parameters, so in fact nothing differs: scales included
    for i in range(n):
        _assert_states_equal(state, wl, ostate, i)


def test_roberta_large_whole_list_two_steps():
    # All 394 tensors in one step (355 M parameters, fp32 gradients, 90 % of the token-embedding gradient rows zero);
    # the oracle follows a sample: the sparse embedding, the odd-length bias and one tensor of every other shape.
    wl = workloads.roberta_large()
    hyper = hyper_of(wl)
    names = {t.name: i for i, t in enumerate(wl.tensors)}
    sample = [names[k] for k in ("emb.word", "emb.pos", "emb.type", "emb.ln.w", "l0.q.w", "l0.q.b", "l11.fc1.w", "l11.fc1.b",
                                 "l23.fc2.w", "head.dense.w", "head.bias")]
    params = [workloads.make_param(t, wl.index, i, device="cuda") for i, t in enumerate(wl.tensors)]
    state = lpmm.state_init(lpmm.default_config(), wl.tensors)
    kinds = [lpmm.state_view(state, i)["kind"] for i in range(len(wl.tensors))]
    assert (kinds.count(lpmm.KIND_RANK1), kinds.count(lpmm.KIND_BLOCK), kinds.count(lpmm.KIND_FP32)) == (147, 1, 246)
    w_ref = {i: params[i].cpu().numpy().ravel().copy() for i in sample}
    ostate = _oracle_states(state, wl, sample)
    for step in (1, 2):
        grads = [workloads.make_grad(t, wl.index, i, step, device="cuda") for i, t in enumerate(wl.tensors)]
        assert float((grads[0].abs().sum(dim=1) == 0).float().mean()) > 0.85          # the sparse-token pattern is there
        lpmm.adamw4_step(state, params, grads, step=step, **hyper)
        torch.cuda.synchronize()
        assert state.last_launches == 4
        for i in sample:
            oracle.adamw4_step(w_ref[i], grads[i].cpu().numpy().ravel(), ostate[i], step=step, **hyper)
            _assert_states_equal(state, wl, ostate, i)
            w = params[i].cpu().numpy().ravel()
            err = np.abs(w - w_ref[i]) / np.maximum(np.abs(w_ref[i]), hyper["lr"])
            assert float(err.max()) <= 1e-6, (wl.tensors[i].name, step, float(err.max()))
            w_ref[i][:] = w                       # the next step starts from a shared state
        del grads
    assert lpmm.device_status(state) == 0


def test_llama_7b_flat_full_size_sampled_tensors():
    # The flattened LLaMA-7B list as the benchmark runs it (34 one-dimensional tensors of up to 202 M elements, bf16
    # gradients, block-wise second moments, folded onto the tiled kernel); the oracle follows one decoder layer's
    # tensor and the head, which ends in a ragged 4096-element tail.
    free, _ = torch.cuda.mem_get_info()
    if free < 60 * 2 ** 30:
        pytest.skip("needs about 50 GB of free device memory")
    wl = workloads.llama_7b_flat()
    hyper = hyper_of(wl)
    names = {t.name: i for i, t in enumerate(wl.tensors)}
    sample = [names["l3"], names["head"]]
    params = [workloads.make_param(t, wl.index, i, device="cuda") for i, t in enumerate(wl.tensors)]
    state = lpmm.state_init(lpmm.default_config(), wl.tensors)
    assert all(lpmm.state_view(state, i)["kind"] == lpmm.KIND_BLOCK for i in range(len(wl.tensors)))
    w_ref = {i: params[i].cpu().numpy().ravel().copy() for i in sample}
    ostate = _oracle_states(state, wl, sample)
    for step in (1, 2):
        grads = [workloads.make_grad(t, wl.index, i, step, device="cuda", dtype=torch.bfloat16) for i, t in enumerate(wl.tensors)]
        lpmm.adamw4_step(state, params, grads, step=step, **hyper)
        torch.cuda.synchronize()
        for i in sample:
            oracle.adamw4_step(w_ref[i], grads[i].float().cpu().numpy().ravel(), ostate[i], step=step, **hyper)
            _assert_states_equal(state, wl, ostate, i)
            w = params[i].cpu().numpy().ravel()
            err = np.abs(w - w_ref[i]) / np.maximum(np.abs(w_ref[i]), hyper["lr"])
            assert float(err.max()) <= 1e-6, (wl.tensors[i].name, step, float(err.max()))
            w_ref[i][:] = w
        del grads
    assert lpmm.device_status(state) == 0


@pytest.mark.parametrize("m_block", [128, 2048])
@pytest.mark.parametrize("v_mode", [lpmm.V_RANK1, lpmm.V_BLOCK, lpmm.V_FACTORED], ids=["rank1", "block", "factored"])
def test_square_8192_sweep_variants_full_size(m_block, v_mode):
    # The quantizer / normalizer sweep as the benchmark runs it: one 8192 x 8192 matrix (67 M elements, many tiles and
    # tile rows), first-moment blocks of 128 and 2048, second moment rank-1, block-wise or factorized; the oracle
    # follows the whole matrix for two steps from a shared state.
    wl = workloads.square_8192()
    hyper = hyper_of(wl)
    spec = wl.tensors[0]
    cfg = lpmm.default_config(m_block=m_block, v_mode=v_mode)
    p = workloads.make_param(spec, wl.index, 0, device="cuda")
    state = lpmm.state_init(cfg, wl.tensors)
    w_ref = p.cpu().numpy().ravel().copy()
    factored = v_mode == lpmm.V_FACTORED
    okind = oracle.BLOCK if v_mode == lpmm.V_BLOCK else oracle.RANK1
    ost = oracle.state_init(spec.rows, spec.cols, okind, m_block=m_block)
    R, Cc = np.zeros(spec.rows, np.float32), np.zeros(spec.cols, np.float32)
    for step in (1, 2):
        g = workloads.make_grad(spec, wl.index, 0, step, device="cuda")
        lpmm.adamw4_step(state, [p], [g], step=step, **hyper)
        torch.cuda.synchronize()
        assert lpmm.device_status(state) == 0
        g_host = g.cpu().numpy().ravel()
        w_prev = w_ref.copy()
        view = lpmm.state_view(state, 0)
        if factored:
            oracle.adamw4_factor_step(w_ref, g_host, ost, R, Cc, step=step, **hyper)
            np.testing.assert_allclose(view["v_s0"].cpu().numpy(), R, rtol=1e-6, atol=0)
            np.testing.assert_allclose(view["v_s1"].cpu().numpy(), Cc, rtol=1e-6, atol=0)
            names = ("m_codes", "m_scale")
        else:
            oracle.adamw4_step(w_ref, g_host, ost, step=step, **hyper)
            names = ("m_codes", "m_scale", "v_codes", "v_s0", "v_s1")
        for name in names:
            ref = getattr(ost, name)
            if ref is not None:
                assert np.array_equal(view[name].cpu().numpy().view(np.uint8), ref.view(np.uint8)), (name, step)
        w = p.cpu().numpy().ravel()
        scale = np.maximum(np.abs(w_ref), hyper["lr"])
        if factored:       # the step an element took joins the normaliser (see the factorized test in test_gpu_parity.py)
            scale = np.maximum(scale, np.abs(w_ref - w_prev))
        err = float(np.max(np.abs(w - w_ref) / scale))
        assert err <= 1e-6, (step, err)
        w_ref[:] = w
