"""Pins of the oracle's compressed SGDM step (Alg. 2), CPU only."""
import numpy as np
import pytest
import torch

import oracle
from oracle import lpmm_oracle_np as onp

TDE = oracle.de_map(4, True)


def _grad(rng, n):
    return (rng.standard_normal(n) * np.exp(rng.standard_normal(n))).astype(np.float32)


def test_fp32_branch_matches_library_sgd_with_momentum():
    rng = np.random.default_rng(0)
    n = 3000
    w0 = (rng.standard_normal(n) * 0.02).astype(np.float32)
    w = w0.copy()
    st = oracle.state_init(n, 1, oracle.FP32)
    p = torch.nn.Parameter(torch.from_numpy(w0.copy()))
    opt = torch.optim.SGD([p], lr=0.01, momentum=0.9, dampening=0.0, nesterov=False, foreach=False)
    for t in range(1, 16):
        g = _grad(rng, n)
        oracle.sgdm4_step(w, g, st, lr=0.01, beta=0.9)
        p.grad = torch.from_numpy(g.copy())
        opt.step()
        ref = p.detach().numpy()                         # the library may fuse w - lr*buf into one rounding
        assert np.max(np.abs(w - ref) / np.maximum(np.abs(ref), 1e-2)) < 3e-7 * t


def test_zero_momentum_is_plain_sgd_and_state_is_the_quantized_gradient():
    rng = np.random.default_rng(1)
    n = 128 * 50 + 17
    w0 = (rng.standard_normal(n) * 0.02).astype(np.float32)
    g = _grad(rng, n)
    w = w0.copy()
    st = oracle.state_init(n, 1, oracle.BLOCK)
    oracle.sgdm4_step(w, g, st, lr=0.1, beta=0.0)
    assert np.array_equal(w, w0 - np.float32(0.1) * g)
    q, s = oracle.quantize_block(g, 128, TDE)
    assert np.array_equal(st.m_scale, s) and np.array_equal(oracle.unpack4(st.m_codes, n), q)


def test_step_is_decompress_update_compress():
    rng = np.random.default_rng(2)
    n = 128 * 40
    w = (rng.standard_normal(n) * 0.02).astype(np.float32)
    st = oracle.state_init(n, 1, oracle.BLOCK)
    for t in range(4):
        g = _grad(rng, n)
        m_old = oracle.dequantize_block(oracle.unpack4(st.m_codes, n), 128, TDE, st.m_scale).astype(np.float64)
        w_prev = w.astype(np.float64)
        oracle.sgdm4_step(w, g, st, lr=0.05, beta=0.9)
        m_new = float(np.float32(0.9)) * m_old + g
        np.testing.assert_allclose(w, w_prev - float(np.float32(0.05)) * m_new, rtol=0, atol=4e-7 * np.max(np.abs(w_prev)) + 4e-7 * 0.05 * np.max(np.abs(m_new)))
        np.testing.assert_allclose(st.m_scale, np.abs(m_new).reshape(-1, 128).max(axis=1), rtol=2e-7)


@pytest.mark.parametrize("n,kind,mb", [(128 * 33 + 5, oracle.BLOCK, 128), (5000, oracle.BLOCK, 2048), (700, oracle.FP32, 128)])
def test_c_and_numpy_writings_agree(n, kind, mb):
    rng = np.random.default_rng(n)
    w_c = (rng.standard_normal(n) * 0.02).astype(np.float32)
    w_n = w_c.copy()
    st = oracle.state_init(n, 1, kind, m_block=mb)
    ns = dict(kind="fp32" if kind == oracle.FP32 else "block", rows=n, cols=1, m_block=mb)
    for k in ("m_codes", "m_scale", "m32"):
        if getattr(st, k) is not None:
            ns[k] = getattr(st, k).copy()
    for t in range(5):
        g = _grad(rng, n)
        oracle.sgdm4_step(w_c, g, st, lr=0.01, beta=0.9)
        w_n = onp.sgdm4_step(w_n, g, ns, lr=0.01, beta=0.9)
        assert np.array_equal(w_c, w_n)
        for k in ("m_codes", "m_scale", "m32"):
            if getattr(st, k) is not None:
                assert np.array_equal(getattr(st, k), ns[k])
