"""Invariants of the oracle's factorized-second-moment step (Sec. 4.3), CPU only.

The paper gives no formula for this variant (it cites Adafactor), so numerical parity with the paper is
unpinned; what is pinned: exactness when the squared gradient has rank one, the row-sum identity of the
reconstruction, independence of the first-moment path, and agreement of two independent writings."""
import numpy as np
import pytest

import oracle
from oracle import lpmm_oracle_np as onp

HYP = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01)


def _state(rows, cols):
    st = oracle.state_init(rows, cols, oracle.RANK1)
    return st, np.zeros(rows, np.float32), np.zeros(cols, np.float32)


def test_rank_one_squared_gradient_is_reconstructed_exactly_and_matches_adam():
    # g_ij = s_ij a_i b_j with |.| separable: then R C^T / sum(R) = (1-beta2) g^2, the ordinary second moment,
    # so the first step equals plain Adam's first step: w_1 = w_0 (1 - lr wd) - lr sign(g).
    rng = np.random.default_rng(0)
    rows, cols = 48, 128
    a = np.exp(rng.standard_normal(rows)); b = np.exp(rng.standard_normal(cols))
    sgn = rng.choice([-1.0, 1.0], size=(rows, cols))
    g = (sgn * a[:, None] * b[None, :]).astype(np.float32).ravel()
    w0 = (rng.standard_normal(rows * cols) * 0.02).astype(np.float32)
    w = w0.copy()
    st, R, C = _state(rows, cols)
    oracle.adamw4_factor_step(w, g, st, R, C, step=1, **HYP)
    want = w0.astype(np.float64) * (1 - 1e-3 * 0.01) - 1e-3 * np.sign(g)
    assert np.max(np.abs(w - want)) < 1e-3 * 3e-5
    g2 = (g.astype(np.float64) ** 2).reshape(rows, cols)
    omb2 = float(np.float32(1) - np.float32(0.999))
    np.testing.assert_allclose(R, omb2 * g2.sum(axis=1), rtol=1e-6)
    np.testing.assert_allclose(C, omb2 * g2.sum(axis=0), rtol=1e-6)


def test_reconstruction_row_and_column_sums_return_the_statistics():
    rng = np.random.default_rng(1)
    rows, cols = 40, 256
    w = np.zeros(rows * cols, np.float32)
    st, R, C = _state(rows, cols)
    for t in range(1, 4):
        g = (rng.standard_normal(rows * cols) * np.exp(rng.standard_normal(rows * cols))).astype(np.float32)
        oracle.adamw4_factor_step(w, g, st, R, C, step=t, **HYP)
    v = (R.astype(np.float64) / R.astype(np.float64).sum())[:, None] * C.astype(np.float64)[None, :]
    np.testing.assert_allclose(v.sum(axis=1), R, rtol=1e-5)          # sum_j v_ij = R_i (sum C = sum R)
    np.testing.assert_allclose(v.sum(axis=0), C, rtol=1e-5)
    np.testing.assert_allclose(R.astype(np.float64).sum(), C.astype(np.float64).sum(), rtol=1e-5)


def test_first_moment_path_equals_the_quantized_adam_step():
    rng = np.random.default_rng(2)
    rows, cols = 64, 128
    wa = (rng.standard_normal(rows * cols) * 0.02).astype(np.float32)
    wb = wa.copy()
    sa, R, C = _state(rows, cols)
    sb = oracle.state_init(rows, cols, oracle.RANK1)
    for t in range(1, 5):
        g = (rng.standard_normal(rows * cols) * np.exp(rng.standard_normal(rows * cols))).astype(np.float32)
        oracle.adamw4_factor_step(wa, g, sa, R, C, step=t, **HYP)
        oracle.adamw4_step(wb, g, sb, step=t, **HYP)
        assert np.array_equal(sa.m_codes, sb.m_codes) and np.array_equal(sa.m_scale, sb.m_scale)


def test_zero_gradient_and_zero_state_only_decay():
    rows, cols = 32, 128
    w0 = np.linspace(-1, 1, rows * cols, dtype=np.float32)
    w = w0.copy()
    st, R, C = _state(rows, cols)
    oracle.adamw4_factor_step(w, np.zeros(rows * cols, np.float32), st, R, C, step=1, **HYP)
    assert np.array_equal(w, w0 * (np.float32(1) - np.float32(1e-3) * np.float32(0.01)))
    assert np.all(R == 0) and np.all(C == 0)


@pytest.mark.parametrize("rows,cols", [(33, 77), (96, 256)])
def test_c_and_numpy_writings_agree(rows, cols):
    rng = np.random.default_rng(rows)
    w_c = (rng.standard_normal(rows * cols) * 0.02).astype(np.float32)
    w_n = w_c.copy()
    st, R, C = _state(rows, cols)
    ns = dict(rows=rows, cols=cols, m_block=128, m_codes=st.m_codes.copy(), m_scale=st.m_scale.copy(),
              R=R.copy(), C=C.copy())
    for t in range(1, 6):
        g = (rng.standard_normal(rows * cols) * np.exp(rng.standard_normal(rows * cols))).astype(np.float32)
        oracle.adamw4_factor_step(w_c, g, st, R, C, step=t, **HYP)
        w_n = onp.adamw4_factor_step(w_n, g, ns, step=t, **HYP)
        assert np.array_equal(st.m_codes, ns["m_codes"]) and np.array_equal(st.m_scale, ns["m_scale"])
        assert np.array_equal(R, ns["R"]) and np.array_equal(C, ns["C"])
        assert np.array_equal(w_c, w_n)
