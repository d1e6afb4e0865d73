"""Pins of the oracle's compressed AdamW step (CPU only)."""
import numpy as np
import pytest
import torch

import oracle
from oracle import lpmm_oracle_np as onp

HYP = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01)
TDE = oracle.de_map(4, True)
TLIN = oracle.linear_map(4)
KIND_NAME = {oracle.FP32: "fp32", oracle.BLOCK: "block", oracle.RANK1: "rank1"}


def _grad(rng, rows, cols, outliers=True):
    g = rng.standard_normal((rows, cols)) * np.exp(rng.standard_normal((rows, 1))) * np.exp(rng.standard_normal((1, cols)))
    if outliers:
        g = np.where(rng.random((rows, cols)) < 1e-3, g * 100, g)
    return g.astype(np.float32).ravel()


def _np_state(st):
    d = dict(kind=KIND_NAME[st.kind], rows=st.rows, cols=st.cols, m_block=st.m_block, v_block=st.v_block)
    for k in ("m_codes", "m_scale", "v_codes", "v_s0", "v_s1", "m32", "v32"):
        a = getattr(st, k)
        if a is not None:
            d[k] = a.copy()
    return d


# ------------------------------------------------------------------ textbook AdamW (fp32 states)

@pytest.mark.parametrize("wd", [0.0, 0.01])
def test_fp32_branch_matches_library_adamw(wd):
    rng = np.random.default_rng(0)
    n = 2000
    w0 = (rng.standard_normal(n) * 0.02).astype(np.float32)
    w = w0.copy()
    st = oracle.state_init(n, 1, oracle.FP32)
    p = torch.nn.Parameter(torch.from_numpy(w0.copy()))
    opt = torch.optim.AdamW([p], lr=1e-3, betas=(0.9, 0.999), eps=1e-8, weight_decay=wd, foreach=False)
    for t in range(1, 21):
        g = _grad(rng, n, 1, outliers=False)
        oracle.adamw4_step(w, g, st, step=t, **{**HYP, "weight_decay": wd})
        p.grad = torch.from_numpy(g.copy())
        opt.step()
        ref = p.detach().numpy()
        # the library evaluates the same formula in another operation order: a few ulp per step, accumulating
        assert np.max(np.abs(w - ref) / np.maximum(np.abs(ref), 1e-3)) < 5e-7 * t + 5e-7
    assert np.max(np.abs(w - w0)) > 1e-3          # the parameters did move


def test_first_step_closed_form():
    # From zero states, step 1 of Eq. 1 gives m^ = g, v^ = g^2, so the update is lr * g/(|g| + eps):
    # w_1 = w_0 (1 - lr wd) - lr sign(g) up to eps and rounding, for every state kind.
    rng = np.random.default_rng(1)
    for rows, cols, kind in [(40, 128, oracle.RANK1), (5000, 1, oracle.BLOCK), (100, 1, oracle.FP32)]:
        w0 = (rng.standard_normal(rows * cols) * 0.02).astype(np.float32)
        g = _grad(rng, rows, cols)
        g[np.abs(g) < 1e-3] = 1e-3
        w = w0.copy()
        st = oracle.state_init(rows, cols, kind)
        oracle.adamw4_step(w, g, st, step=1, **HYP)
        want = w0.astype(np.float64) * (1 - 1e-3 * 0.01) - 1e-3 * np.sign(g)
        assert np.max(np.abs(w - want)) < 1e-3 * 2e-5


def test_zero_gradient_only_decays():
    w0 = np.linspace(-1, 1, 5000, dtype=np.float32)
    for kind, rows, cols in [(oracle.RANK1, 50, 100), (oracle.BLOCK, 5000, 1), (oracle.FP32, 5000, 1)]:
        w = w0.copy()
        st = oracle.state_init(rows, cols, kind)
        oracle.adamw4_step(w, np.zeros(5000, np.float32), st, step=1, **HYP)
        assert np.array_equal(w, w0 * (np.float32(1) - np.float32(1e-3) * np.float32(0.01)))
        if kind != oracle.FP32:
            assert np.all(st.m_scale == 0) and np.all(st.v_s0 == 0)
            assert np.all(oracle.unpack4(st.m_codes, 5000) == 7) and np.all(st.v_codes == 0)


def test_weight_decay_zero_is_plain_adam():
    rng = np.random.default_rng(2)
    w0 = (rng.standard_normal(6000) * 0.02).astype(np.float32)
    g = _grad(rng, 60, 100)
    wa, wb = w0.copy(), w0.copy()
    sa, sb = oracle.state_init(60, 100, oracle.RANK1), oracle.state_init(60, 100, oracle.RANK1)
    oracle.adamw4_step(wa, g, sa, step=1, **{**HYP, "weight_decay": 0.0})
    oracle.adamw4_step(wb, g, sb, step=1, **HYP)
    # decay touches only w: identical states, and wb - wa = -lr*wd*w0 up to rounding
    assert np.array_equal(sa.m_codes, sb.m_codes) and np.array_equal(sa.v_codes, sb.v_codes)
    np.testing.assert_allclose(wb - wa, -1e-3 * 0.01 * w0, atol=1e-8)


# ------------------------------------------------------------------ the state path, piece by piece

def test_step_equals_decompress_update_compress_spelled_out():
    # Alg. 3: new states = compress(EMA(decompress(old states), g)), checked with the quantizer
    # entry points (pinned separately) and the EMAs evaluated in binary64 (tolerance on thresholds).
    rng = np.random.default_rng(3)
    rows, cols = 96, 256
    w = (rng.standard_normal(rows * cols) * 0.02).astype(np.float32)
    st = oracle.state_init(rows, cols, oracle.RANK1)
    for t in range(1, 4):
        g = _grad(rng, rows, cols)
        m_old = oracle.dequantize_block(oracle.unpack4(st.m_codes, rows * cols), 128, TDE, st.m_scale).astype(np.float64)
        v_old = oracle.dequantize_rank1(oracle.unpack4(st.v_codes, rows * cols).reshape(rows, cols), TLIN,
                                        st.v_s0, st.v_s1).astype(np.float64).ravel()
        oracle.adamw4_step(w, g, st, step=t, **HYP)
        b1, b2 = float(np.float32(0.9)), float(np.float32(0.999))     # the binary32 hyper-parameters
        m_new = b1 * m_old + (1 - b1) * g.astype(np.float64)
        v_new = b2 * v_old + (1 - b2) * g.astype(np.float64) ** 2
        np.testing.assert_allclose(st.m_scale, np.abs(m_new).reshape(-1, 128).max(axis=1), rtol=1e-6)
        np.testing.assert_allclose(st.v_s0, v_new.reshape(rows, cols).max(axis=1), rtol=1e-6)
        np.testing.assert_allclose(st.v_s1, v_new.reshape(rows, cols).max(axis=0), rtol=1e-6)
        qm, _ = oracle.quantize_block(m_new.astype(np.float32), 128, TDE)
        qv, _, _ = oracle.quantize_rank1(v_new.astype(np.float32).reshape(rows, cols), TLIN)
        dm = qm.astype(int) - oracle.unpack4(st.m_codes, rows * cols).astype(int)
        dv = qv.ravel().astype(int) - oracle.unpack4(st.v_codes, rows * cols).astype(int)
        assert np.mean(dm != 0) < 1e-3 and np.max(np.abs(dm)) <= 1
        assert np.mean(dv != 0) < 1e-3 and np.max(np.abs(dv)) <= 1


def test_update_uses_unquantized_new_moments():
    # Alg. 3 lines 4-8 use m_t, v_t before compression: from the same decompressed state, the
    # parameter update equals a float64 evaluation of Eq. 1 to rounding accuracy.
    rng = np.random.default_rng(4)
    rows, cols = 64, 128
    w = (rng.standard_normal(rows * cols) * 0.02).astype(np.float32)
    st = oracle.state_init(rows, cols, oracle.RANK1)
    for t in range(1, 5):
        g = _grad(rng, rows, cols)
        m_old = oracle.dequantize_block(oracle.unpack4(st.m_codes, rows * cols), 128, TDE, st.m_scale).astype(np.float64)
        v_old = oracle.dequantize_rank1(oracle.unpack4(st.v_codes, rows * cols).reshape(rows, cols), TLIN,
                                        st.v_s0, st.v_s1).astype(np.float64).ravel()
        w_prev = w.astype(np.float64)
        oracle.adamw4_step(w, g, st, step=t, **HYP)
        g64 = g.astype(np.float64)
        b1, b2 = float(np.float32(0.9)), float(np.float32(0.999))
        m_new = b1 * m_old + (1 - b1) * g64
        v_new = b2 * v_old + (1 - b2) * g64 ** 2
        want = w_prev * (1 - 1e-3 * 0.01) - 1e-3 * (m_new / (1 - b1 ** t)) / (np.sqrt(v_new / (1 - b2 ** t)) + 1e-8)
        assert np.max(np.abs(w - want) / np.maximum(np.abs(want), 1e-3)) < 1e-6


def test_state_path_never_reads_parameters():
    rng = np.random.default_rng(5)
    rows, cols = 48, 256
    wa = (rng.standard_normal(rows * cols)).astype(np.float32)
    wb = np.zeros(rows * cols, np.float32)
    sa, sb = oracle.state_init(rows, cols, oracle.RANK1), oracle.state_init(rows, cols, oracle.RANK1)
    for t in range(1, 6):
        g = _grad(rng, rows, cols)
        oracle.adamw4_step(wa, g, sa, step=t, **HYP)
        oracle.adamw4_step(wb, g, sb, step=t, **{**HYP, "lr": 0.5, "weight_decay": 0.3})
    for k in ("m_codes", "m_scale", "v_codes", "v_s0", "v_s1"):
        assert np.array_equal(getattr(sa, k), getattr(sb, k))


def test_alg3_typo_reading_uses_one_minus_beta2():
    # With beta1 != beta2 the second-moment EMA weight must be (1 - beta2) as in Eq. 1:
    # after one step from zero, v_1 = (1 - beta2) g^2, so the row maxima are (1 - beta2) max g^2.
    rng = np.random.default_rng(6)
    g = _grad(rng, 40, 128)
    w = np.zeros(40 * 128, np.float32)
    st = oracle.state_init(40, 128, oracle.RANK1)
    oracle.adamw4_step(w, g, st, step=1, **HYP)
    omb2 = np.float32(1) - np.float32(0.999)
    np.testing.assert_allclose(st.v_s0, omb2 * (g.reshape(40, 128) ** 2).max(axis=1), rtol=3e-7)


# ------------------------------------------------------------------ two independent writings

@pytest.mark.parametrize("rows,cols,kind,true_div", [
    (96, 256, oracle.RANK1, False), (33, 77, oracle.RANK1, False), (50, 128, oracle.RANK1, True),
    (5001, 1, oracle.BLOCK, False), (4097, 1, oracle.BLOCK, True), (777, 1, oracle.FP32, False),
])
def test_c_and_numpy_writings_agree_bit_for_bit(rows, cols, kind, true_div):
    rng = np.random.default_rng(rows * 7 + cols)
    w_c = (rng.standard_normal(rows * cols) * 0.02).astype(np.float32)
    w_n = w_c.copy()
    st = oracle.state_init(rows, cols, kind)
    ns = _np_state(st)
    for t in range(1, 7):
        g = _grad(rng, rows, cols)
        if t == 3:
            g[: cols * 2] = 0            # whole zero rows (sparse-token gradients)
        oracle.adamw4_step(w_c, g, st, step=t, true_division=true_div, **HYP)
        w_n = onp.adamw4_step(w_n, g, ns, step=t, true_division=true_div, **HYP)
        assert np.array_equal(w_c, w_n)
        for k in ("m_codes", "m_scale", "v_codes", "v_s0", "v_s1", "m32", "v32"):
            a = getattr(st, k)
            if a is not None:
                assert np.array_equal(a, ns[k]), (k, t)


def test_reciprocal_and_division_trajectories_stay_adjacent():
    rng = np.random.default_rng(8)
    rows, cols = 128, 512
    wa = (rng.standard_normal(rows * cols) * 0.02).astype(np.float32)
    wb = wa.copy()
    sa, sb = oracle.state_init(rows, cols, oracle.RANK1), oracle.state_init(rows, cols, oracle.RANK1)
    g = _grad(rng, rows, cols)
    oracle.adamw4_step(wa, g, sa, step=1, true_division=False, **HYP)
    oracle.adamw4_step(wb, g, sb, step=1, true_division=True, **HYP)
    assert np.array_equal(wa, wb) and np.array_equal(sa.v_s0, sb.v_s0) and np.array_equal(sa.m_scale, sb.m_scale)
    for ka in ("m_codes", "v_codes"):
        a = oracle.unpack4(getattr(sa, ka), rows * cols).astype(int)
        b = oracle.unpack4(getattr(sb, ka), rows * cols).astype(int)
        assert np.mean(a != b) < 1e-4 and np.max(np.abs(a - b)) <= 1


def test_bad_arguments_are_rejected():
    st = oracle.state_init(10, 1, oracle.FP32)
    with pytest.raises(ValueError):
        oracle.adamw4_step(np.zeros(10, np.float32), np.zeros(10, np.float32), st, step=0, **HYP)
