"""Pins of the oracle's step for tensors of any rank (Alg. 3 with Alg. 4's normalization), CPU only."""
import numpy as np

import oracle
from oracle import lpmm_oracle_np as onp

HYP = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01)
TLIN = oracle.linear_map(4)


def _grad(rng, dims):
    g = rng.standard_normal(dims)
    for ax, d in enumerate(dims):        # a separable magnitude profile per axis, plus a few outliers
        shape = [1] * len(dims)
        shape[ax] = d
        g = g * np.exp(0.7 * rng.standard_normal(shape))
    g = np.where(rng.random(dims) < 1e-3, g * 50, g)
    return g.astype(np.float32).ravel()


def _fresh(dims, m_block=128):
    numel = int(np.prod(dims))
    return dict(m_codes=np.full((numel + 1) // 2, 0x77, np.uint8), m_scale=np.zeros((numel + m_block - 1) // m_block, np.float32),
                v_codes=np.zeros((numel + 1) // 2, np.uint8), mu=np.zeros(int(sum(dims)), np.float32))


def _run_nd(dims, steps, seed, m_block=128):
    rng = np.random.default_rng(seed)
    numel = int(np.prod(dims))
    w = (rng.standard_normal(numel) * 0.02).astype(np.float32)
    st = _fresh(dims, m_block)
    if numel % 2:
        st["m_codes"][-1] = 0x07
    for t in range(1, steps + 1):
        oracle.adamw4_step_nd(w, _grad(rng, dims), dims, m_block, st["m_codes"], st["m_scale"], st["v_codes"], st["mu"],
                              step=t, **HYP)
    return w, st


def test_rank_two_reduces_to_the_matrix_step():
    # p = 2: mu_1 = r, mu_2 = c, and the step must be the RANK1 branch of the matrix step bit for bit
    dims = (24, 160)
    rng = np.random.default_rng(3)
    w2 = (rng.standard_normal(24 * 160) * 0.02).astype(np.float32)
    wn = w2.copy()
    st2 = oracle.state_init(24, 160, oracle.RANK1)
    stn = _fresh(dims)
    for t in range(1, 6):
        g = _grad(rng, dims)
        oracle.adamw4_step(w2, g, st2, step=t, **HYP)
        oracle.adamw4_step_nd(wn, g, dims, 128, stn["m_codes"], stn["m_scale"], stn["v_codes"], stn["mu"], step=t, **HYP)
        assert np.array_equal(w2, wn)
        assert np.array_equal(st2.m_codes, stn["m_codes"]) and np.array_equal(st2.v_codes, stn["v_codes"])
        assert np.array_equal(st2.m_scale, stn["m_scale"])
        assert np.array_equal(st2.v_s0, stn["mu"][:24]) and np.array_equal(st2.v_s1, stn["mu"][24:])


def test_a_leading_axis_of_extent_one_changes_nothing():
    # shape (1, R, C): the extra statistic is the global maximum, never the minimum, so codes and parameters are
    # those of the R x C matrix
    rng = np.random.default_rng(4)
    R, Cc = 20, 96
    w2 = (rng.standard_normal(R * Cc) * 0.02).astype(np.float32)
    w3 = w2.copy()
    s2, s3 = _fresh((R, Cc)), _fresh((1, R, Cc))
    for t in range(1, 5):
        g = _grad(rng, (R, Cc))
        oracle.adamw4_step_nd(w2, g, (R, Cc), 128, s2["m_codes"], s2["m_scale"], s2["v_codes"], s2["mu"], step=t, **HYP)
        oracle.adamw4_step_nd(w3, g, (1, R, Cc), 128, s3["m_codes"], s3["m_scale"], s3["v_codes"], s3["mu"], step=t, **HYP)
        assert np.array_equal(w2, w3) and np.array_equal(s2["v_codes"], s3["v_codes"]) and np.array_equal(s2["m_codes"], s3["m_codes"])
        assert np.array_equal(s3["mu"][1:], s2["mu"]) and s3["mu"][0] == s2["mu"].max()


def test_statistics_are_the_axis_maxima_of_the_new_second_moment():
    # one step from zero states: v_1 = (1 - beta2) g^2 exactly as computed in binary32, so every statistic can be
    # recomputed by brute force, and every code is the nearest entry of v_1 / min over the element's statistics
    dims = (6, 10, 14)
    rng = np.random.default_rng(5)
    g = _grad(rng, dims)
    w = np.zeros(g.size, np.float32)
    st = _fresh(dims)
    oracle.adamw4_step_nd(w, g, dims, 128, st["m_codes"], st["m_scale"], st["v_codes"], st["mu"], step=1, **HYP)
    omb2 = np.float32(1.0) - np.float32(HYP["beta2"])
    v1 = (omb2 * (g * g)).astype(np.float32).reshape(dims)     # beta2 * 0 + omb2 * g^2
    mu = [v1.max(axis=(1, 2)), v1.max(axis=(0, 2)), v1.max(axis=(0, 1))]
    assert np.array_equal(np.concatenate(mu), st["mu"])
    codes = oracle.unpack4(st["v_codes"], g.size).reshape(dims)
    for idx in [(0, 0, 0), (5, 9, 13), (2, 3, 7), (4, 0, 11)]:
        M = min(mu[0][idx[0]], mu[1][idx[1]], mu[2][idx[2]])
        n = np.float32(v1[idx]) * (np.float32(1.0) / np.float32(M))
        assert codes[idx] == int(np.argmin(np.abs(TLIN.astype(np.float64) - float(n))))
    # normalized values never exceed 1, and each axis has an element that reaches the top code along it
    assert codes.max() == 15


def test_numpy_restatement_agrees_bit_for_bit():
    for dims, seed in [((5, 12, 33), 7), ((3, 4, 6, 40), 8), ((301,), 9)]:
        rng = np.random.default_rng(seed)
        numel = int(np.prod(dims))
        w = (rng.standard_normal(numel) * 0.02).astype(np.float32)
        wn = w.copy()
        st = _fresh(dims)
        if numel % 2:
            st["m_codes"][-1] = 0x07
        stn = dict(dims=dims, m_block=128, m_codes=st["m_codes"].copy(), m_scale=st["m_scale"].copy(), v_codes=st["v_codes"].copy(),
                   mu=[np.zeros(d, np.float32) for d in dims])
        for t in range(1, 5):
            g = _grad(rng, dims)
            oracle.adamw4_step_nd(w, g, dims, 128, st["m_codes"], st["m_scale"], st["v_codes"], st["mu"], step=t, **HYP)
            wn = onp.adamw4_step_nd(wn, g, stn, step=t, **HYP)
            assert np.array_equal(w, wn)
            assert np.array_equal(st["m_codes"], stn["m_codes"]) and np.array_equal(st["v_codes"], stn["v_codes"])
            assert np.array_equal(st["mu"], np.concatenate(stn["mu"]))


def test_dequantized_second_moment_stays_within_half_a_step_of_the_scale():
    # |v~ - v| <= M / 32 wherever v >= M / 16 (linear map without zero, Sec. 4.1), checked through a second step's input
    dims = (8, 16, 24)
    w, st = _run_nd(dims, 3, 11)
    M = oracle.rank1_scale_field(dims, [st["mu"][:8], st["mu"][8:24], st["mu"][24:]])
    v_deq = TLIN[oracle.unpack4(st["v_codes"], int(np.prod(dims)))].reshape(dims) * M
    assert np.all(v_deq <= M * (1 + 1e-6)) and np.all(v_deq >= M / 16 * (1 - 1e-6))
    assert np.isfinite(w).all()
