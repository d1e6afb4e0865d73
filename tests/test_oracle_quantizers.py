"""Pins of the oracle's normalizers, quantizers and packing (CPU only)."""
import numpy as np
import pytest

import oracle
from oracle import lpmm_oracle_np as onp
from conftest import read_golden

EX = read_golden("worked_examples.txt")
TDE = oracle.de_map(4, True)
TLIN = oracle.linear_map(4)


def _fl(key):
    return np.array([float(s) for s in EX[key]], np.float32)


def _il(key):
    return np.array([int(s) for s in EX[key]], np.uint8)


# ------------------------------------------------------------------ hand-worked examples

@pytest.mark.parametrize("impl", [oracle, onp])
def test_rank1_linear_worked_example(impl):
    x = _fl("r1_x").reshape(2, 3)
    codes, r, c = impl.quantize_rank1(x, TLIN)
    assert np.array_equal(r, _fl("r1_r")) and np.array_equal(c, _fl("r1_c"))
    assert np.array_equal(np.asarray(codes).ravel(), _il("r1_codes"))
    deq = impl.dequantize_rank1(np.asarray(codes).reshape(2, 3), TLIN, r, c)
    assert np.array_equal(np.asarray(deq, np.float32).ravel(), _fl("r1_dequant"))
    field = impl.rank1_scale_field((2, 3), impl.rank1_stats(x))
    assert np.array_equal(field.ravel(), _fl("r1_scale"))
    x2 = _fl("r1b_x").reshape(2, 3)
    codes2, r2, c2 = impl.quantize_rank1(x2, TLIN)
    assert np.array_equal(np.asarray(codes2).ravel(), _il("r1b_codes"))
    deq2 = impl.dequantize_rank1(np.asarray(codes2).reshape(2, 3), TLIN, r2, c2)
    assert np.array_equal(np.asarray(deq2, np.float32).ravel(), _fl("r1b_dequant"))


@pytest.mark.parametrize("impl", [oracle, onp])
def test_block_de_worked_example(impl):
    x = _fl("b_x")
    codes, scale = impl.quantize_block(x, 128, TDE)
    assert np.array_equal(scale, _fl("b_absmax"))
    assert np.array_equal(codes, _il("b_codes"))
    packed = impl.pack4(codes)
    assert packed.tobytes().hex() == "".join(EX["b_packed_hex"])
    deq = impl.dequantize_block(codes, 128, TDE, scale)
    np.testing.assert_allclose(deq, _fl("b_dequant"), rtol=1e-7, atol=0)


# ------------------------------------------------------------------ brute force on tiny inputs

def test_block_scales_brute_force_and_short_last_block():
    rng = np.random.default_rng(0)
    for numel, B in [(1, 128), (127, 128), (128, 128), (129, 128), (1000, 128), (5000, 2048), (300, 8)]:
        x = rng.standard_normal(numel).astype(np.float32)
        want = [max(abs(float(v)) for v in x[k:k + B]) for k in range(0, numel, B)]
        for impl in (oracle, onp):
            got = impl.block_scales(x, B)
            assert len(got) == -(-numel // B)                         # ceil(p/B) scales
            assert np.array_equal(got, np.array(want, np.float32))


def test_rank1_stats_brute_force_2d_and_nd():
    rng = np.random.default_rng(1)
    for shape in [(3, 5), (1, 7), (6, 1), (2, 3, 4), (3, 2, 2, 5)]:
        x = rng.standard_normal(shape).astype(np.float32)
        want = [np.zeros(d, np.float32) for d in shape]
        for idx in np.ndindex(*shape):
            for r, j in enumerate(idx):
                want[r][j] = max(want[r][j], abs(x[idx]))
        M = np.zeros(shape, np.float32)
        for idx in np.ndindex(*shape):
            M[idx] = min(want[r][j] for r, j in enumerate(idx))
        for impl in (oracle, onp):
            got = impl.rank1_stats(x)
            for a, b in zip(got, want):
                assert np.array_equal(a, b)
            assert np.array_equal(impl.rank1_scale_field(shape, got), M)


def test_rank1_quantizer_uses_the_alg4_scale_field():
    rng = np.random.default_rng(2)
    x = np.abs(rng.standard_normal((37, 53))).astype(np.float32) ** 3
    codes, r, c = oracle.quantize_rank1(x, TLIN)
    stats = oracle.rank1_stats(x)
    assert np.array_equal(r, stats[0]) and np.array_equal(c, stats[1])
    field = oracle.rank1_scale_field(x.shape, stats)
    via_field = oracle.map_codes(x, field, TLIN)          # n = x * rcp(min(r,c))
    assert np.array_equal(codes, via_field)               # max(rcp r, rcp c) == rcp(min(r, c))
    brute = np.array([[np.argmin(np.abs(float(x[i, j]) * float(np.float32(1) / field[i, j]) -
                                        TLIN.astype(np.float64))) for j in range(53)] for i in range(37)])
    # float64 product here is not the binary32 product; allow only threshold-adjacent disagreements
    assert np.mean(brute != codes) < 0.002 and np.max(np.abs(brute.astype(int) - codes.astype(int))) <= 1


# ------------------------------------------------------------------ invariants

def test_normalized_range_and_extremes():
    rng = np.random.default_rng(3)
    x = rng.standard_normal(128 * 40 + 17).astype(np.float32) * np.exp(rng.standard_normal(128 * 40 + 17)).astype(np.float32)
    codes, scale = oracle.quantize_block(x, 128, TDE)
    for k in range(len(scale)):
        blk = x[k * 128:(k + 1) * 128]
        q = codes[k * 128:(k + 1) * 128]
        i = int(np.argmax(np.abs(blk)))
        assert q[i] == (15 if blk[i] > 0 else 0)          # block extreme: n = +-1 -> top / bottom entry
    v = (rng.standard_normal((64, 96)).astype(np.float32)) ** 2
    qv, r, c = oracle.quantize_rank1(v, TLIN)
    i, j = np.unravel_index(np.argmax(v), v.shape)
    assert qv[i, j] == 15                                 # global maximum normalizes to 1
    assert np.all(qv[np.arange(64), np.argmax(v, axis=1)] == 15)   # every row maximum too (c_j >= r_i there)
    assert np.all(qv[np.argmax(v, axis=0), np.arange(96)] == 15)   # and every column maximum
    n = v * np.maximum(onp.rcp(r)[:, None], onp.rcp(c)[None, :])
    assert float(n.max()) <= 1.0 + 2e-7


def test_second_moment_dequantizes_strictly_positive():
    rng = np.random.default_rng(4)
    v = (rng.standard_normal((50, 70)).astype(np.float32)) ** 2
    v[7, :] *= 1e-12
    v[:, 3] *= 1e6
    qv, r, c = oracle.quantize_rank1(v, TLIN)
    deq = oracle.dequantize_rank1(qv, TLIN, r, c)
    s = np.minimum(r[:, None], c[None, :])
    assert np.all(deq >= s / 16) and np.all(deq > 0)      # zero-free map: v~ >= scale/16 > 0
    qb, sb = oracle.quantize_block(v.ravel(), 128, TLIN)
    deqb = oracle.dequantize_block(qb, 128, TLIN, sb)
    assert np.all(deqb > 0)
    # the signed DE map, by contrast, has a zero: small entries collapse to exactly 0
    qd, sd = oracle.quantize_block(v.ravel(), 128, TDE)
    assert np.any(oracle.dequantize_block(qd, 128, TDE, sd) == 0)


def test_zero_scale_convention():
    x = np.zeros(300, np.float32)
    qm, sm = oracle.quantize_block(x, 128, TDE)
    assert np.all(sm == 0) and np.all(qm == 7) and TDE[7] == 0
    qv, sv = oracle.quantize_block(x, 128, TLIN)
    assert np.all(qv == 0) and np.all(oracle.dequantize_block(qv, 128, TLIN, sv) == 0)
    v = np.zeros((4, 6), np.float32)
    v[1, 2] = 5.0
    q, r, c = oracle.quantize_rank1(v, TLIN)
    assert q[1, 2] == 15 and np.all(np.delete(q.ravel(), 8) == 0)
    assert np.array_equal(oracle.dequantize_rank1(q, TLIN, r, c), v)   # zero rows / columns stay exactly zero


# ------------------------------------------------------------------ round trips

def test_round_trip_with_stored_scales_reproduces_codes():
    rng = np.random.default_rng(6)
    x = (rng.standard_normal(128 * 64 + 50) * np.exp(2 * rng.standard_normal(128 * 64 + 50))).astype(np.float32)
    q, s = oracle.quantize_block(x, 128, TDE)
    deq = oracle.dequantize_block(q, 128, TDE, s)
    q2, _ = oracle.quantize_block(deq, 128, TDE, scale=s)
    assert np.array_equal(q, q2)
    v = (x[:128 * 64].reshape(64, 128)) ** 2
    qv, r, c = oracle.quantize_rank1(v, TLIN)
    dv = oracle.dequantize_rank1(qv, TLIN, r, c)
    qv2, _, _ = oracle.quantize_rank1(dv, TLIN, r=r, c=c)
    assert np.array_equal(qv, qv2)


def test_round_trip_with_recomputed_scales():
    rng = np.random.default_rng(7)
    v = (rng.standard_normal((96, 160)).astype(np.float32)) ** 2
    qv, r, c = oracle.quantize_rank1(v, TLIN)
    dv = oracle.dequantize_rank1(qv, TLIN, r, c)
    qv2, r2, c2 = oracle.quantize_rank1(dv, TLIN)
    assert np.array_equal(r, r2) and np.array_equal(c, c2) and np.array_equal(qv, qv2)
    qb, sb = oracle.quantize_block(v.ravel(), 128, TLIN)
    db = oracle.dequantize_block(qb, 128, TLIN, sb)
    qb2, sb2 = oracle.quantize_block(db, 128, TLIN)
    assert np.array_equal(sb, sb2) and np.array_equal(qb, qb2)
    # signed DE: reproduces when the block extreme is positive (entry +1 exists) ...
    x = rng.standard_normal(128 * 32).astype(np.float32)
    blocks = x.reshape(32, 128)
    idx = np.argmax(np.abs(blocks), axis=1)
    blocks[np.arange(32), idx] = np.abs(blocks[np.arange(32), idx])
    q, s = oracle.quantize_block(blocks.ravel(), 128, TDE)
    d = oracle.dequantize_block(q, 128, TDE, s)
    q2, s2 = oracle.quantize_block(d, 128, TDE)
    assert np.array_equal(s, s2) and np.array_equal(q, q2)
    # ... and shrinks the scale to 0.8875 s when it is negative (-1 is not in the table)
    blocks[np.arange(32), idx] *= -1
    q, s = oracle.quantize_block(blocks.ravel(), 128, TDE)
    d = oracle.dequantize_block(q, 128, TDE, s)
    _, s2 = oracle.quantize_block(d, 128, TDE)
    has_top = np.any(q.reshape(32, 128) == 15, axis=1)        # another entry rounded up to +1
    want = np.where(has_top, s, s * np.float32(0.8875))
    assert np.any(~has_top)
    np.testing.assert_allclose(s2, want, rtol=3e-7)


def test_reciprocal_versus_true_division_agree_up_to_threshold_cases():
    rng = np.random.default_rng(8)
    x = (rng.standard_normal(128 * 2048) * np.exp(rng.standard_normal(128 * 2048))).astype(np.float32)
    q0, _ = oracle.quantize_block(x, 128, TDE, true_division=False)
    q1, _ = oracle.quantize_block(x, 128, TDE, true_division=True)
    diff = q0.astype(int) - q1.astype(int)
    assert np.mean(diff != 0) < 1e-5 and np.max(np.abs(diff)) <= 1
    v = (x.reshape(512, 512)) ** 2
    a, _, _ = oracle.quantize_rank1(v, TLIN, true_division=False)
    b, _, _ = oracle.quantize_rank1(v, TLIN, true_division=True)
    diff = a.astype(int) - b.astype(int)
    assert np.mean(diff != 0) < 1e-5 and np.max(np.abs(diff)) <= 1


# ------------------------------------------------------------------ packing and the two writings

def test_pack_unpack_layout():
    codes = np.array([1, 2, 3, 4, 15, 0, 9], np.uint8)
    for impl in (oracle, onp):
        p = impl.pack4(codes)
        assert p.tolist() == [0x21, 0x43, 0x0F, 0x09]                 # even element -> low nibble
        assert np.array_equal(impl.unpack4(p, 7), codes)
    rng = np.random.default_rng(9)
    c = rng.integers(0, 16, 1001).astype(np.uint8)
    assert np.array_equal(oracle.unpack4(oracle.pack4(c), 1001), c)
    assert len(oracle.pack4(c)) == 501


def test_c_and_numpy_writings_agree_on_quantizers():
    rng = np.random.default_rng(10)
    x = (rng.standard_normal(128 * 300 + 77) * np.exp(2 * rng.standard_normal(128 * 300 + 77))).astype(np.float32)
    for T in (TDE, TLIN):
        for td in (False, True):
            xin = x if T is TDE else np.abs(x)
            a, sa = oracle.quantize_block(xin, 128, T, true_division=td)
            b, sb = onp.quantize_block(xin, 128, T, true_division=td)
            assert np.array_equal(a, b) and np.array_equal(sa, sb)
    v = (x[:240 * 160].reshape(240, 160)) ** 2
    for td in (False, True):
        a, ra, ca = oracle.quantize_rank1(v, TLIN, true_division=td)
        b, rb, cb = onp.quantize_rank1(v, TLIN, true_division=td)
        assert np.array_equal(a, b) and np.array_equal(ra, rb) and np.array_equal(ca, cb)


def test_bf16_widening_is_exact():
    import torch
    t = torch.randn(1000, dtype=torch.float32).to(torch.bfloat16)
    bits = t.view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(oracle.bf16_bits_to_f32(bits), t.float().numpy())


def test_kind_rule():
    assert oracle.kind_of(64, 64, 2) == oracle.FP32            # 4096 elements: not quantized
    assert oracle.kind_of(4097, 1, 1) == oracle.BLOCK
    assert oracle.kind_of(65, 64, 2) == oracle.RANK1
    assert oracle.kind_of(1, 8192, 2) == oracle.BLOCK          # an extent of 1 counts as 1-D
    assert oracle.kind_of(8192, 1, 2) == oracle.BLOCK
    assert oracle.kind_of(4096, 1, 1, force=1) == oracle.BLOCK
    assert oracle.kind_of(128, 128, 2, force=2) == oracle.FP32
    assert oracle.kind_of(100, 100, 2, min_quant_numel=0) == oracle.RANK1
