"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle on the same seeded inputs.

Bar: packed codes and scales bit for bit; parameters within 1e-6 * max(|w|, lr) after one step from a
shared state; over a 100-step trajectory parameters within 1e-4 and at most 1e-6 of the codes off by
one adjacent code (none is expected: the state path never reads the parameters).
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2309_01507_b200 import lpmm, workloads
from paper_2309_01507_b200.workloads import TensorSpec
from parity_util import ORACLE_KIND, Pair, hyper_of

pytestmark = pytest.mark.gpu

TDE = oracle.de_map(4, True)
TLIN = oracle.linear_map(4)

# Both orders of the work inside a step (maxima pass and update pass as separate launches, or one fused launch whose
# tiles wait for one another) must give the same bits: the tests of the default quantizers run under each.
SCHEDULES = pytest.mark.parametrize("schedule", [lpmm.SCHEDULE_TWO_PASS, lpmm.SCHEDULE_FUSED], ids=["two_pass", "fused"])


# ... and, on lists with several rank-1 tensors, the overlapped form of the two-pass schedule (two streams, three groups).
SCHEDULES3 = pytest.mark.parametrize("schedule", [lpmm.SCHEDULE_TWO_PASS, lpmm.SCHEDULE_FUSED, lpmm.SCHEDULE_OVERLAP],
                                     ids=["two_pass", "fused", "overlap"])


def _launches(schedule, two_pass):
    return 1 if schedule == lpmm.SCHEDULE_FUSED else two_pass


def _mat(r, c, **kw):
    return TensorSpec(f"m{r}x{c}", r, c, 2, **kw)


def _vec(n, **kw):
    return TensorSpec(f"v{n}", n, 1, 1, **kw)


# ------------------------------------------------------------------ stand-alone quantizer

def _threshold_probe():
    pts = [0.0, -0.0, 1.0, -1.0, 1.5, -1.5, 1e-30, -1e-30, 1e-45]
    for T in (TDE, TLIN):
        for a, b in zip(T[:-1], T[1:]):
            p = np.float32((float(a) + float(b)) / 2)
            for _ in range(6):
                p = np.nextafter(p, np.float32(-np.inf), dtype=np.float32)
            for _ in range(13):
                pts.append(float(p))
                p = np.nextafter(p, np.float32(np.inf), dtype=np.float32)
        pts += [float(t) for t in T]
    rng = np.random.default_rng(0)
    pts += list(rng.uniform(-1.1, 1.1, 3000))
    x = np.array(pts, dtype=np.float32)
    pad = (-x.size) % 128
    return np.concatenate([x, np.zeros(pad, np.float32)])


@pytest.mark.parametrize("map_, T", [(lpmm.MAP_DE_SIGNED, TDE), (lpmm.MAP_LINEAR_NOZERO, TLIN)])
def test_nearest_entry_at_every_threshold(map_, T):
    x = _threshold_probe()
    ones = torch.ones(x.size // 128, device="cuda")
    codes, _, _ = lpmm.quantize(torch.from_numpy(x).cuda(), lpmm.NORM_BLOCK, map_, 128, scales=(ones, None))
    want, _ = oracle.quantize_block(x, 128, T, scale=np.ones(x.size // 128, np.float32))
    assert np.array_equal(codes.cpu().numpy(), oracle.pack4(want))


@pytest.mark.parametrize("numel,block", [(1, 128), (127, 128), (128, 128), (129, 128), (50265, 128), (5000, 2048),
                                         (128 * 2000 + 3, 128), (2048 * 37 + 1111, 2048)])
@pytest.mark.parametrize("map_", [lpmm.MAP_DE_SIGNED, lpmm.MAP_LINEAR_NOZERO])
def test_block_quantizer_matches_oracle(numel, block, map_):
    rng = np.random.default_rng(numel)
    x = (rng.standard_normal(numel) * np.exp(2 * rng.standard_normal(numel))).astype(np.float32)
    if map_ == lpmm.MAP_LINEAR_NOZERO:
        x = x * x
    T = TDE if map_ == lpmm.MAP_DE_SIGNED else TLIN
    codes, s0, _ = lpmm.quantize(torch.from_numpy(x).cuda(), lpmm.NORM_BLOCK, map_, block)
    want, ws = oracle.quantize_block(x, block, T)
    assert np.array_equal(s0.cpu().numpy(), ws)
    assert np.array_equal(codes.cpu().numpy(), oracle.pack4(want))
    deq = lpmm.dequantize(codes, s0, None, numel, 1, lpmm.NORM_BLOCK, map_, block)
    assert np.array_equal(deq.cpu().numpy(), oracle.dequantize_block(want, block, T, ws))
    # round trip with the stored scales reproduces every code
    codes2, _, _ = lpmm.quantize(deq, lpmm.NORM_BLOCK, map_, block, scales=(s0, None))
    assert torch.equal(codes, codes2)


@pytest.mark.parametrize("rows,cols", [(2, 3), (1, 300), (300, 1), (37, 53), (96, 256), (513, 1000), (1024, 4096)])
def test_rank1_quantizer_matches_oracle(rows, cols):
    rng = np.random.default_rng(rows * 31 + cols)
    x = (rng.standard_normal((rows, cols)) * np.exp(rng.standard_normal((rows, 1))) *
         np.exp(rng.standard_normal((1, cols)))).astype(np.float32) ** 2
    x[rng.random((rows, cols)) < 0.01] = 0
    if rows > 4:
        x[3, :] = 0
    codes, r, c = lpmm.quantize(torch.from_numpy(x).cuda(), lpmm.NORM_RANK1, lpmm.MAP_LINEAR_NOZERO)
    want, wr, wc = oracle.quantize_rank1(x, TLIN)
    assert np.array_equal(r.cpu().numpy(), wr) and np.array_equal(c.cpu().numpy(), wc)
    assert np.array_equal(codes.cpu().numpy(), oracle.pack4(want))
    deq = lpmm.dequantize(codes, r, c, rows, cols, lpmm.NORM_RANK1, lpmm.MAP_LINEAR_NOZERO)
    ref = oracle.dequantize_rank1(want, TLIN, wr, wc)
    assert np.array_equal(deq.cpu().numpy().reshape(rows, cols), ref)
    assert np.all(ref[np.minimum(wr[:, None], wc[None, :]) > 0] > 0)     # zero-free map
    # recomputed scales reproduce themselves and the codes (Rank-1/Linear round trip)
    codes2, r2, c2 = lpmm.quantize(deq.reshape(rows, cols).contiguous(), lpmm.NORM_RANK1, lpmm.MAP_LINEAR_NOZERO)
    assert torch.equal(r, r2) and torch.equal(c, c2) and torch.equal(codes, codes2)


def _hot_path_probe():
    """Gradients that put the step's own quantizers (the table-driven signed search and the round-up linear rule) on,
    just below and just above every decision threshold: with beta1 = beta2 = 0, Eq. 1 gives m_t = g and v_t = g*g."""
    pts = []
    for a, b in zip(TDE[:-1], TDE[1:]):                      # first moment: g itself around each midpoint
        p = np.float32((float(a) + float(b)) / 2)
        for _ in range(6):
            p = np.nextafter(p, np.float32(-np.inf), dtype=np.float32)
        for _ in range(13):
            pts.append(float(p))
            p = np.nextafter(p, np.float32(np.inf), dtype=np.float32)
    for a, b in zip(TLIN[:-1], TLIN[1:]):                    # second moment: g around the square root of each midpoint
        p = np.float32(np.sqrt((float(a) + float(b)) / 2))
        for _ in range(8):
            p = np.nextafter(p, np.float32(-np.inf), dtype=np.float32)
        for _ in range(17):
            pts.append(float(p))
            pts.append(-float(p))
            p = np.nextafter(p, np.float32(np.inf), dtype=np.float32)
    pts += [float(t) for t in TDE] + [0.0, -0.0, 1e-30, -1e-30, 1e-45, 0.99999994, -0.99999994]
    rng = np.random.default_rng(1)
    pts += list(rng.uniform(-1.0, 1.0, 2000))
    return np.array(pts, dtype=np.float32)


@pytest.mark.parametrize("layout", ["vector", "long_vector", "matrix"])
@pytest.mark.parametrize("step_kind", ["adamw_two_pass", "adamw_fused", "sgdm"])
def test_step_quantizers_at_every_threshold(layout, step_kind):
    # One 1.0 per 128-block (and per row and column of the matrix) makes every scale exactly 1, so n = m_t and n = v_t.
    x = _hot_path_probe()
    per = 127
    nblk = -(-x.size // per)
    if layout == "long_vector":
        nblk = max(nblk, 65536 // 128)                      # long enough to be folded onto the tiled path
    g = np.zeros((nblk, 128), np.float32)
    g[:, 0] = 1.0
    flat = np.resize(x, nblk * per)
    g[:, 1:] = flat.reshape(nblk, per)
    if layout == "matrix":
        g[0, :] = 1.0                                       # every column maximum is 1 as well
        spec = _mat(nblk, 128, force_quant=True)
    else:
        spec = _vec(nblk * 128, force_quant=True)
    gt = torch.from_numpy(g.reshape(spec.shape)).cuda()
    w = torch.zeros(spec.shape, device="cuda")
    sched = lpmm.SCHEDULE_FUSED if step_kind == "adamw_fused" else lpmm.SCHEDULE_TWO_PASS
    st = lpmm.state_init(lpmm.default_config(schedule=sched), [spec])
    kind = ORACLE_KIND[lpmm.state_view(st, 0)["kind"]]
    ost = oracle.state_init(spec.rows, spec.cols, kind)
    w_ref = np.zeros(spec.numel, np.float32)
    if step_kind == "sgdm":
        lpmm.sgdm4_step(st, [w], [gt], lr=0.0, beta=0.0)
        oracle.sgdm4_step(w_ref, g.ravel(), ost, lr=0.0, beta=0.0)
        names = ("m_codes", "m_scale")
    else:
        hyper = dict(lr=0.0, beta1=0.0, beta2=0.0, eps=1e-8, weight_decay=0.0)
        lpmm.adamw4_step(st, [w], [gt], step=1, **hyper)
        oracle.adamw4_step(w_ref, g.ravel(), ost, step=1, **hyper)
        names = ("m_codes", "m_scale", "v_codes", "v_s0", "v_s1")
    torch.cuda.synchronize()
    view = lpmm.state_view(st, 0)
    assert np.all(ost.m_scale == 1.0)
    for name in names:
        ref = getattr(ost, name)
        if ref is not None:
            assert np.array_equal(view[name].cpu().numpy(), ref), name
    assert len(np.unique(oracle.unpack4(ost.m_codes, spec.numel))) == 16


# ------------------------------------------------------------------ the fused step

@SCHEDULES
@pytest.mark.parametrize("update_math", [lpmm.UPDATE_FAST, lpmm.UPDATE_IEEE])
def test_single_matrix_config_ten_steps(update_math, schedule):
    wl = workloads.single_matrix()
    pair = Pair(wl.tensors, hyper_of(wl), workload_index=wl.index, config=lpmm.default_config(update_math=update_math),
                schedule=schedule)
    assert pair.state.schedule == schedule
    kinds = [lpmm.state_view(pair.state, i)["kind"] for i in range(2)]
    assert kinds == [lpmm.KIND_RANK1, lpmm.KIND_BLOCK]          # bias forced onto the quantized 1-D path
    seen_v, seen_m = set(), set()
    for t in range(1, wl.steps + 1):
        pair.step(t, pair.grads_for(t))
        # IEEE update math follows the oracle's operation order: parameters are then bit-identical too
        pair.compare(tol=1e-6, exact_params=(update_math == lpmm.UPDATE_IEEE))
        seen_m |= set(np.unique(oracle.unpack4(pair.ostate[0].m_codes, 1024 * 4096)).tolist())
        seen_v |= set(np.unique(oracle.unpack4(pair.ostate[0].v_codes, 1024 * 4096)).tolist())
    assert seen_m == set(range(16)) and seen_v == set(range(16))
    assert pair.state.last_launches == _launches(schedule, 4)     # two-pass: maxima, reciprocals, tiled update, the bias' own update kernel


@pytest.mark.parametrize("grad_dtype,update_math", [(torch.float32, lpmm.UPDATE_FAST), (torch.bfloat16, lpmm.UPDATE_FAST),
                                                    (torch.float32, lpmm.UPDATE_IEEE)])
@SCHEDULES3
def test_shape_zoo_multi_tensor(grad_dtype, update_math, schedule):
    specs = [_mat(96, 256), _mat(33, 77), _mat(5, 1000), _mat(130, 384), _mat(64, 1024), _mat(8, 2048),
             _mat(1, 8192), _mat(8192, 1), _mat(300, 640), _mat(257, 129), _mat(70, 128),
             _vec(50265), _vec(4097), _vec(4096), _vec(4096, force_quant=True), _vec(1), _vec(300),
             _mat(16, 16), _mat(64, 64), _mat(65, 64), _vec(12345), _mat(77, 1992), _mat(260, 264)]
    hyper = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01)
    pair = Pair(specs, hyper, grad_dtype=grad_dtype, workload_index=7, config=lpmm.default_config(update_math=update_math),
                schedule=schedule)
    for t in range(1, 6):
        grads = pair.grads_for(t, outlier_p=0.0 if t % 2 == 0 else 1e-3)
        if t == 3:
            for g in grads[:4]:
                g[: max(1, g.shape[0] // 3)] = 0           # zero rows
            grads[11].zero_()                              # an all-zero gradient
        if t == 4:
            grads[0][5, 7] = 3.0e4                         # one huge outlier
            grads[3].mul_(1e-18)                           # second moments in the denormal range
            grads[9].mul_(1e-18)
            grads[12].mul_(1e-18)
        pair.step(t, grads)
        pair.compare(tol=1e-6)
    assert pair.state.schedule == schedule


@pytest.mark.parametrize("m_block,grad_dtype", [(128, torch.float32), (128, torch.bfloat16), (2048, torch.bfloat16),
                                                (2048, torch.float32)])
def test_block_mode_for_matrices(m_block, grad_dtype):
    # Block-wise second moments on matrices (the B128/Linear rows of the ablation, Tab. 1), with both first-moment block
    # sizes and both gradient types: matrices whose rows hold whole blocks ride the tiled kernel, the others the
    # element-indexed one.
    cfg = lpmm.default_config(v_mode=lpmm.V_BLOCK, m_block=m_block)
    specs = [_mat(96, 256), _mat(133, 77), _mat(512, 1024), _mat(24, 4096), _mat(64, 2048), _vec(70016)]
    hyper = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0)
    pair = Pair(specs, hyper, config=cfg, workload_index=8, grad_dtype=grad_dtype)
    assert all(lpmm.state_view(pair.state, i)["kind"] == lpmm.KIND_BLOCK for i in range(len(specs)))
    for t in range(1, 4):
        pair.step(t, pair.grads_for(t, outlier_p=0.0 if t == 2 else 1e-3))
        pair.compare(tol=1e-6)
    assert pair.state.last_launches == 2     # no maxima pass at all: the tiled update kernel and the element-indexed one


@pytest.mark.parametrize("grad_dtype", [torch.float32, torch.bfloat16])
def test_first_moment_block_2048(grad_dtype):
    # B2048 for m (the block size of the 8-bit optimizers, Sec. 2.2) with rank-1 / B128 v as before.
    cfg = lpmm.default_config(m_block=2048)
    specs = [_mat(64, 2048), _mat(24, 4096), _mat(130, 384), _mat(96, 256), _mat(33, 77), _vec(50265), _vec(4097),
             _vec(2048 * 3, force_quant=True), _mat(40, 1024)]
    hyper = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01)
    pair = Pair(specs, hyper, config=cfg, grad_dtype=grad_dtype, workload_index=11)
    for t in range(1, 5):
        pair.step(t, pair.grads_for(t, outlier_p=0.0 if t % 2 == 0 else 1e-3))
        pair.compare(tol=1e-6)
    assert pair.ostate[0].m_scale.size == 64     # one scale per 2048 elements


@SCHEDULES3
def test_transformer_base_three_steps_one_launch_per_pass(schedule):
    wl = workloads.transformer_base()
    pair = Pair(wl.tensors, hyper_of(wl), workload_index=wl.index, schedule=schedule)
    kinds = [lpmm.state_view(pair.state, i)["kind"] for i in range(len(wl.tensors))]
    assert kinds.count(lpmm.KIND_RANK1) == 61 and kinds.count(lpmm.KIND_FP32) == 120
    for t in range(1, 4):
        pair.step(t, pair.grads_for(t))
        pair.compare(tol=1e-6)
    # two-pass: maxima + reciprocals + update cover all 181 tensors (the small fp32 ones ride in the tiled update kernel);
    # overlapped: the same three per group of tensors
    assert pair.state.last_launches == {lpmm.SCHEDULE_TWO_PASS: 3, lpmm.SCHEDULE_FUSED: 1, lpmm.SCHEDULE_OVERLAP: 9}[schedule]


@SCHEDULES
def test_sparse_token_rows_and_lm_head_bias(schedule):
    # RoBERTa-shaped slice: token-sparse embedding gradients (90% of rows zero) and the odd-length 50265 bias.
    specs = [TensorSpec("emb.word", 50265, 1024, 2, sparse_rows=0.9), TensorSpec("emb.pos", 514, 1024, 2),
             TensorSpec("emb.type", 1, 1024, 2), _vec(1024), TensorSpec("fc1", 4096, 1024, 2),
             TensorSpec("head.bias", 50265, 1, 1)]
    hyper = dict(lr=1e-5, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01)
    pair = Pair(specs, hyper, workload_index=2, schedule=schedule)
    for t in range(1, 4):
        pair.step(t, pair.grads_for(t))
        pair.compare(tol=1e-6)
    r = pair.ostate[0].v_s0
    assert np.sum(r == 0) > 0.5 * r.size * 0.9 ** 3      # rows never touched keep scale 0 and dequantize to 0


@SCHEDULES
def test_trajectory_100_steps(schedule):
    specs = [_mat(256, 1024), _vec(8192)]
    hyper = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01)
    pair = Pair(specs, hyper, workload_index=5, schedule=schedule)
    for t in range(1, 101):
        pair.step(t, pair.grads_for(t))
        if t % 25 == 0 or t < 3:
            pair.compare(tol=1e-4, share_params=False)       # oracle keeps its own fp32 trajectory
    pair.compare(tol=1e-4, share_params=False)


@pytest.mark.parametrize("sched_a,sched_b", [(lpmm.SCHEDULE_TWO_PASS, lpmm.SCHEDULE_TWO_PASS), (lpmm.SCHEDULE_FUSED, lpmm.SCHEDULE_FUSED),
                                             (lpmm.SCHEDULE_TWO_PASS, lpmm.SCHEDULE_FUSED), (lpmm.SCHEDULE_FUSED, lpmm.SCHEDULE_TWO_PASS)])
def test_checkpoint_attach_resumes_bit_exactly(sched_a, sched_b):
    # 50 steps, save, 50 more; against: restore the copy (into a state that may run the other schedule) and 50 steps.
    specs = [_mat(128, 512), _mat(130, 384), _vec(5000), _vec(100)]
    hyper = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01)
    a = Pair(specs, hyper, workload_index=6, schedule=sched_a)
    for t in range(1, 51):
        lpmm.adamw4_step(a.state, a.params, a.grads_for(t), step=t, **hyper)
    saved = a.state.arena.clone()
    phase = a.state.phase
    params_copy = [p.clone() for p in a.params]
    for t in range(51, 101):
        lpmm.adamw4_step(a.state, a.params, a.grads_for(t), step=t, **hyper)
    cfg_b = lpmm.default_config(schedule=sched_b)
    arena_b = torch.zeros(lpmm.state_bytes(cfg_b, specs), dtype=torch.uint8, device="cuda")
    k = min(saved.numel(), arena_b.numel())
    arena_b[:k] = saved[:k]
    resumed = lpmm.state_attach(cfg_b, specs, arena_b, phase)
    assert resumed.schedule == sched_b
    for t in range(51, 101):
        lpmm.adamw4_step(resumed, params_copy, a.grads_for(t), step=t, **hyper)
    torch.cuda.synchronize()
    assert lpmm.device_status(a.state) == 0 and lpmm.device_status(resumed) == 0
    for i in range(len(specs)):
        va, vb = lpmm.state_view(a.state, i), lpmm.state_view(resumed, i)
        for k in ("m_codes", "m_scale", "v_codes", "v_s0", "v_s1", "m32", "v32"):
            if va[k] is not None:
                assert torch.equal(va[k], vb[k]), (i, k)
        assert torch.equal(a.params[i], params_copy[i])


def test_fused_state_interleaved_with_two_pass_steps():
    # A state on the fused schedule also serves the entry points that always run two-pass (the bfloat16 copy, the
    # host-buffer step); the two kinds of step hand the rotating statistics buffers and their "cleared" status to each
    # other. Every step is checked against the oracle.
    specs = [_mat(128, 512), _mat(130, 384), _mat(33, 77), _mat(5, 1000), _vec(5000), _vec(100)]
    hyper = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01)
    pair = Pair(specs, hyper, workload_index=19, schedule=lpmm.SCHEDULE_FUSED)
    copies = [torch.empty(s.numel, dtype=torch.bfloat16, device="cuda") for s in specs]
    nbytes = lpmm.stage_bytes(pair.state)
    dp = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    dg = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    for t in range(1, 10):
        grads = pair.grads_for(t)
        if t in (3, 4, 8):          # two-pass with the bfloat16 copy
            lpmm.adamw4_step(pair.state, pair.params, grads, step=t, params_bf16=copies, **hyper)
            launches = pair.state.last_launches
            assert launches > 1
        elif t == 6:                # two-pass through host buffers
            h_params = [p.detach().cpu().pin_memory() for p in pair.params]
            h_grads = [g.cpu().pin_memory() for g in grads]
            lpmm.adamw4_step_host(pair.state, h_params, h_grads, dp, dg, step=t, **hyper)
            torch.cuda.synchronize()
            for p, h in zip(pair.params, h_params):
                p.copy_(h.reshape(p.shape))
        else:
            lpmm.adamw4_step(pair.state, pair.params, grads, step=t, **hyper)
            assert pair.state.last_launches == 1
        for i, g in enumerate(grads):
            oracle.adamw4_step(pair.w_ref[i], g.float().cpu().numpy().ravel(), pair.ostate[i], step=t, **hyper)
        torch.cuda.synchronize()
        pair.compare(tol=1e-6)


def test_fused_work_list_invariants():
    # The fused launch's correctness rests on its host-built list: every tile of either pass exactly once, and every
    # update tile of a rank-1 tensor behind all of that tensor's maxima tiles (its CTA waits for them; items are handed
    # out in list order). The list lies behind the states in the arena: two words per item (tensor | flags, tile).
    for wl, kw in ((workloads.transformer_base(), {}), (workloads.single_matrix(), {}),
                   (workloads.transformer_base(), dict(lead_melems=1, gap_items=7, tile_elems=4096, tile_elems_maxima=8192))):
        cfg = lpmm.default_config(schedule=lpmm.SCHEDULE_FUSED, **kw)
        st = lpmm.state_init(cfg, wl.tensors)
        torch.cuda.synchronize()
        states_end = lpmm.state_bytes(lpmm.default_config(schedule=lpmm.SCHEDULE_TWO_PASS, **kw), wl.tensors)
        words = st.arena[states_end:].view(torch.int32).cpu().numpy().view(np.uint32).reshape(-1, 2)
        tensor = words[:, 0] & 0x0fffffff
        update = (words[:, 0] & 0x40000000) != 0
        keep = (words[:, 0] & 0x80000000) != 0
        kinds = [lpmm.state_view(st, i)["kind"] for i in range(len(wl.tensors))]
        seen = {}
        last_maxima, first_update = {}, {}
        pos = 0
        for pos in range(len(words)):
            t, u, tile = int(tensor[pos]), bool(update[pos]), int(words[pos, 1])
            if t >= len(wl.tensors):
                break
            key = (t, u, tile)
            if key in seen:
                break                      # padding behind the list (zeros repeat item (0, maxima, 0))
            seen[key] = pos
            if u:
                first_update.setdefault(t, pos)
            else:
                last_maxima[t] = pos
                assert kinds[t] == lpmm.KIND_RANK1
        for t, k in enumerate(kinds):
            ups = sorted(tile for (tt, u, tile) in seen if tt == t and u)
            assert ups == list(range(len(ups))) and len(ups) > 0, t          # every update tile once, none missing
            mxs = sorted(tile for (tt, u, tile) in seen if tt == t and not u)
            assert mxs == list(range(len(mxs)))
            if k == lpmm.KIND_RANK1:
                assert len(mxs) > 0 and last_maxima[t] < first_update[t], t  # dependency order
            else:
                assert len(mxs) == 0
        assert not np.any(keep & update)                                     # only maxima tiles carry the keep flag


def test_attach_refuses_an_arena_that_is_something_else():
    specs = [_mat(128, 512), _vec(5000)]
    cfg = lpmm.default_config()
    st = lpmm.state_init(cfg, specs)
    torch.cuda.synchronize()
    good = st.arena.clone()
    assert lpmm.state_attach(cfg, specs, good.clone(), 0).n == 2
    cases = {
        "not an arena": torch.zeros_like(good),
        "other shapes": (good.clone(), [_mat(128, 512), _vec(5001)]),
        "other block size": (good.clone(), specs, lpmm.default_config(m_block=2048)),
    }
    for name, case in cases.items():
        arena, shp, c = (case, specs, cfg) if torch.is_tensor(case) else (case + (cfg,))[:3]
        big = torch.zeros(max(arena.numel(), lpmm.state_bytes(c, shp)), dtype=torch.uint8, device="cuda")
        big[:arena.numel()] = arena
        with pytest.raises(lpmm.LpmmError) as ei:
            lpmm.state_attach(c, shp, big, 0)
        assert ei.value.status == lpmm.ERR_INVALID_ARG, name
    bad_version = good.clone()
    bad_version[36] += 1                 # the layout-version word of the header
    with pytest.raises(lpmm.LpmmError) as ei:
        lpmm.state_attach(cfg, specs, bad_version, 0)
    assert ei.value.status == lpmm.ERR_INVALID_ARG
    with pytest.raises(lpmm.LpmmError) as ei:
        lpmm.state_attach(cfg, specs, good.clone(), 3)       # phases are 0, 1, 2
    assert ei.value.status == lpmm.ERR_INVALID_ARG


def test_bounded_wait_gives_up_and_reports():
    # The fused schedule's CTAs wait for one another with a limit; here two CTAs wait for a counter nothing advances.
    st = lpmm.state_init(lpmm.default_config(schedule=lpmm.SCHEDULE_FUSED), [_mat(128, 512)])
    gave_up, word = lpmm.selftest_wait(st)
    assert gave_up == 2 and word == 2
    assert lpmm.device_status(st) == 0          # the self-test cleans up after itself
    p = torch.zeros(128, 512, device="cuda")
    g = torch.ones(128, 512, device="cuda")
    lpmm.adamw4_step(st, [p], [g], step=1, lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0)
    torch.cuda.synchronize()
    assert lpmm.device_status(st) == 0 and torch.all(p < 0)


def test_host_buffer_step_matches_device_step():
    specs = [_mat(128, 512), _vec(5000), _vec(100)]
    hyper = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01)
    a = Pair(specs, hyper, workload_index=4)
    b_state = lpmm.state_init(a.config, specs)
    h_params = [p.detach().cpu().pin_memory() for p in a.params]
    nbytes = lpmm.stage_bytes(b_state)
    dp = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    dg = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    for t in range(1, 4):
        grads = a.grads_for(t)
        a.step(t, grads)
        h_grads = [g.cpu().pin_memory() for g in grads]
        lpmm.adamw4_step_host(b_state, h_params, h_grads, dp, dg, step=t, **hyper)
        torch.cuda.synchronize()
        for i in range(len(specs)):
            assert torch.equal(h_params[i], a.params[i].cpu())


def test_argument_errors_do_not_launch():
    cfg = lpmm.default_config()
    st = lpmm.state_init(cfg, [_mat(64, 128)])
    p = torch.zeros(64, 128, device="cuda")
    g = torch.zeros(64, 128, device="cuda")
    ok = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0)
    for bad in (dict(step=0), dict(step=1, beta1=1.0), dict(step=1, lr=-1.0), dict(step=1, eps=float("nan"))):
        with pytest.raises(lpmm.LpmmError) as ei:
            lpmm.adamw4_step(st, [p], [g], **{**ok, "step": 1, **bad})
        assert ei.value.status == lpmm.ERR_INVALID_ARG
    flat = torch.zeros(64 * 128 + 4, device="cuda")
    with pytest.raises(lpmm.LpmmError) as ei:
        lpmm.adamw4_step(st, [flat[1:64 * 128 + 1]], [g], step=1, **ok)
    assert ei.value.status == lpmm.ERR_ALIGNMENT
    with pytest.raises(lpmm.LpmmError) as ei:
        lpmm.quantize(p, lpmm.NORM_RANK1, lpmm.MAP_DE_SIGNED)
    assert ei.value.status == lpmm.ERR_UNSUPPORTED
    torch.cuda.synchronize()
    assert torch.count_nonzero(p) == 0


@pytest.mark.parametrize("grad_dtype,m_block", [(torch.float32, 128), (torch.bfloat16, 128), (torch.float32, 2048)])
def test_sgdm_step_matches_oracle_bit_for_bit(grad_dtype, m_block):
    # Alg. 2 (compressed SGDM): the first moment in 4 bits, parameters in the algorithm's own operation order.
    cfg = lpmm.default_config(m_block=m_block)
    specs = [_mat(96, 256), _mat(33, 77), _mat(130, 384), _mat(64, 2048), _vec(50265), _vec(4097), _vec(300), _vec(1)]
    params = [workloads.make_param(s, 12, i, device="cuda") for i, s in enumerate(specs)]
    state = lpmm.state_init(cfg, specs)
    w_ref = [p.cpu().numpy().ravel().copy() for p in params]
    ost = [oracle.state_init(s.rows, s.cols, oracle.FP32 if lpmm.state_view(state, i)["kind"] == lpmm.KIND_FP32 else oracle.BLOCK,
                             m_block=m_block) for i, s in enumerate(specs)]
    for t in range(1, 6):
        grads = [workloads.make_grad(s, 12, i, t, device="cuda", dtype=grad_dtype) for i, s in enumerate(specs)]
        lpmm.sgdm4_step(state, params, grads, lr=0.01, beta=0.9)
        torch.cuda.synchronize()
        for i, s in enumerate(specs):
            oracle.sgdm4_step(w_ref[i], grads[i].float().cpu().numpy().ravel(), ost[i], lr=0.01, beta=0.9)
            view = lpmm.state_view(state, i)
            for name in ("m_codes", "m_scale", "m32"):
                ref = getattr(ost[i], name)
                if ref is not None:
                    assert np.array_equal(view[name].cpu().numpy(), ref), (s.name, name, t)
            assert np.array_equal(params[i].cpu().numpy().ravel(), w_ref[i]), (s.name, t)
    assert state.last_launches == 1


@pytest.mark.parametrize("grad_dtype,m_block", [(torch.float32, 128), (torch.bfloat16, 128), (torch.bfloat16, 2048)])
def test_factorized_second_moment_matches_oracle(grad_dtype, m_block):
    # "4-bit Factor": m in 4 bits (bit-exact), v reconstructed from fp32 row/column statistics. The GPU adds the squares
    # in binary32 inside a tile (a lane's eight in order, a shuffle tree per row strip, compensated sums down a column)
    # and the tiles' partial sums in binary64 in a fixed order; the oracle adds everything in binary64. R, C therefore
    # agree within a few ulp (1e-6 relative). Parameters: within 1e-6 of the larger of |w|, lr and the step the element
    # took - with a factorized v an outlier gradient moves a parameter by many times lr (v_ij is not g_ij^2), and the
    # few-ulp difference in v scales with that step; 1-D and small tensors behave as in the default mode.
    cfg = lpmm.default_config(v_mode=lpmm.V_FACTORED, m_block=m_block)
    specs = [_mat(96, 256), _mat(40, 1024), _mat(130, 384), _mat(33, 77), _vec(50265), _vec(300), _mat(64, 128)]
    if m_block == 2048:      # rows must hold whole first-moment blocks
        specs = [_mat(24, 4096), _mat(40, 2048), _mat(7, 6144), _mat(33, 77), _vec(50265), _vec(300), _mat(64, 2048)]
    hyper = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01)
    params = [workloads.make_param(s, 13, i, device="cuda") for i, s in enumerate(specs)]
    state = lpmm.state_init(cfg, specs)
    kinds = [lpmm.state_view(state, i)["kind"] for i in range(len(specs))]
    assert kinds == [lpmm.KIND_FACTORED, lpmm.KIND_FACTORED, lpmm.KIND_FACTORED, lpmm.KIND_FP32, lpmm.KIND_BLOCK,
                     lpmm.KIND_FP32, lpmm.KIND_FACTORED]
    w_ref = [p.cpu().numpy().ravel().copy() for p in params]
    ost, Rs, Cs = [], [], []
    for i, s in enumerate(specs):
        k = {lpmm.KIND_FACTORED: oracle.RANK1, lpmm.KIND_FP32: oracle.FP32, lpmm.KIND_BLOCK: oracle.BLOCK}[kinds[i]]
        ost.append(oracle.state_init(s.rows, s.cols, k, m_block=m_block))
        Rs.append(np.zeros(s.rows, np.float32)); Cs.append(np.zeros(s.cols, np.float32))
    for t in range(1, 6):
        grads = [workloads.make_grad(s, 13, i, t, device="cuda", dtype=grad_dtype) for i, s in enumerate(specs)]
        lpmm.adamw4_step(state, params, grads, step=t, **hyper)
        torch.cuda.synchronize()
        assert lpmm.device_status(state) == 0
        for i, s in enumerate(specs):
            g = grads[i].float().cpu().numpy().ravel()
            view = lpmm.state_view(state, i)
            w_prev = w_ref[i].copy()
            if kinds[i] == lpmm.KIND_FACTORED:
                oracle.adamw4_factor_step(w_ref[i], g, ost[i], Rs[i], Cs[i], step=t, **hyper)
                assert view["v_codes"] is None
                np.testing.assert_allclose(view["v_s0"].cpu().numpy(), Rs[i], rtol=1e-6, atol=0)
                np.testing.assert_allclose(view["v_s1"].cpu().numpy(), Cs[i], rtol=1e-6, atol=0)
                tol = 1e-6
            else:
                oracle.adamw4_step(w_ref[i], g, ost[i], step=t, **hyper)
                tol = 1e-6
            for name in ("m_codes", "m_scale", "m32", "v32"):
                ref = getattr(ost[i], name)
                if ref is not None:
                    assert np.array_equal(view[name].cpu().numpy(), ref), (s.name, name, t)
            w = params[i].cpu().numpy().ravel()
            scale = np.maximum(np.maximum(np.abs(w_ref[i]), hyper["lr"]), np.abs(w_ref[i] - w_prev))
            err = np.max(np.abs(w - w_ref[i]) / scale)
            assert err <= tol, (s.name, t, err)
            w_ref[i][:] = w
    assert state.last_launches == 4      # sums pass, finalize kernel, tiled update, element-indexed / fp32 update
    # a matrix whose rows do not hold whole first-moment blocks is refused in this mode
    with pytest.raises(lpmm.LpmmError) as ei:
        lpmm.state_init(cfg, [_mat(257, 129)])
    assert ei.value.status == lpmm.ERR_UNSUPPORTED


def test_factorized_statistics_are_reproducible_bit_for_bit():
    # Partial sums are written per tile and added in a fixed order (no floating-point atomics): two runs from the same
    # inputs give identical bits, on a matrix large enough for many tiles and a ragged last one.
    cfg = lpmm.default_config(v_mode=lpmm.V_FACTORED)
    specs = [_mat(3000, 4096), _mat(1111, 1408), _vec(50265)]
    hyper = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01)
    runs = []
    for _ in range(2):
        params = [workloads.make_param(s, 18, i, device="cuda") for i, s in enumerate(specs)]
        state = lpmm.state_init(cfg, specs)
        for t in range(1, 4):
            grads = [workloads.make_grad(s, 18, i, t, device="cuda") for i, s in enumerate(specs)]
            lpmm.adamw4_step(state, params, grads, step=t, **hyper)
        torch.cuda.synchronize()
        views = [lpmm.state_view(state, i) for i in range(2)]
        runs.append((params, [(v["v_s0"].clone(), v["v_s1"].clone(), v["m_codes"].clone()) for v in views]))
    for i in range(2):
        for x, y in zip(runs[0][1][i], runs[1][1][i]):
            assert torch.equal(x, y)
    for x, y in zip(runs[0][0], runs[1][0]):
        assert torch.equal(x, y)
    # and against the oracle's binary64 sums on the large matrix
    g = workloads.make_grad(specs[0], 18, 0, 1, device="cuda")
    st = lpmm.state_init(cfg, specs[:1])
    p = workloads.make_param(specs[0], 18, 0, device="cuda")
    lpmm.adamw4_step(st, [p], [g], step=1, **hyper)
    torch.cuda.synchronize()
    gg = (g.cpu().numpy().astype(np.float32) ** 2).astype(np.float64)
    omb2 = np.float32(1) - np.float32(0.999)
    want_r = (omb2 * gg.sum(axis=1).astype(np.float32)).astype(np.float32)
    want_c = (omb2 * gg.sum(axis=0).astype(np.float32)).astype(np.float32)
    v = lpmm.state_view(st, 0)
    np.testing.assert_allclose(v["v_s0"].cpu().numpy(), want_r, rtol=1e-6, atol=0)
    np.testing.assert_allclose(v["v_s1"].cpu().numpy(), want_c, rtol=1e-6, atol=0)


def _nd(*dims):
    rows = int(np.prod(dims[:-1]))
    return workloads.TensorSpec("t" + "x".join(map(str, dims)), rows, dims[-1], len(dims), dims=tuple(dims))


@SCHEDULES3
@pytest.mark.parametrize("grad_dtype,update_math", [(torch.float32, lpmm.UPDATE_IEEE), (torch.bfloat16, lpmm.UPDATE_FAST)])
def test_tensors_with_three_and_four_axes_match_oracle(grad_dtype, update_math, schedule):
    # Alg. 4 in its general form: one vector of maxima per axis, scale = minimum over the element's axes.
    # Codes, block scales and every axis' statistics bit-exact; parameters bit-exact with IEEE update math,
    # within 1e-6 * max(|w|, lr) with the approximate one. A matrix rides along to cover mixed lists.
    cfg = lpmm.default_config(update_math=update_math, schedule=schedule, overlap_groups=3)
    # (under the two-pass schedule the tensors whose trailing axes multiply to whole 128-blocks - the last five - run on
    # the tiled kernels as composite matrices with expanded statistics; the others, and all of them under the fused
    # schedule, on the element-indexed ones)
    specs = [_nd(6, 10, 200), _nd(3, 5, 7, 64), _nd(16, 33, 9), _mat(96, 256), _nd(2, 4099, 3), _nd(1, 40, 128),
             _nd(4, 6, 256), _nd(3, 4, 8, 128), _nd(5, 3, 384), _nd(37, 128, 3, 3)]
    hyper = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01)
    params = [workloads.make_param(s, 14, i, device="cuda") for i, s in enumerate(specs)]
    state = lpmm.state_init(cfg, specs)
    assert all(lpmm.state_view(state, i)["kind"] == lpmm.KIND_RANK1 for i in range(len(specs)))
    w_ref = [p.cpu().numpy().ravel().copy() for p in params]
    ref = []
    for s in specs:
        dims = s.shape
        ref.append(dict(m_codes=np.full((s.numel + 1) // 2, 0x77, np.uint8), m_scale=np.zeros((s.numel + 127) // 128, np.float32),
                        v_codes=np.zeros((s.numel + 1) // 2, np.uint8), mu=np.zeros(int(sum(dims)), np.float32)))
        if s.numel % 2:
            ref[-1]["m_codes"][-1] = 0x07
    for t in range(1, 5):
        grads = [workloads.make_grad(s, 14, i, t, device="cuda", dtype=grad_dtype) for i, s in enumerate(specs)]
        lpmm.adamw4_step(state, params, grads, step=t, **hyper)
        torch.cuda.synchronize()
        assert lpmm.device_status(state) == 0
        for i, s in enumerate(specs):
            r = ref[i]
            oracle.adamw4_step_nd(w_ref[i], grads[i].float().cpu().numpy().ravel(), s.shape, 128, r["m_codes"], r["m_scale"],
                                  r["v_codes"], r["mu"], step=t, **hyper)
            view = lpmm.state_view(state, i)
            for name in ("m_codes", "m_scale", "v_codes"):
                assert np.array_equal(view[name].cpu().numpy(), r[name]), (s.name, name, t)
            mu = np.concatenate([lpmm.state_view_axis(state, i, a).cpu().numpy() for a in range(len(s.shape))])
            assert np.array_equal(mu, r["mu"]), (s.name, "mu", t)
            w = params[i].cpu().numpy().ravel()
            if update_math == lpmm.UPDATE_IEEE:
                assert np.array_equal(w, w_ref[i]), (s.name, t)
            else:
                err = np.max(np.abs(w - w_ref[i]) / np.maximum(np.abs(w_ref[i]), hyper["lr"]))
                assert err <= 1e-6, (s.name, t, err)
                w_ref[i][:] = w
    with pytest.raises(lpmm.LpmmError) as ei:      # five axes: not supported
        lpmm.state_init(cfg, [_nd(2, 2, 2, 2, 300)])
    assert ei.value.status == lpmm.ERR_UNSUPPORTED


@pytest.mark.parametrize("grad_dtype,m_block,schedule", [(torch.bfloat16, 128, lpmm.SCHEDULE_AUTO), (torch.float32, 2048, lpmm.SCHEDULE_AUTO),
                                                         (torch.bfloat16, 128, lpmm.SCHEDULE_TWO_PASS)])
def test_bf16_copy_of_the_parameters(grad_dtype, m_block, schedule):
    # lpmm_adamw4_step_bf16w: states and fp32 parameters exactly as the plain step leaves them, plus a bfloat16 copy
    # that is the nearest-even rounding of the new fp32 parameters, on every kind of tensor and on ragged tails.
    # (AUTO puts this small list on the fused schedule for the plain step, so the two states also compare the schedules;
    # under TWO_PASS the tensors with three axes whose trailing axes fill 128-blocks are composite matrices in both)
    cfg = lpmm.default_config(m_block=m_block, schedule=schedule)
    specs = [_mat(96, 256), _mat(64, 2048), _mat(130, 384), _mat(33, 77), _mat(257, 129), _vec(50265), _vec(4097), _vec(300), _vec(1),
             _nd(6, 10, 200), _nd(5, 3, 384), _vec(196608)]      # the last one is folded into rows and updated by a launch of its own
    hyper = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01)
    pa = [workloads.make_param(s, 15, i, device="cuda") for i, s in enumerate(specs)]
    pb = [p.clone() for p in pa]
    copies = [torch.full((s.numel,), -7.0, dtype=torch.bfloat16, device="cuda") for s in specs]
    sa, sb = lpmm.state_init(cfg, specs), lpmm.state_init(cfg, specs)
    for t in range(1, 4):
        grads = [workloads.make_grad(s, 15, i, t, device="cuda", dtype=grad_dtype) for i, s in enumerate(specs)]
        lpmm.adamw4_step(sa, pa, grads, step=t, **hyper)
        lpmm.adamw4_step(sb, pb, grads, step=t, params_bf16=copies, **hyper)
        torch.cuda.synchronize()
        assert lpmm.device_status(sb) == 0
        for i, s in enumerate(specs):
            assert torch.equal(pa[i], pb[i]), (s.name, t)
            va, vb = lpmm.state_view(sa, i), lpmm.state_view(sb, i)
            for name in ("m_codes", "m_scale", "v_codes", "m32", "v32"):
                if va[name] is not None:
                    assert torch.equal(va[name], vb[name]), (s.name, name, t)
            want = oracle.f32_to_bf16_bits(pb[i].cpu().numpy().ravel())
            got = copies[i].view(torch.int16).cpu().numpy().view(np.uint16)
            assert np.array_equal(got, want), (s.name, t)
    # (the bfloat16 copy always runs the two-pass schedule: maxima, reciprocals, tiled update, element-indexed update, and
    # the folded tensor's own update launch; three more small kernels where a composite tensor is present)
    assert sb.last_launches == (8 if schedule == lpmm.SCHEDULE_TWO_PASS else 5)
    # refused with the factorized second moment, and with a missing pointer array
    sf = lpmm.state_init(lpmm.default_config(v_mode=lpmm.V_FACTORED), [_mat(96, 256)])
    with pytest.raises(lpmm.LpmmError) as ei:
        lpmm.adamw4_step(sf, [pa[0]], [grads[0]], step=1, params_bf16=[copies[0]], **hyper)
    assert ei.value.status == lpmm.ERR_UNSUPPORTED


@SCHEDULES
@pytest.mark.parametrize("grad_dtype", [torch.bfloat16, torch.float32])
def test_pointers_aligned_to_16_but_not_32_bytes_give_the_same_result(grad_dtype, schedule):
    # The tiled update pass moves a lane's eight fp32 values with one 256-bit access when every pointer is 32-byte
    # aligned and with two 128-bit accesses otherwise; both must leave identical parameters and states.
    cfg = lpmm.default_config(schedule=schedule)
    specs = [_mat(96, 256), _mat(64, 1024), _mat(130, 384), _vec(5000)]
    hyper = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01)
    pa = [workloads.make_param(s, 16, i, device="cuda") for i, s in enumerate(specs)]
    store = [torch.empty(s.numel + 16, device="cuda") for s in specs]           # fp32: 4 elements = 16 bytes
    pb = [b[4:4 + s.numel] for b, s in zip(store, specs)]
    for a, b in zip(pa, pb):
        b.copy_(a.ravel())
        assert a.data_ptr() % 32 == 0 and b.data_ptr() % 32 == 16
    sa, sb = lpmm.state_init(cfg, specs), lpmm.state_init(cfg, specs)
    for t in range(1, 4):
        grads = [workloads.make_grad(s, 16, i, t, device="cuda", dtype=grad_dtype) for i, s in enumerate(specs)]
        per = 16 // grads[0].element_size()
        gstore = [torch.empty(s.numel + 2 * per, device="cuda", dtype=grad_dtype) for s in specs]
        gb = [b[per:per + s.numel] for b, s in zip(gstore, specs)]
        for g, b in zip(grads, gb):
            b.copy_(g.ravel())
        lpmm.adamw4_step(sa, pa, grads, step=t, **hyper)
        lpmm.adamw4_step(sb, pb, gb, step=t, **hyper)
        torch.cuda.synchronize()
        for i, s in enumerate(specs):
            assert torch.equal(pa[i].ravel(), pb[i]), (s.name, t)
            va, vb = lpmm.state_view(sa, i), lpmm.state_view(sb, i)
            for name in ("m_codes", "m_scale", "v_codes", "v_s0", "v_s1"):
                if va[name] is not None:
                    assert torch.equal(va[name], vb[name]), (s.name, name, t)


@pytest.mark.parametrize("grad_dtype,m_block,v_mode", [(torch.bfloat16, 128, lpmm.V_RANK1), (torch.float32, 128, lpmm.V_BLOCK),
                                                       (torch.float32, 2048, lpmm.V_RANK1)])
def test_long_one_dimensional_tensors_folded_into_rows(grad_dtype, m_block, v_mode):
    # 1-D tensors of at least 65536 elements whose length is a multiple of 128 (2048 with B2048) are folded into rows
    # and take the tiled update path (in a state that is not block-wise: in a launch of their own); block-wise
    # quantization does not see the folding, so codes and scales must equal the oracle's 1-D result bit for bit.
    cfg = lpmm.default_config(m_block=m_block, v_mode=v_mode)
    specs = [_vec(196608), _vec(70016 if m_block == 128 else 67584), _vec(65536 + 2048 * 5), _mat(96, 256), _vec(66000), _vec(300)]
    hyper = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01)
    pair = Pair(specs, hyper, grad_dtype=grad_dtype, config=cfg, workload_index=17)
    for t in range(1, 5):
        grads = pair.grads_for(t, outlier_p=0.0 if t % 2 == 0 else 1e-3)
        if t == 3:
            grads[0][:70000] = 0
        pair.step(t, grads)
        pair.compare(tol=1e-6)
    # two-pass: maxima + reciprocal + update (+ the folded tensors' own update launch); this small list of the default
    # quantizers runs the fused schedule: one launch + the folded tensors' own
    want = {(128, lpmm.V_RANK1): 2, (2048, lpmm.V_RANK1): 5}.get((m_block, v_mode), 2)
    assert pair.state.last_launches == want
