"""The allocation-free rank-1 quantizer against the CPU oracle and the ordinary entry point (collected last on purpose).

lpmm_quantize_rank1_noalloc serves callers that cannot obtain device memory when they call (all GPU
memory already owned by a framework pool, a fixed memory budget, no cudaMalloc allowed because it
synchronizes the device): its only intermediate buffer is a fixed array inside the library. The test
drives it through the C ABI twice in a row - a large problem, then a smaller one that leaves stale
values from the first call in the shared array - and requires, bit for bit (the tolerance of the other
quantizer tests), the oracle's rank-1 statistics and packed codes (Sec. 4.2 normalization, Sec. 4.1 linear
map), which are also what lpmm_quantize returns.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2309_01507_b200 import lpmm

pytestmark = pytest.mark.gpu


def _input(rows, cols, seed):
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)
    x = torch.randn(rows, cols, generator=g, device="cuda")
    x = x * torch.exp(torch.randn(rows, 1, generator=g, device="cuda")) * torch.exp(torch.randn(1, cols, generator=g, device="cuda"))
    x = x * x
    x[rows // 3, :] = 0          # a zero row: its maximum is 0 and its reciprocal must be 0, not inf
    return x.contiguous()


def test_noalloc_matches_oracle_and_quantize_on_two_calls_in_a_row():
    tlin = oracle.linear_map(4)
    for call, (rows, cols) in enumerate([(1500, 2048), (257, 129)]):
        x = _input(rows, cols, 100 + call)
        o_codes, o_r, o_c = oracle.quantize_rank1(x.cpu().numpy(), tlin)          # the checker: CPU, from the paper
        want_codes, want_r, want_c = lpmm.quantize(x, lpmm.NORM_RANK1, lpmm.MAP_LINEAR_NOZERO)
        codes = torch.full(((rows * cols + 1) // 2,), 0xAB, dtype=torch.uint8, device="cuda")
        r = torch.full((rows,), 7.0, device="cuda")
        c = torch.full((cols,), 7.0, device="cuda")
        before = torch.cuda.memory_allocated()
        lpmm.quantize_rank1_noalloc(x, codes, r, c)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == before          # the binding allocated nothing either
        assert np.array_equal(r.cpu().numpy(), o_r) and np.array_equal(c.cpu().numpy(), o_c), f"call {call}: scales differ from the oracle's"
        assert np.array_equal(codes.cpu().numpy(), oracle.pack4(o_codes)), f"call {call}: codes differ from the oracle's"
        assert torch.equal(r, want_r) and torch.equal(c, want_c), f"call {call}: scales differ from lpmm_quantize's"
        assert torch.equal(codes, want_codes), f"call {call}: codes differ from lpmm_quantize's"
        assert len(np.unique(codes.cpu().numpy())) > 16             # not a degenerate comparison


def test_noalloc_rejects_sizes_beyond_its_capacity():
    L = lpmm.lib()
    big = lpmm.NOALLOC_MAX_SCALES
    # host-side check only: nothing is launched and the pointers are never touched
    assert L.lpmm_quantize_rank1_noalloc(0x1000, big, 8, 0x1000, 0x1000, 0x1000, None) == lpmm.ERR_TOO_LARGE
    assert L.lpmm_quantize_rank1_noalloc(0x1000, 8, big, 0x1000, 0x1000, 0x1000, None) == lpmm.ERR_TOO_LARGE
    assert L.lpmm_quantize_rank1_noalloc(None, 8, 8, 0x1000, 0x1000, 0x1000, None) == lpmm.ERR_INVALID_ARG
    assert b"capacity" in L.lpmm_status_string(lpmm.ERR_TOO_LARGE)


def test_binding_checks_the_buffers_before_calling_the_library():
    x = _input(64, 96, 7)
    codes = torch.empty(64 * 96 // 2, dtype=torch.uint8, device="cuda")
    r, c = torch.empty(64, device="cuda"), torch.empty(96, device="cuda")
    for bad in (dict(x=x.t()), dict(x=x.double()), dict(x=x[0]), dict(codes=codes[:-1]), dict(r=r[:-1]), dict(c=c[::2]),
                dict(c=c.cpu()), dict(codes=codes.float())):
        args = dict(x=x, codes=codes, r=r, c=c)
        args.update(bad)
        with pytest.raises(ValueError):
            lpmm.quantize_rank1_noalloc(args["x"], args["codes"], args["r"], args["c"])
