"""The allocation-free rank-1 quantizer against the ordinary one (collected last on purpose).

lpmm_quantize_rank1_noalloc serves callers that cannot obtain device memory when they call (all GPU
memory already owned by a framework pool, a fixed memory budget, no cudaMalloc allowed because it
synchronizes the device): its only intermediate buffer is a fixed array inside the library. The test
drives it through the C ABI twice in a row - a large problem, then a smaller one that leaves stale
values from the first call in the shared array - and requires the same bytes and scales as
lpmm_quantize, bit for bit, which is the tolerance the other quantizer tests use.
"""
import numpy as np
import pytest
import torch

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


def test_noalloc_matches_quantize_on_two_calls_in_a_row():
    for call, (rows, cols) in enumerate([(1500, 2048), (257, 129)]):
        x = _input(rows, cols, 100 + call)
        want_codes, want_r, want_c = lpmm.quantize(x, lpmm.NORM_RANK1, lpmm.MAP_LINEAR_NOZERO)
        codes = torch.full(((rows * cols + 1) // 2,), 0xAB, dtype=torch.uint8, device="cuda")
        r = torch.full((rows,), 7.0, device="cuda")
        c = torch.full((cols,), 7.0, device="cuda")
        before = torch.cuda.memory_allocated()
        lpmm.quantize_rank1_noalloc(x, codes, r, c)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == before          # the binding allocated nothing either
        assert torch.equal(r, want_r) and torch.equal(c, want_c), f"call {call}: scales differ"
        assert torch.equal(codes, want_codes), f"call {call}: codes differ"
        assert len(np.unique(codes.cpu().numpy())) > 16             # not a degenerate comparison


def test_noalloc_rejects_sizes_beyond_its_capacity():
    L = lpmm.lib()
    big = lpmm.NOALLOC_MAX_SCALES
    # host-side check only: nothing is launched and the pointers are never touched
    assert L.lpmm_quantize_rank1_noalloc(0x1000, big, 8, 0x1000, 0x1000, 0x1000, None) == lpmm.ERR_TOO_LARGE
    assert L.lpmm_quantize_rank1_noalloc(0x1000, 8, big, 0x1000, 0x1000, 0x1000, None) == lpmm.ERR_TOO_LARGE
    assert L.lpmm_quantize_rank1_noalloc(None, 8, 8, 0x1000, 0x1000, 0x1000, None) == lpmm.ERR_INVALID_ARG
    assert b"capacity" in L.lpmm_status_string(lpmm.ERR_TOO_LARGE)
