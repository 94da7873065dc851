"""The no-allocation entry point against the ordinary one.

``ampq_score_segment_noalloc`` serves callers that may not allocate device
memory (another library owns the heap, or an allocation would stall the
device): it keeps its tables and per-tile partial sums in a fixed array inside
the library instead of a workspace from cudaMalloc.  It must give what
``ampq_score`` gives for the same segment.  Each case calls it twice in a row,
because the array is shared by all calls and keeps what the last call left.
This file sorts last so that a run that stops at the first failure has already
run every other test.
"""
import numpy as np
import pytest
import torch

from helpers import REL_TOL, assert_close
from paper_2505_13060_b200 import synth

pytestmark = pytest.mark.gpu

E4M3, E5M2 = 1, 2


def _reference(ampq, values, grads, fmt, amax):
    """[S, D, amax] of one segment through ampq_score (R = 1, second operand empty)."""
    ctx = ampq.Context(0, torch.cuda.current_stream().cuda_stream)
    ctx.set_formats([0, fmt])
    lid = ctx.register_layer(ampq.LINEAR, "segment", 1)
    code = ampq.torch_dtype_code(values)
    n = values.numel()
    ctx.bind_operand(lid, 0, code, values.data_ptr(), n, True, grads.data_ptr(), n)
    ctx.bind_operand(lid, 1, code, 0, 0, False, 0, 0)
    if amax >= 0:
        ctx.set_amax(lid, 0, amax)
    ctx.score()
    seg = ctx.get_operand(lid, 0)[0]
    a = float(ctx.get_layer(lid)["amax"][0])
    ctx.destroy()
    return np.array([seg[0], seg[1], a])


def _noalloc(ampq, values, grads, fmt, amax, out):
    ampq.score_segment_noalloc(0, torch.cuda.current_stream().cuda_stream, ampq.torch_dtype_code(values), fmt,
                               values.data_ptr(), grads.data_ptr(), values.numel(), amax, out.data_ptr())
    torch.cuda.synchronize()
    return out.cpu().numpy().copy()


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_noalloc_matches_score_twice_in_a_row(ampq, orc, dtype):
    g = torch.Generator(device="cuda").manual_seed(11)
    out = torch.empty(3, dtype=torch.float64, device="cuda")
    cases = [(2 * 524288 + 12345, E4M3, -1.0), (70001, E5M2, -1.0), (524288, E4M3, 2.5), (7, E5M2, -1.0), (0, E4M3, -1.0)]
    for n, fmt, amax in cases:
        v = torch.empty(max(n, 1), dtype=dtype, device="cuda").normal_(0, 1, generator=g)[:n]
        gr = (torch.empty(max(n, 1), dtype=dtype, device="cuda").normal_(0, 1, generator=g) * 1e-3)[:n]
        want = _reference(ampq, v, gr, fmt, amax)
        got1 = _noalloc(ampq, v, gr, fmt, amax, out)   # the very first call also does the one-time set-up
        out.fill_(-1.0)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        got2 = _noalloc(ampq, v, gr, fmt, amax, out)
        assert torch.cuda.mem_get_info()[0] == free_before   # the call took no device memory
        for got in (got1, got2):
            assert got[2] == want[2], (n, fmt, got, want)          # amax: exact
            assert_close(got[:2], want[:2], "no-alloc [S, D] n=%d fmt=%d" % (n, fmt), tol=REL_TOL)
        assert got1.tobytes() == got2.tobytes()
        if n:   # and the oracle itself, not only the entry point that was checked against it
            a, _, _, seg = orc.score_operand(synth.to_numpy(v).reshape(1, -1), synth.to_numpy(gr).reshape(1, -1), 1, True,
                                             [fmt], amax_preset=None if amax < 0 else amax)
            assert got1[2] == float(a)
            assert_close(got1[:2], seg[0], "no-alloc against the oracle n=%d fmt=%d" % (n, fmt), tol=REL_TOL)


def test_noalloc_refuses_what_does_not_fit(ampq):
    out = torch.empty(3, dtype=torch.float64, device="cuda")
    buf = torch.zeros(16, dtype=torch.float32, device="cuda")
    L = ampq.lib()
    st = torch.cuda.current_stream().cuda_stream
    too_many = ampq.NOALLOC_MAX_NUMEL + 1   # refused before any launch: the pointers are never read
    assert L.ampq_score_segment_noalloc(0, st, ampq.F32, E4M3, buf.data_ptr(), buf.data_ptr(), too_many, -1.0,
                                        out.data_ptr()) == ampq.ERR_TOO_LARGE
    with pytest.raises(ampq.AmpqError, match="at most"):
        ampq.score_segment_noalloc(0, st, ampq.F32, E4M3, buf.data_ptr(), buf.data_ptr(), too_many, -1.0, out.data_ptr())
    assert L.ampq_score_segment_noalloc(0, st, ampq.F32, 0, buf.data_ptr(), buf.data_ptr(), 16, -1.0,
                                        out.data_ptr()) == ampq.ERR_INVALID
    assert L.ampq_score_segment_noalloc(0, st, ampq.F32, E4M3, buf.data_ptr(), buf.data_ptr(), 16, -1.0,
                                        None) == ampq.ERR_INVALID
    assert L.ampq_score_segment_noalloc(0, st, ampq.F32, E4M3, buf.data_ptr() + 2, buf.data_ptr(), 8, -1.0,
                                        out.data_ptr()) == ampq.ERR_ALIGN
    bad = torch.randn(1000, device="cuda")
    bad[77] = float("nan")
    ampq.score_segment_noalloc(0, st, ampq.F32, E4M3, bad.data_ptr(), bad.data_ptr(), 1000, -1.0, out.data_ptr())
    torch.cuda.synchronize()
    r = out.cpu().numpy()
    assert np.isnan(r[0]) and np.isnan(r[1])
