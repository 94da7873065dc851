"""Triangular (causal) operands: declaring the zero triangle must change no
result -- amax and scales bit for bit and the sums to 1e-6 against the dense run
of the same library (the same terms in another order), within the usual
tolerance against the oracle (which always reads everything) -- for short and
long rows, both element types, and the cases that fall back to the dense path."""
import numpy as np
import pytest
import torch

from helpers import assert_close, compare_layer, oracle_layer
from paper_2505_13060_b200 import synth

pytestmark = pytest.mark.gpu

E4M3, E5M2 = 1, 2


def _layer(R, H, T, dtype, seed):
    """An (P, V)-shaped BGEMM layer: P = causal softmax [R, H, T, T], V [R, H, T, 64]."""
    spec = synth.LayerSpec("av", synth.BGEMM, R, dtype,
                           synth.OperandSpec((R, H, T, T), True, 1.0, 1e-4, "causal_softmax"),
                           synth.OperandSpec((R, H, T, 64), True, 1.0, 1e-4))
    return synth.make_layer(spec, "cuda", seed=seed)


def _score(ampq, lt, fmts, T, offset=0):
    ctx = ampq.Context(0, torch.cuda.current_stream().cuda_stream)
    ctx.set_formats(list(fmts))
    lid = ctx.register_layer(lt.spec.kind, lt.spec.name, lt.spec.R)
    ampq.bind_layer_tensors(ctx, lid, lt)
    if T:
        ctx.set_causal(lid, 0, T)
    ctx.score()
    out = (ctx.get_layer(lid), ctx.get_operand(lid, 0), ctx.get_operand(lid, 1), ctx.last_launch_count())
    return ctx, lid, out


@pytest.mark.parametrize("dtype,R,H,T", [
    (torch.bfloat16, 3, 4, 256),    # 16 rows per 8 KiB chunk
    (torch.bfloat16, 2, 3, 64),     # the smallest T: 64 rows per chunk
    (torch.bfloat16, 1, 1, 4096),   # one row per chunk
    (torch.bfloat16, 1, 1, 8192),   # two chunks per row: whole chunks are skipped
    (torch.float32, 2, 2, 512),     # fp32: 4 rows per chunk
    (torch.float32, 1, 1, 2048),    # fp32: one row per chunk
    (torch.float32, 1, 1, 4096),    # fp32: whole chunks are skipped
])
def test_causal_equals_dense_and_oracle(ampq, orc, dtype, R, H, T):
    lt = _layer(R, H, T, dtype, seed=T + R)
    assert float(lt.values[0][0, 0].triu(1).abs().max()) == 0.0
    fmts = (0, E4M3, E5M2)
    dctx, dl, dense = _score(ampq, lt, fmts, 0)
    cctx, cl, causal = _score(ampq, lt, fmts, T)
    assert causal[3] == dense[3] + 1   # the triangular operand really took its own launch
    for k in ("amax", "scale", "inv_scale"):
        assert np.asarray(dense[0][k]).tobytes() == np.asarray(causal[0][k]).tobytes(), k
    for k in ("s_per_sample", "d_meas_per_sample", "d_model", "d_meas"):   # same terms, another summation order
        assert_close(causal[0][k], dense[0][k], "causal vs dense " + k, tol=1e-6)
    assert_close(causal[1], dense[1], "causal vs dense operand 0", tol=1e-6)
    assert_close(causal[2], dense[2], "the other operand", tol=1e-6)   # untouched; its tiles may be larger
    if lt.values[0].numel() <= 1 << 24:
        compare_layer(ampq, cctx, cl, oracle_layer(orc, lt, [E4M3, E5M2], threads=8), 3, "causal T=%d" % T)
    dctx.destroy()
    cctx.destroy()


def test_causal_fallbacks_and_contract(ampq, orc):
    # T that is not a power of two, or too small: scored densely, same numbers
    lt = _layer(2, 2, 96, torch.bfloat16, seed=3)
    d = _score(ampq, lt, (0, E4M3), 0)
    c = _score(ampq, lt, (0, E4M3), 96)
    assert d[2][1].tobytes() == c[2][1].tobytes()
    c2 = _score(ampq, lt, (0, E4M3), 32)   # 96*96 is a multiple of 32*32, but 32 < 64: dense
    assert d[2][1].tobytes() == c2[2][1].tobytes()
    for x in (d, c, c2):
        x[0].destroy()
    # a slice that is not a whole number of matrices: dense
    lt = _layer(1, 1, 128, torch.bfloat16, seed=4)
    ctx = ampq.Context(0, torch.cuda.current_stream().cuda_stream)
    lid = ctx.register_layer(ampq.BGEMM, "x", 1)
    ampq.bind_layer_tensors(ctx, lid, lt)
    ctx.set_causal(lid, 0, 256)
    ctx.score()
    ref = oracle_layer(orc, lt, [E4M3])
    compare_layer(ampq, ctx, lid, ref, 2, "T does not divide")
    # misaligned slices: dense
    n = 128 * 128
    buf = torch.zeros(n + 8, dtype=torch.bfloat16, device="cuda")
    gbuf = torch.randn(n + 8, device="cuda").to(torch.bfloat16)
    buf[1:n + 1] = lt.values[0].reshape(-1)
    ctx.bind_operand(lid, 0, ampq.BF16, buf.data_ptr() + 2, n, True, gbuf.data_ptr() + 2, n)
    ctx.set_causal(lid, 0, 128)
    ctx.score()
    lt2 = _layer(1, 1, 128, torch.bfloat16, seed=4)
    lt2.grads[0] = gbuf[1:n + 1].reshape(1, 1, 128, 128)
    compare_layer(ampq, ctx, lid, oracle_layer(orc, lt2, [E4M3]), 2, "misaligned causal")
    # a broken promise (non-zero triangle) lands between the zeroed and the dense operand
    full = torch.randn(1, 2, 256, 256, device="cuda").to(torch.bfloat16).abs()
    lt3 = _layer(1, 2, 256, torch.bfloat16, seed=5)
    lt3.values[0] = full
    l3 = ctx.register_layer(ampq.BGEMM, "y", 1)
    ampq.bind_layer_tensors(ctx, l3, lt3)
    ctx.set_causal(l3, 0, 256)
    ctx.score()
    s_got = ctx.get_operand(l3, 0)[0, 0]
    s_dense = oracle_layer(orc, lt3, [E4M3])["ops"][0]["seg"][0, 0]
    lt3.values[0] = full.tril()
    s_tril = oracle_layer(orc, lt3, [E4M3])["ops"][0]["seg"][0, 0]
    assert s_tril < s_got < s_dense
    assert ampq.lib().ampq_set_causal(ctx._h, l3, 0, -1) == ampq.ERR_INVALID
    ctx.destroy()
