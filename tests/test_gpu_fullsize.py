"""GPU parity at the full sizes and launch geometry of the benchmark's
workloads: one whole Llama-7B-shaped block, one attention layer (dense and
with the causal declaration) inside a score large enough for the largest
scoring tile, and the cast of every fp32 bit pattern.  Each test checks for
free device memory first.  Run with -m gpu on a B200."""
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import pytest
import torch

from helpers import assert_close, compare_layer, gpu_codes, oracle_layer
from paper_2505_13060_b200 import synth

pytestmark = pytest.mark.gpu

E4M3, E5M2 = 1, 2
THREADS = 16


def _need(gb):
    free, _ = torch.cuda.mem_get_info()
    if free < gb * 1e9:
        pytest.skip("needs %d GB of free device memory" % gb)


def _same_as_block0(ctx, ids, per_block, blocks):
    first = [ctx.get_layer(ids[i]) for i in range(per_block)]
    for b in range(1, blocks):
        for i in range(per_block):
            got = ctx.get_layer(ids[per_block * b + i])
            for key in ("amax", "s_per_sample", "d_meas_per_sample"):
                assert first[i][key].tobytes() == got[key].tobytes(), (b, i, key)


def test_full_size_llama7b_block_whole(ampq, orc):
    """All 7 linear layers of one full-size Llama-7B-shaped block (R = 4 samples
    of 2048 tokens; 3.2 GB scored), every value against the oracle.  The block is
    bound 32 times (as the benchmark binds resident slots, pointer sharing off)
    so that the score uses the tiles of the 32-block workload: 2^21 elements."""
    import bench

    _need(12)
    specs = bench.workload_specs("llama7b")
    blocks = 32
    ctx = ampq.Context(0, torch.cuda.current_stream().cuda_stream)
    ctx.set_formats([0, E4M3, E5M2])
    slots, ids, scored = bench.bind_workload(ctx, specs, blocks, 1, torch.device("cuda", 0), seed=21)
    assert scored == blocks * sum(s.scored_bytes() for s in specs)
    ctx.score()
    assert ctx.last_tile_shift() == 21
    for i, lt in enumerate(slots[0]):
        ref = oracle_layer(orc, lt, [E4M3, E5M2], threads=THREADS)
        compare_layer(ampq, ctx, ids[i], ref, 3, "7B block " + lt.spec.name)
        assert 0.2 * ref["d_model"][1] < ref["d_meas"][1] < 1.2 * ref["d_model"][1]
    _same_as_block0(ctx, ids, len(specs), blocks)
    ctx.destroy()


@pytest.mark.parametrize("causal", [False, True])
def test_full_size_attention_layer(ampq, orc, causal):
    """One full-size attention layer (Q,K and P,V with R = 4, 32 heads, T = 2048,
    head size 128; P a causal softmax) bound 16 times so that the score takes the
    largest tile (2^21 elements, as the 32-layer workload does): dense, and with the causal declaration (tiles of a matrix are
    then visited in rotated order and only the lower triangle is read).  Both
    against the oracle, which always scores the full operand; amax and scales bit
    for bit, FP8 codes of one (sample, head) slice of P bit for bit."""
    import bench

    _need(10)
    specs = bench.workload_specs("attention")
    blocks = 16
    ctx = ampq.Context(0, torch.cuda.current_stream().cuda_stream)
    ctx.set_formats([0, E4M3])
    slots, ids, scored = bench.bind_workload(ctx, specs, blocks, 1, torch.device("cuda", 0), seed=22, causal=causal)
    ctx.score()
    assert ctx.last_tile_shift() == 21   # a 2048 x 2048 matrix spans two tiles: the rotated visiting order is in play
    dense_bytes = blocks * sum(s.scored_bytes() for s in specs)
    assert scored < 0.6 * dense_bytes if causal else scored == dense_bytes
    pb = ctx.get_pass_bytes()
    assert (pb["score"] < 0.6 * dense_bytes) if causal else (pb["score"] == dense_bytes)
    refs = []
    for i, lt in enumerate(slots[0]):
        ref = oracle_layer(orc, lt, [E4M3], threads=THREADS)
        refs.append(ref)
        compare_layer(ampq, ctx, ids[i], ref, 2, "attention " + lt.spec.name + (" causal" if causal else ""))
    _same_as_block0(ctx, ids, len(specs), blocks)
    P = slots[0][1].values[0]          # [R, heads, T, T]
    T = P.shape[-1]
    codes = torch.empty(P.numel(), dtype=torch.uint8, device="cuda")
    ctx.export_codes(ids[1], 0, E4M3, codes.data_ptr())
    torch.cuda.synchronize()
    r, h = 2, 17
    piece = codes.view(P.shape)[r, h].cpu().numpy().reshape(-1)
    want = orc.codes(synth.to_numpy(P[r, h]), E4M3, refs[1]["ops"][0]["inv"][0])
    assert np.array_equal(piece, want)
    assert (want.reshape(T, T)[np.triu_indices(T, 1)] == 0).all() and (want != 0).sum() > T
    ctx.destroy()


def test_every_fp32_bit_pattern_through_the_cast(ampq, orc):
    """All 2^32 fp32 bit patterns in 16 chunks of 2^28 (Inf/NaN patterns, which
    the contract excludes, replaced by 0), one scale that is not a power of two,
    E4M3 and E5M2: the exported codes equal the oracle's bit for bit."""
    _need(6)
    n = 1 << 28
    a = np.float32(12345.678)
    vals = torch.empty(n, dtype=torch.float32, device="cuda")
    ctx = ampq.Context(0, torch.cuda.current_stream().cuda_stream)
    ctx.set_formats([0, E4M3, E5M2])
    lid = ctx.register_layer(ampq.LINEAR, "cast32", 1)
    pieces = 32
    step = n // pieces
    with ThreadPoolExecutor(max_workers=THREADS) as pool:
        for chunk in range(16):
            bits = np.arange(n, dtype=np.uint32) + np.uint32(chunk * n)
            bits[(bits & 0x7F800000) == 0x7F800000] = 0
            host = bits.view(np.float32)
            vals.copy_(torch.from_numpy(host))
            for k in range(2):   # the gradient is irrelevant to the codes: the values stand in for it
                ctx.bind_operand(lid, k, ampq.F32, vals.data_ptr(), n, False, vals.data_ptr(), n)
                ctx.set_amax(lid, k, float(a))
            ctx.score()
            for f in (E4M3, E5M2):
                _, iv = orc.scales(f, a)
                got = gpu_codes(ctx, lid, 0, f, n)
                want = list(pool.map(lambda i: orc.codes(host[i * step:(i + 1) * step], f, iv), range(pieces)))
                assert np.array_equal(got, np.concatenate(want)), (chunk, f)
    ctx.destroy()
