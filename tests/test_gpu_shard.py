"""Sample-sharded calibration on one GPU: two contexts stand for two ranks that
each hold half of the calibration samples (run one after the other; nothing
waits on anything).  amax pass per rank, maximum over ranks, scoring with that
amax, R-weighted merge of the per-layer rows: equal to one context over all
samples, and to the oracle.  Also the power-of-two scale mode."""
import numpy as np
import pytest
import torch

from helpers import assert_close, compare_layer, oracle_layer
from paper_2505_13060_b200 import shard, synth

pytestmark = pytest.mark.gpu

E4M3 = 1


class _View:
    pass


def _rank_view(lt, r0, r1):
    """The tensors a rank holding samples r0..r1-1 sees."""
    v = _View()
    sp = lt.spec
    v.spec = synth.LayerSpec(sp.name, sp.kind, r1 - r0, sp.dtype,
                             synth.OperandSpec((r1 - r0,) + tuple(sp.op0.shape[1:]), True),
                             synth.OperandSpec(sp.op1.shape, False))
    v.values = [lt.values[0][r0:r1].contiguous(), lt.values[1]]
    v.grads = [lt.grads[0][r0:r1].contiguous(), lt.grads[1][r0:r1].contiguous()]
    return v


def test_two_sample_shards_equal_one_context(ampq, orc):
    specs = synth.llama7b_block(32)[:3] + synth.toy_mlp(R=4, tokens=64, width=128, layers=1)
    lts = [synth.make_layer(s, "cuda", seed=14, layer=i) for i, s in enumerate(specs)]
    F = 2
    st = torch.cuda.current_stream().cuda_stream
    ranks = []
    for r0, r1 in ((0, 1), (1, 4)):   # unequal shards: 1 and 3 samples
        ctx = ampq.Context(0, st)
        views = [_rank_view(lt, r0, r1) for lt in lts]
        ids = []
        for v in views:
            lid = ctx.register_layer(v.spec.kind, v.spec.name, v.spec.R)
            ampq.bind_layer_tensors(ctx, lid, v)
            ids.append(lid)
        ctx.measure_amax()
        ranks.append((ctx, ids, views, np.stack([ctx.get_amax(i) for i in ids]), r1 - r0))
    amax = np.maximum(ranks[0][3], ranks[1][3])   # what reduce_amax returns over two ranks
    tables = []
    for ctx, ids, views, _, Rl in ranks:
        for k, lid in enumerate(ids):
            for op in range(2):
                ctx.set_amax(lid, op, float(amax[k, op]))
        ctx.score()
        tables.append((np.stack([shard.layer_row(ctx.get_layer(i), F) for i in ids]), Rl))
    merged = ampq.merge_sample_tables(np.stack([t for t, _ in tables]), [R for _, R in tables])   # what merge_sample_rows calls
    one = ampq.Context(0, st)
    oid = []
    for lt in lts:
        lid = one.register_layer(lt.spec.kind, lt.spec.name, lt.spec.R)
        ampq.bind_layer_tensors(one, lid, lt)
        oid.append(lid)
    one.score()
    for k, (lid, lt) in enumerate(zip(oid, lts)):
        ref = oracle_layer(orc, lt, [E4M3])
        got = compare_layer(ampq, one, lid, ref, F, lt.spec.name)
        assert got["amax"].tobytes() == amax[k].tobytes()
        assert_close(merged[k], shard.layer_row(got, F), "merged rows of " + lt.spec.name, tol=1e-12)
    for ctx, *_ in ranks:
        ctx.destroy()
    # measure_amax alone, then get_amax before any score; state errors
    one.set_amax(oid[0], 0, 3.0)
    one.measure_amax()
    assert one.get_amax(oid[0])[0] == np.float32(3.0) and one.get_amax(oid[1]).tobytes() == amax[1].tobytes()
    assert ampq.lib().ampq_get_layer(one._h, oid[0], *([None] * 8)) == ampq.ERR_STATE   # amax only, nothing scored
    one.destroy()


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_power_of_two_scale_mode(ampq, orc, dtype):
    specs = [synth.LayerSpec("p2", synth.LINEAR, 2, dtype,
                             synth.OperandSpec((2, 50001), True, 1.0, 1e-3, "normal", ("element", 0.01, 20.0)),
                             synth.OperandSpec((70001,), False, 0.02, 1e-3))]
    lt = synth.make_layer(specs[0], "cuda", seed=15)
    ctx = ampq.Context(0, torch.cuda.current_stream().cuda_stream)
    ctx.set_formats([0, 1, 2])
    ctx.set_scale_mode(ampq.SCALE_POW2)
    lid = ctx.register_layer(ampq.LINEAR, "p2", 2)
    ampq.bind_layer_tensors(ctx, lid, lt)
    ctx.score()
    got = ctx.get_layer(lid)
    segs = []
    for k, op in enumerate((lt.spec.op0, lt.spec.op1)):
        v, g = synth.to_numpy(lt.values[k]), synth.to_numpy(lt.grads[k])
        a, sc, iv, seg = orc.score_operand(v.reshape(2, -1) if op.per_sample else v.reshape(-1), g.reshape(2, -1), 2,
                                           op.per_sample, [1, 2], pow2=True)
        assert got["amax"][k] == a and got["scale"][k, 1:].tobytes() == sc.tobytes()
        assert got["inv_scale"][k, 1:].tobytes() == iv.tobytes()
        assert_close(ctx.get_operand(lid, k), seg, "pow2 operand %d" % k)
        segs.append(seg)
    ref = orc.layer_combine(segs[0], segs[1], [0, 1, 2])
    assert_close(got["d_meas"], ref["d_meas"], "pow2 d_meas")
    # exhaustive amax values around the m = 1.75 boundary and at the range ends
    z = torch.zeros(8, dtype=torch.float32, device="cuda")
    for a in [448.0, np.nextafter(np.float32(448.0), np.float32(1e9)), 447.99, 1.75, 1.7500001, 1e-38, 3e38, 1e-44, 2.0 ** -119]:
        for f in (1, 2):
            c2 = ampq.Context(0, torch.cuda.current_stream().cuda_stream)
            c2.set_formats([0, f])
            c2.set_scale_mode(ampq.SCALE_POW2)
            l2 = c2.register_layer(ampq.LINEAR, "a", 1)
            for k in range(2):
                c2.bind_operand(l2, k, ampq.F32, z.data_ptr(), 8, False, z.data_ptr(), 8)
                c2.set_amax(l2, k, float(np.float32(a)))
            c2.score()
            r = c2.get_layer(l2)
            sc, iv = orc.scales(f, np.float32(a), pow2=True)
            assert r["scale"][0, 1] == sc and r["inv_scale"][0, 1] == iv, (a, f)
            c2.destroy()
    ctx.destroy()
