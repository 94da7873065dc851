"""Sharded scoring by two processes that share the one GPU, meeting over gloo
(host tensors).  By layer: each rank scores the layers `assign_layers` gives it
with `ampq_score`, the ranks exchange the per-layer table, and each runs the
sub-graph sums and the selection.  By sample: each rank holds every layer but
only its own calibration samples; the ranks exchange the per-tensor amax (MAX)
between the amax pass and the scoring pass and merge their per-layer means
afterwards.  Tables and plans must equal those of a single process that scores
everything, and the oracle's.  The two processes' kernels are independent
(nothing waits on the other process).  Run with -m gpu."""
import json
import os
import socket
import subprocess
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
E4M3 = 1
F = 2


def _specs():
    from paper_2505_13060_b200 import synth

    return synth.llama7b_block(32, prefix="a.") + synth.llama7b_block(32, prefix="b.") + synth.attention_bgemm(16, prefix="a.")


def _groups(rng):
    groups = []
    for members in ([0, 1, 2, 3], [4, 5, 6], [7, 8, 9, 10], [11, 12, 13], [14, 15]):
        Q = np.array([[0, 1]] * len(members), dtype=np.uint8)
        groups.append((members, Q, np.array([0.0, rng.uniform(0.5, 2.0)])))
    return groups


def _score(which):
    """Scores the layers `which` (global indices) in one context on cuda:0; returns {index: row}."""
    import torch

    from paper_2505_13060_b200 import binding, shard, synth

    specs = _specs()
    ctx = binding.Context(0, torch.cuda.current_stream().cuda_stream)
    ctx.set_formats([0, E4M3])
    keep, ids = [], {}
    for i in which:
        lt = synth.make_layer(specs[i], "cuda", seed=13, layer=i)
        keep.append(lt)
        ids[i] = ctx.register_layer(lt.spec.kind, lt.spec.name, lt.spec.R)
        binding.bind_layer_tensors(ctx, ids[i], lt)
    ctx.score()
    rows = {i: shard.layer_row(ctx.get_layer(lid), F) for i, lid in ids.items()}
    bulk = ctx.get_layer_table(list(ids.values()))   # the same rows in one call
    assert all(np.array_equal(bulk[k], rows[i]) for k, i in enumerate(ids))
    ctx.destroy()
    return rows


def worker(rank, world, port, out):
    import torch.distributed as dist

    from paper_2505_13060_b200 import binding, shard

    specs = _specs()
    dist.init_process_group("gloo", init_method="tcp://127.0.0.1:%d" % port, rank=rank, world_size=world)
    owner = shard.assign_layers([s.scored_bytes() for s in specs], world)
    mine = [i for i in range(len(specs)) if owner[i] == rank]
    table = shard.gather_layer_table(_score(mine), len(specs), F)
    groups = _groups(np.random.default_rng(4))
    res = {}
    for mode in (binding.D_MODEL, binding.D_MEASURED):
        col = 1 + 1 if mode == binding.D_MODEL else 1 + F + 1
        all_low = float(np.sum(table[:, col]))
        for frac in (0.05, 0.3, 0.7):
            p, c, d = shard.select_from_table(binding, table, F, groups, mode, frac * all_low)
            res["%d_%g" % (mode, frac)] = [p.tolist(), c, d]
    dist.barrier()
    dist.destroy_process_group()
    with open(os.path.join(out, "rank%d.json" % rank), "w") as f:
        json.dump({"mine": mine, "table": table.tolist(), "res": res}, f)


def _sample_specs():
    from paper_2505_13060_b200 import synth

    return synth.llama7b_block(32)[:4] + synth.toy_mlp(R=4, tokens=64, width=128, layers=2)


def sample_worker(rank, world, port, out):
    """Rank 0 holds sample 0, rank 1 samples 1..3 of every layer (R = 4)."""
    import torch
    import torch.distributed as dist

    from paper_2505_13060_b200 import binding, shard, synth

    specs = _sample_specs()
    dist.init_process_group("gloo", init_method="tcp://127.0.0.1:%d" % port, rank=rank, world_size=world)
    r0, r1 = (0, 1) if rank == 0 else (1, 4)
    ctx = binding.Context(0, torch.cuda.current_stream().cuda_stream)
    ctx.set_formats([0, E4M3])
    keep, ids = [], []
    for i, sp in enumerate(specs):
        lt = synth.make_layer(sp, "cuda", seed=17, layer=i)   # the same tensors on both ranks; each binds its samples
        x, gx = lt.values[0][r0:r1].contiguous(), lt.grads[0][r0:r1].contiguous()
        w, gw = lt.values[1], lt.grads[1][r0:r1].contiguous()
        keep += [x, gx, w, gw]
        lid = ctx.register_layer(sp.kind, sp.name, r1 - r0)
        code = binding.torch_dtype_code(x)
        ctx.bind_operand(lid, 0, code, x.data_ptr(), x.numel(), True, gx.data_ptr(), x.numel() // (r1 - r0))
        ctx.bind_operand(lid, 1, code, w.data_ptr(), w.numel(), False, gw.data_ptr(), w.numel())
        ids.append(lid)
    ctx.measure_amax()
    amax = shard.reduce_amax(np.stack([ctx.get_amax(i) for i in ids]))
    for k, lid in enumerate(ids):
        for op in range(2):
            ctx.set_amax(lid, op, float(amax[k, op]))
    ctx.score()
    table = shard.merge_sample_rows(binding, ctx.get_layer_table(ids), r1 - r0)
    ctx.destroy()
    dist.barrier()
    dist.destroy_process_group()
    with open(os.path.join(out, "sample_rank%d.json" % rank), "w") as f:
        json.dump({"amax": amax.tolist(), "table": table.tolist()}, f)


def _spawn(tmp_path, mode):
    sock = socket.socket()
    sock.bind(("127.0.0.1", 0))
    port = sock.getsockname()[1]
    sock.close()
    procs = [subprocess.Popen([sys.executable, os.path.abspath(__file__), mode, str(r), "2", str(port), str(tmp_path)])
             for r in range(2)]
    for p in procs:
        assert p.wait(timeout=600) == 0


@pytest.mark.gpu
def test_two_processes_score_their_samples_and_merge(tmp_path, ampq, orc):
    import torch

    from helpers import REL_TOL, compare_layer, oracle_layer
    from paper_2505_13060_b200 import shard, synth

    _spawn(tmp_path, "samples")
    got = [json.load(open(tmp_path / ("sample_rank%d.json" % r))) for r in range(2)]
    assert got[0] == got[1]   # both ranks end with the same amax and the same merged table, bit for bit
    specs = _sample_specs()
    one = ampq.Context(0, torch.cuda.current_stream().cuda_stream)
    one.set_formats([0, E4M3])
    lts = [synth.make_layer(sp, "cuda", seed=17, layer=i) for i, sp in enumerate(specs)]
    ids = []
    for lt in lts:
        lid = one.register_layer(lt.spec.kind, lt.spec.name, lt.spec.R)
        ampq.bind_layer_tensors(one, lid, lt)
        ids.append(lid)
    one.score()
    whole = one.get_layer_table(ids)
    merged = np.array(got[0]["table"])
    assert np.allclose(merged, whole, rtol=1e-12, atol=0)   # a mean of means against one mean: the order of additions
    for k, (lid, lt) in enumerate(zip(ids, lts)):
        ref = oracle_layer(orc, lt, [E4M3])
        res = compare_layer(ampq, one, lid, ref, F, lt.spec.name)
        assert res["amax"].tobytes() == np.array(got[0]["amax"][k], np.float32).tobytes()
        want = shard.layer_row(ref, F)
        assert np.all(np.abs(merged[k] - want) <= REL_TOL * np.abs(want))
    one.destroy()


@pytest.mark.gpu
def test_two_processes_score_their_layers_and_meet_in_the_table(tmp_path, ampq, orc):
    import torch

    from helpers import REL_TOL, oracle_layer
    from paper_2505_13060_b200 import shard, synth

    _spawn(tmp_path, "layers")
    got = [json.load(open(tmp_path / ("rank%d.json" % r))) for r in range(2)]
    specs = _specs()
    L = len(specs)
    assert got[0]["table"] == got[1]["table"] and got[0]["res"] == got[1]["res"]
    assert sorted(got[0]["mine"] + got[1]["mine"]) == list(range(L)) and got[0]["mine"] and got[1]["mine"]
    # one process scoring everything: the same kernels on the same tensors (the tile size, and with it the
    # order of the fp64 additions, may differ with the amount scored per context)
    rows = _score(range(L))
    table = np.stack([rows[i] for i in range(L)])
    assert np.allclose(table, np.array(got[0]["table"]), rtol=1e-9, atol=0)
    # the oracle's table (within the tolerance of the fp32 sums) and its plans
    ref = np.stack([shard.layer_row(oracle_layer(orc, synth.make_layer(specs[i], "cuda", seed=13, layer=i), [E4M3],
                                                 threads=8), F) for i in range(L)])
    assert np.all(np.abs(table - ref) <= REL_TOL * np.abs(ref))
    groups = _groups(np.random.default_rng(4))
    for mode, key in ((ampq.D_MODEL, 1), (ampq.D_MEASURED, 1 + F)):
        d_tabs = [orc.group_costs(m, Q, ref[:, key:key + F]) for m, Q, _ in groups]
        all_low = float(np.sum(ref[:, key + 1]))
        for frac in (0.05, 0.3, 0.7):
            want = orc.select_bruteforce([c for _, _, c in groups], d_tabs, frac * all_low)
            p, c, d = got[0]["res"]["%d_%g" % (mode, frac)]
            assert p == want[0].tolist() and c == want[1]
    torch.cuda.synchronize()


if __name__ == "__main__":
    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    fn = sample_worker if sys.argv[1] == "samples" else worker
    fn(int(sys.argv[2]), int(sys.argv[3]), int(sys.argv[4]), sys.argv[5])
