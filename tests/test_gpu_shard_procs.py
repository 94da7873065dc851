"""Layer-sharded scoring by two processes that share the one GPU: each rank
scores the layers `assign_layers` gives it with `ampq_score`, the ranks exchange
the per-layer table over gloo (host tensors), and each runs the sub-graph sums
and the selection.  Table and plan must equal those of a single process that
scores everything, and the oracle's.  The two processes' kernels are independent
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


@pytest.mark.gpu
def test_two_processes_score_their_layers_and_meet_in_the_table(tmp_path, ampq, orc):
    import torch

    from helpers import REL_TOL, oracle_layer
    from paper_2505_13060_b200 import shard, synth

    sock = socket.socket()
    sock.bind(("127.0.0.1", 0))
    port = sock.getsockname()[1]
    sock.close()
    procs = [subprocess.Popen([sys.executable, os.path.abspath(__file__), str(r), "2", str(port), str(tmp_path)])
             for r in range(2)]
    for p in procs:
        assert p.wait(timeout=600) == 0
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
    worker(int(sys.argv[1]), int(sys.argv[2]), int(sys.argv[3]), sys.argv[4])
