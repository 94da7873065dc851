"""Layer-sharded scoring across two processes (gloo, CPU): the host side of the
multi-GPU path.  Each rank takes the layers `assign_layers` gives it, produces
their per-layer rows, the ranks exchange the table with one all-reduce, and each
runs the sub-graph sums and the selection through the C ABI.  No GPU here, so
the per-layer rows come from the CPU oracle instead of `ampq_score`; what is
tested is the assignment, the exchange and the table-based group sums and
selection, against a single process that does everything itself."""
import json
import os
import socket
import subprocess
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
E4M3 = 1
F = 2


def _layers():
    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    from paper_2505_13060_b200 import synth

    specs = synth.llama7b_block(64, prefix="a.") + synth.llama7b_block(64, prefix="b.")
    return specs, [synth.make_layer(s, "cpu", seed=9, layer=i) for i, s in enumerate(specs)]


def _groups(specs, rng):
    groups = []
    for g0 in (0, 4, 7, 11):   # attention linears and MLP linears of both blocks
        members = list(range(g0, g0 + (4 if g0 in (0, 7) else 3)))
        Q = np.array([[0, 1]] * len(members), dtype=np.uint8)
        groups.append((members, Q, np.array([0.0, rng.uniform(0.5, 2.0)])))
    return groups


def _rows(lts, which):
    from helpers import oracle_layer
    from oracle import ampq_oracle as orc
    from paper_2505_13060_b200 import shard

    orc.build()
    return {i: shard.layer_row(oracle_layer(orc, lts[i], [E4M3]), F) for i in which}


def worker(rank, world, port, out):
    import torch.distributed as dist

    from paper_2505_13060_b200 import binding, shard

    specs, lts = _layers()
    dist.init_process_group("gloo", init_method="tcp://127.0.0.1:%d" % port, rank=rank, world_size=world)
    owner = shard.assign_layers([s.scored_bytes() for s in specs], world)
    mine = [i for i in range(len(specs)) if owner[i] == rank]
    table = shard.gather_layer_table(_rows(lts, mine), len(specs), F)
    groups = _groups(specs, np.random.default_rng(3))
    res = {}
    for mode in (binding.D_MODEL, binding.D_MEASURED):
        col = 1 + 1 if mode == binding.D_MODEL else 1 + F + 1
        all_low = float(np.sum(table[:, col]))
        for frac in (0.05, 0.5):
            p, c, d = shard.select_from_table(binding, table, F, groups, mode, frac * all_low)
            res["%d_%g" % (mode, frac)] = [p.tolist(), c, d]
    # sample-sharded exchanges: MAX of amax, R-weighted mean of the rows
    a = np.array([[1.0 + rank, 5.0 - rank], [0.25, 0.25 * (rank + 1)]], np.float32)
    amax = shard.reduce_amax(a)
    R_local = 3 if rank == 0 else 5
    rows = np.array([[1.0, 0.0, 2.0, 0.0, 4.0], [8.0, 0.0, 1.0, 0.0, 0.5]]) * (rank + 1)
    merged = shard.merge_sample_rows(binding, rows, R_local)
    dist.barrier()
    dist.destroy_process_group()
    with open(os.path.join(out, "rank%d.json" % rank), "w") as f:
        json.dump({"owner": owner.tolist(), "mine": mine, "table": table.tolist(), "res": res,
                   "amax": amax.tolist(), "merged": merged.tolist()}, f)


def test_two_ranks_agree_with_one_process(tmp_path, ampq, orc):
    sock = socket.socket()
    sock.bind(("127.0.0.1", 0))
    port = sock.getsockname()[1]
    sock.close()
    procs = [subprocess.Popen([sys.executable, os.path.abspath(__file__), str(r), "2", str(port), str(tmp_path)])
             for r in range(2)]
    for p in procs:
        assert p.wait(timeout=300) == 0
    got = [json.load(open(tmp_path / ("rank%d.json" % r))) for r in range(2)]
    # sample-sharded exchanges: element-wise maximum; (3*rows + 5*2*rows)/8
    assert got[0]["amax"] == got[1]["amax"] == [[2.0, 5.0], [0.25, 0.5]]
    base = np.array([[1.0, 0.0, 2.0, 0.0, 4.0], [8.0, 0.0, 1.0, 0.0, 0.5]])
    assert got[0]["merged"] == got[1]["merged"] == (base * 13.0 / 8.0).tolist()
    # both ranks hold the same table and the same plans, bit for bit
    assert got[0]["table"] == got[1]["table"] and got[0]["res"] == got[1]["res"]
    assert got[0]["owner"] == got[1]["owner"]
    assert sorted(got[0]["mine"] + got[1]["mine"]) == list(range(14)) and got[0]["mine"] and got[1]["mine"]
    # balanced by scored bytes: no rank carries more than the mean plus the largest layer
    specs, lts = _layers()
    cost = np.array([s.scored_bytes() for s in specs], float)
    loads = [cost[got[r]["mine"]].sum() for r in range(2)]
    assert max(loads) <= cost.sum() / 2 + cost.max()
    # one process, everything itself
    from paper_2505_13060_b200 import shard

    rows = _rows(lts, range(len(specs)))
    table = np.stack([rows[i] for i in range(len(specs))])
    assert table.tolist() == got[0]["table"]
    groups = _groups(specs, np.random.default_rng(3))
    for mode, key in ((ampq.D_MODEL, 1), (ampq.D_MEASURED, 1 + F)):
        d_layer = table[:, key:key + F]
        d_tabs = [orc.group_costs(m, Q, d_layer) for m, Q, _ in groups]
        for j, (m, Q, _) in enumerate(groups):
            assert ampq.group_costs_table(m, Q, d_layer).tolist() == d_tabs[j].tolist()
        all_low = float(np.sum(d_layer[:, 1]))
        for frac in (0.05, 0.5):
            want = orc.select_bruteforce([c for _, _, c in groups], d_tabs, frac * all_low)
            p, c, d = got[0]["res"]["%d_%g" % (mode, frac)]
            assert p == want[0].tolist() and c == want[1] and d == want[2]


def test_assign_layers_is_deterministic_and_balanced():
    sys.path.insert(0, ROOT)
    from paper_2505_13060_b200 import shard

    rng = np.random.default_rng(0)
    for world in (1, 2, 3, 8):
        cost = rng.integers(1, 1000, 57)
        a = shard.assign_layers(cost, world)
        assert (a == shard.assign_layers(cost.copy(), world)).all() and a.min() >= 0 and a.max() < world
        loads = np.bincount(a, weights=cost, minlength=world)
        assert loads.max() - loads.min() <= cost.max()


if __name__ == "__main__":
    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    worker(int(sys.argv[1]), int(sys.argv[2]), int(sys.argv[3]), sys.argv[4])
