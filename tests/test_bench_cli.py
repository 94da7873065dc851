"""Host logic of bench.py that needs no GPU: the plausibility check of a line,
the start of N ranks for --gpus N, the per-block selection groups."""
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import bench  # noqa: E402


def test_a_line_that_reads_faster_than_hbm_is_rejected():
    peak = 6549.4
    ok = {"value": 5022.0}
    assert not bench.reject_implausible(ok, peak, {"whole_pass_traffic.gbs": 6974.0, "roofline.amax_kernel_gbs": 7318.0,
                                                   "scoring launches": 6856.0})
    assert ok == {"value": 5022.0}
    # the numbers of a step whose amax pass skipped nine tenths of its reads
    bad = {"value": 6450.6}
    assert bench.reject_implausible(bad, peak, {"whole_pass_traffic.gbs": 8958.0, "roofline.amax_kernel_gbs": 32466.0,
                                                "scoring launches": 6997.0})
    assert bad["value"] is None and bad["rejected_value"] == 6450.6
    assert "whole_pass_traffic.gbs" in bad["invalid"] and "amax_kernel_gbs" in bad["invalid"]
    json.dumps(bad)
    assert not bench.reject_implausible({"value": 1.0}, peak, {"amax (nothing measured)": None})


def test_gpus_n_without_a_launcher_starts_n_ranks(monkeypatch):
    calls = []
    monkeypatch.setattr(bench.subprocess, "call", lambda cmd: calls.append(cmd) or 0)
    monkeypatch.setattr(sys, "argv", ["bench.py", "--gpus", "4", "--steps", "2", "--warmup", "3"])
    monkeypatch.delenv("WORLD_SIZE", raising=False)
    try:
        bench.main()
        raise AssertionError("main() should exit with the launcher's status")
    except SystemExit as e:
        assert e.code == 0
    (cmd,) = calls
    assert cmd[1:4] == ["-m", "torch.distributed.run", "--nnodes=1"]
    assert cmd[cmd.index("--nproc-per-node") + 1] == "4" and cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert cmd[-6:] == ["--gpus", "4", "--steps", "2", "--warmup", "3"] and cmd[-7].endswith("bench.py")


def test_selection_groups_are_one_per_block():
    class Spec:
        pass

    groups = bench.selection_groups([Spec()] * 7, 5, seed=1)
    assert [g[0] for g in groups] == [list(range(7 * b, 7 * b + 7)) for b in range(5)]
    for _, Q, c in groups:
        assert Q.shape == (7, 2) and Q[:, 0].tolist() == [0] * 7 and Q[:, 1].tolist() == [1] * 7
        assert c[0] == 0.0 and 0.5 <= c[1] <= 2.0
    assert groups[0][2][1] != groups[1][2][1]
    again = bench.selection_groups([Spec()] * 7, 5, seed=1)
    assert all(np.array_equal(a[2], b[2]) for a, b in zip(groups, again))
