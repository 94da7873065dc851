"""The one device-side failure path: a bounded wait inside the scoring kernel
that runs out.  A test build (-DAMPQ_TEST_SHORT_WAITS) lets the stage waits of
the shared-memory ring give up after a handful of polls -- long before the
bulk copy they wait for can land -- while the producer's final drain keeps its
full limit, so every copy that was issued still completes before a CTA exits:
nothing hangs, nothing faults, the wait merely gives up first.  The getters
must then report AMPQ_ERR_TIMEOUT for that score; the context must stay usable
(a score that does not go through the ring succeeds on it and equals the
oracle), and the release build must score the same tensors normally afterwards.
The test build runs in a process of its own (AMPQ_LIBRARY picks it)."""
import os
import subprocess
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

pytestmark = pytest.mark.gpu


def _tensors():
    import torch

    g = torch.Generator(device="cuda").manual_seed(33)
    n = 128 * 1024 * 1024   # 16-byte aligned bf16, far larger than L2: the scoring warps keep catching up with HBM
    v = torch.empty(n, dtype=torch.bfloat16, device="cuda").normal_(0, 1, generator=g)
    gr = torch.empty(n, dtype=torch.bfloat16, device="cuda").normal_(0, 1e-3, generator=g)
    return v, gr


def _bind(ampq, ctx, lid, v, gr, offset, n=None):
    n = n or v.numel() - 8
    es = v.element_size()
    ctx.bind_operand(lid, 0, ampq.BF16, v.data_ptr() + offset * es, n, True, gr.data_ptr() + offset * es, n)
    ctx.bind_operand(lid, 1, ampq.BF16, 0, 0, False, 0, 0)
    return n


def worker():
    import torch

    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    from oracle import ampq_oracle as orc
    from paper_2505_13060_b200 import binding as ampq
    from paper_2505_13060_b200 import synth

    orc.build()
    v, gr = _tensors()
    ctx = ampq.Context(0, torch.cuda.current_stream().cuda_stream)
    ctx.set_formats([0, 1])
    lid = ctx.register_layer(ampq.LINEAR, "ring", 1)
    _bind(ampq, ctx, lid, v, gr, 0)
    ctx.score()
    rc = ampq.lib().ampq_get_layer(ctx._h, lid, *([None] * 8))
    assert rc == ampq.ERR_TIMEOUT, rc
    assert "wait" in ampq.lib().ampq_last_error(ctx._h).decode()
    assert ampq.lib().ampq_get_operand(ctx._h, lid, 0, np.zeros(2).ctypes.data) == ampq.ERR_TIMEOUT
    torch.cuda.synchronize()   # the device is fine: no error is pending
    # the same context, same tensors one element off the 16-byte grid: nothing goes through the ring
    n = _bind(ampq, ctx, lid, v, gr, 1, 4 * 1024 * 1024)
    ctx.score()
    got = ctx.get_operand(lid, 0)[0]
    a, _, _, seg = orc.score_operand(synth.to_numpy(v)[1:1 + n].reshape(1, -1), synth.to_numpy(gr)[1:1 + n].reshape(1, -1),
                                     1, True, [1])
    assert float(ctx.get_layer(lid)["amax"][0]) == float(a)
    assert np.all(np.abs(got - seg[0]) <= 1e-4 * np.abs(seg[0]))
    ctx.destroy()
    print("TIMEOUT-PATH-OK")


def test_stage_wait_that_runs_out_is_reported_and_leaves_the_context_usable(tmp_path, ampq, orc):
    import torch

    from paper_2505_13060_b200 import build, synth

    short = build.build(out=str(tmp_path / "libampq_short_waits.so"), defines=["AMPQ_TEST_SHORT_WAITS"])
    env = dict(os.environ, AMPQ_LIBRARY=short)
    out = subprocess.run([sys.executable, os.path.abspath(__file__)], env=env, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0 and "TIMEOUT-PATH-OK" in out.stdout, out.stderr[-3000:]
    # the release build on the same device, same tensors through the ring
    v, gr = _tensors()
    ctx = ampq.Context(0, torch.cuda.current_stream().cuda_stream)
    ctx.set_formats([0, 1])
    lid = ctx.register_layer(ampq.LINEAR, "ring", 1)
    n = _bind(ampq, ctx, lid, v, gr, 0, 16 * 1024 * 1024)
    ctx.score()
    got = ctx.get_operand(lid, 0)[0]
    _, _, _, seg = orc.score_operand(synth.to_numpy(v)[:n].reshape(1, -1), synth.to_numpy(gr)[:n].reshape(1, -1), 1, True, [1])
    assert np.all(np.abs(got - seg[0]) <= 1e-4 * np.abs(seg[0]))
    ctx.destroy()


if __name__ == "__main__":
    worker()
