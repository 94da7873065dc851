"""The self-checking debug build (-DAMPQ_BOUNDS_CHECK): every scoring tile is
checked against the extent of its tensor on the device and reported, not read,
when it falls outside.  A mixed workload -- ragged and misaligned operands,
shared weights with several sample groups, inputs shared by several layers, a
triangular operand, streamed samples -- must pass the check and give, bit for bit, what the release build
gives.  Each build runs in a process of its own (AMPQ_LIBRARY picks it)."""
import hashlib
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

pytestmark = pytest.mark.gpu


def worker():
    import numpy as np
    import torch

    sys.path.insert(0, ROOT)
    from paper_2505_13060_b200 import binding as ampq
    from paper_2505_13060_b200 import synth

    h = hashlib.sha256()
    ctx = ampq.Context(0, torch.cuda.current_stream().cuda_stream)
    ctx.set_formats([0, 1, 2])
    specs = synth.llama7b_block(16) + synth.attention_bgemm(8) + synth.toy_mlp(R=5, tokens=33, width=97, layers=2)
    lts = [synth.make_layer(s, "cuda", seed=21, layer=i) for i, s in enumerate(specs)]
    synth.share_block_inputs(lts[:7])   # q, k, v and gate, up read one input each: scored as groups
    ids = []
    for lt in lts:
        lid = ctx.register_layer(lt.spec.kind, lt.spec.name, lt.spec.R)
        ampq.bind_layer_tensors(ctx, lid, lt)
        ids.append(lid)
    ctx.set_causal(ids[8], 0, 256)   # the softmax operand of the (P, V) product
    ctx.score()
    for lid in ids:
        r = ctx.get_layer(lid)
        for k in ("amax", "scale", "s_per_sample", "d_meas_per_sample"):
            h.update(np.ascontiguousarray(r[k]).tobytes())
    ctx.stream_begin()
    lt = lts[0]
    for r in range(lt.spec.R):
        x, gx = lt.values[0][r], lt.grads[0][r]
        ctx.stream_sample(ids[0], 0, r, ampq.BF16, x.data_ptr(), gx.data_ptr(), x.numel())
    ctx.stream_end()
    h.update(ctx.get_operand(ids[0], 0).tobytes())
    ctx.destroy()
    print("DIGEST", h.hexdigest())


def test_bounds_checking_build_agrees_with_release_build(tmp_path):
    sys.path.insert(0, ROOT)
    from paper_2505_13060_b200 import build

    if build.needs_build():
        build.build()
    checked = build.build(out=str(tmp_path / "libampq_bounds.so"), defines=["AMPQ_BOUNDS_CHECK"])
    digests = []
    for lib in (build.LIB, checked):
        env = dict(os.environ, AMPQ_LIBRARY=lib)
        out = subprocess.run([sys.executable, os.path.abspath(__file__)], env=env, capture_output=True, text=True, timeout=600)
        assert out.returncode == 0, out.stderr[-2000:]
        digests.append([l for l in out.stdout.splitlines() if l.startswith("DIGEST")][0])
    assert digests[0] == digests[1]


if __name__ == "__main__":
    worker()
