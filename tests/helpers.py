"""Shared test plumbing: run the same seeded tensors through the CUDA library
and through the CPU oracle, and compare.  No arithmetic of the method here."""
import numpy as np
import torch

from paper_2505_13060_b200 import synth

REL_TOL = 1e-4  # bound on |gpu - oracle| / oracle for the fp32-accumulated sums


def oracle_layer(orc, lt, low_fmts, amax_presets=(None, None), threads=1):
    """Oracle values of one layer from its tensors (any device)."""
    spec = lt.spec
    ops = []
    for k, op in enumerate((spec.op0, spec.op1)):
        v = synth.to_numpy(lt.values[k])
        g = synth.to_numpy(lt.grads[k])
        a, sc, iv, seg = orc.score_operand(v.reshape(spec.R, -1) if op.per_sample else v.reshape(-1),
                                           g.reshape(spec.R, -1), spec.R, op.per_sample, list(low_fmts),
                                           amax_preset=amax_presets[k], threads=threads)
        ops.append(dict(amax=a, scale=sc, inv=iv, seg=seg))
    fmts = [orc.FMT_BASE] + list(low_fmts)
    out = orc.layer_combine(ops[0]["seg"], ops[1]["seg"], fmts)
    out["ops"] = ops
    return out


def assert_close(got, ref, what, tol=REL_TOL):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape, (what, got.shape, ref.shape)
    err = np.abs(got - ref)
    bad = err > tol * np.abs(ref)
    assert not bad.any(), "%s: max rel err %.3e (tol %.1e)\n got %s\n ref %s" % (
        what, float(np.max(err / np.maximum(np.abs(ref), 1e-300))), tol, got.ravel()[:8], ref.ravel()[:8])


def compare_layer(ampq, ctx, lid, ref, F, what=""):
    """Bit-exact amax and scales, sums within REL_TOL."""
    got = ctx.get_layer(lid)
    for k in range(2):
        o = ref["ops"][k]
        assert got["amax"][k].tobytes() == np.float32(o["amax"]).tobytes(), (what, k, got["amax"][k], o["amax"])
        assert got["scale"][k, 0] == 1.0 and got["inv_scale"][k, 0] == 1.0
        assert got["scale"][k, 1:].tobytes() == o["scale"].tobytes(), (what, k)
        assert got["inv_scale"][k, 1:].tobytes() == o["inv"].tobytes(), (what, k)
        assert_close(ctx.get_operand(lid, k), o["seg"], "%s operand %d [S, D_f]" % (what, k))
    assert_close(got["s_per_sample"], ref["s_per_sample"], what + " s^r")
    assert_close(got["s_mean"], ref["s_mean"], what + " s")
    assert_close(got["d_meas_per_sample"], ref["d_meas_per_sample"], what + " d_meas^r")
    assert_close(got["d_model"], ref["d_model"], what + " d_model")
    assert_close(got["d_meas"], ref["d_meas"], what + " d_meas")
    assert got["d_model"][0] == 0.0 and got["d_meas"][0] == 0.0
    return got


def gpu_codes(ctx, lid, operand, fmt, numel):
    out = torch.empty(max(numel, 1), dtype=torch.uint8, device="cuda")
    ctx.export_codes(lid, operand, fmt, out.data_ptr())
    torch.cuda.synchronize()
    return out[:numel].cpu().numpy()
