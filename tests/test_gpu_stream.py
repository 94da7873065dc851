"""GPU parity of the streaming calibration calls, the fake quantisation, and a
miniature of the paper's model validation (Sec. 3.2): predicted against
measured loss MSE on a random toy MLP calibrated through module hooks."""
import numpy as np
import pytest
import torch

from helpers import assert_close, compare_layer, oracle_layer
from paper_2505_13060_b200 import synth

pytestmark = pytest.mark.gpu

E4M3, E5M2 = 1, 2


def _ctx(ampq, fmts):
    ctx = ampq.Context(0, torch.cuda.current_stream().cuda_stream)
    ctx.set_formats(list(fmts))
    return ctx


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_streamed_samples_match_oracle_and_full_score(ampq, orc, dtype):
    """Sample by sample with a static amax on the activations and a measured one
    on the weights: every value equals the oracle's, and the full score of the
    same tensors gives the same numbers up to the order of fp64 additions."""
    R = 3
    specs = [synth.LayerSpec("s%d" % i, synth.LINEAR, R, dtype,
                             synth.OperandSpec((R, nx), True, 1.0, 1e-3, "normal", ("element", 0.01, 20.0)),
                             synth.OperandSpec((nw,), False, 0.02, 1e-3))
             for i, (nx, nw) in enumerate([(70001, 40000), (3 * 32768, 65536 + 7), (5, 1 << 20)])]
    lts = [synth.make_layer(s, "cuda", seed=12, layer=i) for i, s in enumerate(specs)]
    code = ampq.torch_dtype_code(lts[0].values[0])
    ctx = _ctx(ampq, (0, E4M3, E5M2))
    ids = [ctx.register_layer(lt.spec.kind, lt.spec.name, R) for lt in lts]
    amax_x = [float(lt.values[0].float().abs().max()) for lt in lts]   # plumbing: a static scale from anywhere
    for lid, a in zip(ids, amax_x):
        ctx.set_amax(lid, 0, a)
    ctx.stream_begin()
    # settings that shape the results cannot change under a streaming pass
    L = ampq.lib()
    fm = (__import__("ctypes").c_int * 2)(0, E5M2)
    assert L.ampq_set_formats(ctx._h, fm, 2) == ampq.ERR_STATE
    assert L.ampq_set_scale_mode(ctx._h, ampq.SCALE_POW2) == ampq.ERR_STATE
    assert L.ampq_set_measured(ctx._h, 0) == ampq.ERR_STATE
    for r in range(R):   # samples arrive one at a time, layers in any order
        for lid, lt in reversed(list(zip(ids, lts))):
            x, gx = lt.values[0][r], lt.grads[0][r]
            ctx.stream_sample(lid, 0, r, code, x.data_ptr(), gx.data_ptr(), x.numel())
            w, gw = lt.values[1], lt.grads[1][r]
            ctx.stream_sample(lid, 1, r, code, w.data_ptr(), gw.data_ptr(), w.numel())
    ctx.stream_end()
    streamed = []
    for lid, lt, a in zip(ids, lts, amax_x):
        ref = oracle_layer(orc, lt, [E4M3, E5M2], amax_presets=(a, None))
        streamed.append((compare_layer(ampq, ctx, lid, ref, 3, "streamed " + lt.spec.name),
                         ctx.get_operand(lid, 0), ctx.get_operand(lid, 1)))
    # a sample streamed twice is overwritten, not added; an unstreamed one counts as 0
    ctx.stream_begin()
    lt = lts[0]
    for _ in range(2):
        ctx.stream_sample(ids[0], 0, 1, code, lt.values[0][1].data_ptr(), lt.grads[0][1].data_ptr(), lt.values[0][1].numel())
    ctx.stream_end()
    o = ctx.get_operand(ids[0], 0)
    assert o[1].tobytes() == streamed[0][1][1].tobytes() and not o[0].any() and not o[2].any()
    assert not ctx.get_operand(ids[1], 0).any()
    # the full score over the same tensors
    for lid, lt in zip(ids, lts):
        ampq.bind_layer_tensors(ctx, lid, lt)
    ctx.score()
    for lid, (got, o0, o1) in zip(ids, streamed):
        full = ctx.get_layer(lid)
        assert full["amax"].tobytes() == got["amax"].tobytes()
        assert_close(full["s_per_sample"], got["s_per_sample"], "full vs streamed s", tol=1e-12)
        assert_close(full["d_meas_per_sample"], got["d_meas_per_sample"], "full vs streamed d", tol=1e-12)
    # calls out of order are refused
    L = ampq.lib()
    assert L.ampq_stream_sample(ctx._h, ids[0], 0, 0, code, lt.values[0].data_ptr(), lt.grads[0].data_ptr(), 8) == ampq.ERR_STATE
    assert L.ampq_stream_end(ctx._h) == ampq.ERR_STATE
    ctx.stream_begin()
    assert L.ampq_stream_sample(ctx._h, ids[0], 0, R, code, lt.values[0].data_ptr(), lt.grads[0].data_ptr(), 8) == ampq.ERR_INVALID
    assert L.ampq_stream_sample(ctx._h, ids[0], 2, 0, code, lt.values[0].data_ptr(), lt.grads[0].data_ptr(), 8) == ampq.ERR_INVALID
    ctx.stream_end()
    ctx.destroy()


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("fmt", [E4M3, E5M2])
def test_fake_quant_bit_exact(ampq, orc, dtype, fmt):
    g = torch.Generator(device="cuda").manual_seed(31)
    ctx = _ctx(ampq, (0, E4M3, E5M2))
    code = 0 if dtype == torch.float32 else 1
    for n, amax in ((100003, -1.0), (1, -1.0), (65536, 1.5), (0, -1.0)):
        x = (torch.empty(max(n, 1), device="cuda").normal_(0, 1, generator=g)
             * torch.exp(torch.empty(max(n, 1), device="cuda").uniform_(-8, 2, generator=g))).to(dtype)[:n]
        out = torch.full((max(n, 1),), 7.0, dtype=dtype, device="cuda")[:n]
        ctx.fake_quant(code, fmt, x.data_ptr(), n, amax, out.data_ptr())
        torch.cuda.synchronize()
        if n == 0:
            continue
        host = synth.to_numpy(x)
        a = orc.amax(host) if amax < 0 else np.float32(amax)
        sc, iv = orc.scales(fmt, a)
        want = orc.fake_quant(host, fmt, sc, iv)
        assert np.array_equal(synth.to_numpy(out).view(want.dtype), want), (n, amax)
        # in place
        ctx.fake_quant(code, fmt, x.data_ptr(), n, float(a), x.data_ptr())
        torch.cuda.synchronize()
        assert np.array_equal(synth.to_numpy(x).view(want.dtype), want)
    with pytest.raises(ampq.AmpqError):
        _ctx(ampq, (0, E4M3)).fake_quant(code, E5M2, out.data_ptr(), 0, -1.0, out.data_ptr())
    ctx.destroy()


def test_toy_mlp_hooks_and_predicted_vs_measured_loss_mse(ampq, orc):
    """A random 4-layer MLP, R = 48 samples of 64 tokens.  Calibrate through the
    hooks (first pass: the amax of every layer input over all samples; second
    pass: scores with that static scale), check one layer against the oracle
    from tensors captured independently, then run the model with every layer in
    E4M3 and compare the measured loss MSE with the predicted one.  The first-order
    model says E[(g^ - g)^2] = sum_l d_l; per sample the squared sum of many
    small independent errors is chi-square distributed around it, so the mean
    over the samples must land within a factor of two."""
    from paper_2505_13060_b200 import hooks

    torch.manual_seed(0)
    R, tokens, width = 48, 64, 256
    model = torch.nn.Sequential(torch.nn.Linear(width, width), torch.nn.GELU(), torch.nn.Linear(width, width),
                                torch.nn.GELU(), torch.nn.Linear(width, width), torch.nn.GELU(),
                                torch.nn.Linear(width, 16)).cuda()
    xs = torch.randn(R, tokens, width, device="cuda")
    ys = torch.randint(0, 16, (R, tokens), device="cuda")

    def loss_of(r):
        return torch.nn.functional.cross_entropy(model(xs[r]), ys[r])

    ctx = _ctx(ampq, (0, E4M3))
    cal = hooks.Calibrator(ctx, model, R)
    assert len(cal.layer_ids) == 4
    # pass 1: per-sample scales; the amax reported is the largest over the samples
    cal.begin()
    for r in range(R):
        with cal.sample(r):
            loss_of(r).backward()
    first = cal.end()
    amax_x = [float(res["amax"][0]) for res in first]
    for lid, a in zip(cal.layer_ids, amax_x):
        ctx.set_amax(lid, 0, a)
    # pass 2: one static scale per layer input
    captured = {}
    h1 = model[2].register_forward_hook(lambda m, i, o: captured.setdefault("x", []).append(i[0].detach().clone()))
    h2 = model[2].register_full_backward_hook(
        lambda m, gi, go: captured.setdefault("g", []).append((gi[0].detach().clone(), go[0].detach().clone())))
    g = []
    cal.begin()
    for r in range(R):
        with cal.sample(r):
            l = loss_of(r)
            l.backward()
            g.append(float(l.detach()))
    res = cal.end()
    h1.remove(); h2.remove()
    # layer 1 (the second Linear) against the oracle, from independently captured tensors
    X = torch.stack(captured["x"])
    GX = torch.stack([a for a, _ in captured["g"]])
    GW = torch.stack([gy.t() @ x for x, (_, gy) in zip(captured["x"], captured["g"])])
    x_amax = float(X.abs().max())   # the oracle's static scale comes from torch, not from the library
    assert x_amax == amax_x[1]

    class LT:
        pass

    lt = LT()
    lt.spec = synth.LayerSpec("fc1", synth.LINEAR, R, torch.float32, synth.OperandSpec((R, tokens, width), True),
                              synth.OperandSpec((width, width), False))
    lt.values = [X, model[2].weight.detach()]
    lt.grads = [GX, GW]
    compare_layer(ampq, ctx, cal.layer_ids[1], oracle_layer(orc, lt, [E4M3], amax_presets=(x_amax, None)), 2, "hooked fc1")
    # predicted: every layer in E4M3
    d_meas = sum(r_["d_meas"][1] for r_ in res)
    d_model = sum(r_["d_model"][1] for r_ in res)
    # measured: run the model with inputs and weights rounded to E4M3
    with torch.no_grad(), cal.quantised([E4M3] * 4, amax_x):
        gq = [float(loss_of(r)) for r in range(R)]
    measured = float(np.mean((np.array(gq) - np.array(g)) ** 2))
    assert measured > 0
    print("toy MLP: measured / predicted loss MSE = %.3f (measured error), %.3f (noise model)" % (measured / d_meas, measured / d_model))
    assert 0.5 < measured / d_meas < 2.0, (measured, d_meas, d_model)
    assert 0.15 < measured / d_model < 1.2, (measured, d_meas, d_model)
    # nothing is left quantised
    with torch.no_grad():
        assert [float(loss_of(r)) for r in range(3)] == g[:3]
    ctx.destroy()


def test_algorithm_1_end_to_end_on_a_toy_model(ampq, orc):
    """Algorithm 1 in one piece on a random MLP: partition the model graph,
    calibrate through the hooks (sensitivities and mean-square loss), build the
    MAC time-gain tables, solve the integer program for several thresholds tau.
    The plan must equal the oracle's enumeration over the same tables, meet the
    budget tau^2 E[g^2], and move from all-baseline (tau = 0) to all-FP8."""
    from oracle import ampq_host_oracle as ho
    from paper_2505_13060_b200 import hooks

    torch.manual_seed(1)
    R, tokens, width = 16, 32, 128
    dims = [width, 256, 128, 256, 64, 10]
    mods = []
    for a, b in zip(dims[:-1], dims[1:]):
        mods += [torch.nn.Linear(a, b), torch.nn.GELU()]
    model = torch.nn.Sequential(*mods[:-1]).cuda()
    xs = torch.randn(R, tokens, width, device="cuda")
    ys = torch.randint(0, 10, (R, tokens), device="cuda")
    # step 1: the graph is a chain Linear, GELU, Linear, ...; only the Linear vertices can be quantised
    n = len(model)
    edges = [(i, i + 1) for i in range(n - 1)]
    quant = [isinstance(m, torch.nn.Linear) for m in model]
    group_of, J = ampq.partition(n, edges, quant)
    assert (group_of.tolist(), J) == ho.partition(n, edges, quant) and J == 5
    # step 2: calibration (with every layer's tensors captured on the side for the oracle)
    ctx = _ctx(ampq, (0, E4M3))
    cal = hooks.Calibrator(ctx, model, R)
    lin = [m for m in model if isinstance(m, torch.nn.Linear)]
    cap = [dict(x=[], gx=[], gy=[]) for _ in lin]
    hs = []
    for c_, m in zip(cap, lin):
        hs.append(m.register_forward_hook(lambda mod, i, o, c_=c_: c_["x"].append(i[0].detach().clone())))

        def grab(mod, gi, go, c_=c_):
            c_["gx"].append(None if gi[0] is None else gi[0].detach().clone())
            c_["gy"].append(go[0].detach().clone())

        hs.append(m.register_full_backward_hook(grab))
    losses = []
    cal.begin()
    for r in range(R):
        with cal.sample(r):
            l = torch.nn.functional.cross_entropy(model(xs[r]), ys[r])
            l.backward()
            losses.append(float(l.detach()))
    res = cal.end()
    for h in hs:
        h.remove()
    # the oracle's sensitivities from the captured tensors: s^r = S(X, dX) + S(W, dW), s = mean_r
    s_oracle = []
    for c_, m in zip(cap, lin):
        w = m.weight.detach()
        tot = 0.0
        for r in range(R):
            x, gy = c_["x"][r], c_["gy"][r]
            gx = c_["gx"][r] if c_["gx"][r] is not None else gy @ w
            gw = gy.t() @ x
            for v, gr in ((x, gx), (w, gw)):
                tot += orc.score_segment(synth.to_numpy(v), synth.to_numpy(gr.contiguous()), [E4M3], [1.0], [1.0])[0]
        s_oracle.append(tot / R)
    # step 3 stand-in: theoretical time gain from MAC counts (Sec. 2.3.2), one group per layer
    c_orc, d_gpu, d_orc = [], [], []
    for j, (m, lid) in enumerate(zip(lin, cal.layer_ids)):
        shape = (ampq.LINEAR, R * tokens, m.in_features, m.out_features)
        c = ampq.gain_table(ampq.GAIN_MAC, [shape], [[0, 1]], [0.0, 1e-12])
        c_orc.append(ho.gain_table(ho.GAIN_MAC, [shape], [[0, 1]], [0.0, 1e-12]))
        assert c.tolist() == c_orc[-1]
        ctx.define_group([lid], np.array([[0, 1]], np.uint8), c)
        d_gpu.append(ctx.group_costs(j, ampq.D_MODEL))
        d_orc.append(np.array([0.0, orc.alpha(3) * s_oracle[j]]))
        assert_close(d_gpu[-1][1], d_orc[-1][1], "d_model of layer %d" % j)
    # step 4: the integer program under tau^2 E[g^2]: the library on its tables, the oracle on its own
    all_low = sum(d[1] for d in d_orc)
    plans = []
    for tau in (0.0, 1e-4, 1e-3, 3e-3, 1e-2, 1.0):
        budget = ampq.budget_from_tau(tau, losses)
        assert budget == orc.budget_from_tau(tau, losses)
        p, c, d = ctx.select(ampq.D_MODEL, budget)
        want = orc.select_bruteforce(c_orc, d_orc, budget)
        assert p.tolist() == want[0].tolist() and c == want[1] and d <= budget
        assert_close(d, want[2], "selected loss MSE") if want[2] else None
        plans.append(int(p.sum()))
    assert plans[0] == 0 and plans == sorted(plans)
    assert plans[-1] == 5 or ampq.budget_from_tau(1.0, losses) < all_low
    ctx.destroy()


class _Attention(torch.nn.Module):
    """One causal self-attention block with its two batched products as modules."""

    def __init__(self, width, heads):
        super().__init__()
        from paper_2505_13060_b200 import hooks

        self.h, self.d = heads, width // heads
        self.q, self.k, self.v, self.o = (torch.nn.Linear(width, width) for _ in range(4))
        self.qk, self.av = hooks.BatchedMatmul(), hooks.BatchedMatmul()
        self.head = torch.nn.Linear(width, 8)

    def forward(self, x):   # x: [tokens, width]
        T = x.shape[0]
        split = lambda t: t.reshape(T, self.h, self.d).transpose(0, 1)   # [heads, tokens, d]
        s = self.qk(split(self.q(x)), split(self.k(x)).transpose(1, 2)) / self.d ** 0.5
        mask = torch.ones(T, T, dtype=torch.bool, device=x.device).triu(1)
        p = torch.softmax(s.masked_fill(mask, float("-inf")), dim=-1)
        y = self.av(p, split(self.v(x))).transpose(0, 1).reshape(T, -1)
        return self.head(x + self.o(y))


def test_attention_block_with_batched_products_through_hooks(ampq, orc):
    """Linear and batched-GEMM layers of a causal attention block calibrated
    through the hooks: the two products against the oracle from tensors captured
    independently, and predicted against measured loss MSE with all seven
    layers (five of them the paper's attention sub-graph) in E4M3."""
    from paper_2505_13060_b200 import hooks

    torch.manual_seed(3)
    R, tokens, width, heads = 32, 64, 128, 2
    model = _Attention(width, heads).cuda()
    xs = torch.randn(R, tokens, width, device="cuda")
    ys = torch.randint(0, 8, (R, tokens), device="cuda")
    loss_of = lambda r: torch.nn.functional.cross_entropy(model(xs[r]), ys[r])
    ctx = _ctx(ampq, (0, E4M3))
    cal = hooks.Calibrator(ctx, model, R)
    names = [n for n, _ in cal.modules]
    assert sorted(names) == sorted(["q", "k", "v", "o", "qk", "av", "head"])
    cap = {"qk": [], "av": []}
    hs = []
    for key in cap:
        m = getattr(model, key)
        hs.append(m.register_forward_hook(lambda mod, i, o, key=key: cap[key].append([t.detach().clone() for t in i])))
        hs.append(m.register_full_backward_hook(lambda mod, gi, go, key=key: cap[key][-1].extend(t.detach().clone() for t in gi)))
    g = []
    cal.begin()
    for r in range(R):
        with cal.sample(r):
            l = loss_of(r)
            l.backward()
            g.append(float(l.detach()))
    res = cal.end()
    for h in hs:
        h.remove()
    for key in ("qk", "av"):
        a = torch.stack([c[0].contiguous() for c in cap[key]])
        b = torch.stack([c[1].contiguous() for c in cap[key]])
        ga = torch.stack([c[2].contiguous() for c in cap[key]])
        gb = torch.stack([c[3].contiguous() for c in cap[key]])

        class LT:
            pass

        lt = LT()
        lt.spec = synth.LayerSpec(key, synth.BGEMM, R, torch.float32, synth.OperandSpec(tuple(a.shape), True),
                                  synth.OperandSpec(tuple(b.shape), True))
        lt.values, lt.grads = [a, b], [ga, gb]
        # without presets every sample was scaled by its own amax: compare sample by sample
        lid = cal.layer_ids[names.index(key)]
        for k, (v, gr) in enumerate(((a, ga), (b, gb))):
            got = ctx.get_operand(lid, k)
            for r in (0, R // 2, R - 1):
                hv, hg = synth.to_numpy(v[r]), synth.to_numpy(gr[r])
                _, _, _, seg = orc.score_operand(hv.reshape(-1), hg.reshape(1, -1), 1, False, [E4M3])
                assert_close(got[r], seg[0], "%s operand %d sample %d" % (key, k, r))
        if key == "av":
            assert float(a[0, 0].triu(1).abs().max()) == 0.0   # P is causal: exact zeros above the diagonal
    # predicted against measured with everything in E4M3 (per-call scales on both sides)
    d_meas = sum(r_["d_meas"][1] for r_ in res)
    with torch.no_grad(), cal.quantised([E4M3] * len(names)):
        gq = [float(loss_of(r)) for r in range(R)]
    measured = float(np.mean((np.array(gq) - np.array(g)) ** 2))
    print("attention block: measured / predicted loss MSE = %.3f" % (measured / d_meas))
    assert 0.4 < measured / d_meas < 2.5, (measured, d_meas)
    ctx.destroy()


@pytest.mark.parametrize("own_stream", [False, True])
def test_hook_calibration_memory_does_not_grow_with_samples(ampq, orc, own_stream):
    """Streaming calibration exists so that the R per-sample weight gradients
    never live together: the peak device memory of a hooked calibration with
    R = 24 samples stays at that of R = 3 (a kept gradient per sample would add
    21 x 3 x 4 MiB here), whether the context runs on torch's stream or on one
    of its own, and both give the same per-sample values."""
    from paper_2505_13060_b200 import hooks

    torch.manual_seed(1)
    width, tokens = 1024, 32
    model = torch.nn.Sequential(torch.nn.Linear(width, width), torch.nn.GELU(), torch.nn.Linear(width, width),
                                torch.nn.GELU(), torch.nn.Linear(width, width)).cuda()
    side = torch.cuda.Stream() if own_stream else None

    def run(R):
        xs = torch.randn(R, tokens, width, device="cuda")
        ctx = ampq.Context(0, (side or torch.cuda.current_stream()).cuda_stream)
        ctx.set_formats([0, E4M3])
        cal = hooks.Calibrator(ctx, model, R)
        torch.cuda.synchronize()
        torch.cuda.reset_peak_memory_stats()
        base = torch.cuda.memory_allocated()
        cal.begin()
        for r in range(R):
            with cal.sample(r):
                model(xs[r]).square().mean().backward()
            model.zero_grad(set_to_none=True)
        res = cal.end()
        peak = torch.cuda.max_memory_allocated() - base
        ctx.destroy()
        return peak, res

    run(2)   # warm the allocator and the library's workspace
    small, res3 = run(3)
    large, res24 = run(24)
    assert large < small + 6 * width * width * 4, (small, large)
    assert np.all(res24[1]["s_per_sample"] > 0)
