#!/usr/bin/env python
"""Benchmark of the loss-MSE sensitivity pass: GB/s scored on the Llama-70B-shaped workload.

One step = one ``ampq_score`` over all 80 blocks x 7 linear layers of the
70B-shaped configuration (hidden 8192, KV 1024, FFN 28672, R = 2 samples of 4096
tokens, bf16): amax pass, scales, the fused FP8 cast / error / gradient
weighting / reduction, ordered finalize and the per-layer combine, for
614.7 GB of scored operand and gradient bytes.  80 blocks do not fit in HBM at
once, so block b is bound to device slot b mod ``--resident-blocks`` (each slot
is a full block of distinct random tensors, 7.68 GB); two passes over a slot are
tens of GB of other traffic apart, far beyond the 126 MB L2, so every byte
comes from HBM.  Because the slots stand for different blocks, the library's
pointer-based sharing (one amax pass and one read for layers bound to the very
same values) is switched off for these bindings: every one of the 1120 operands
is measured and scored in full.  A line whose byte rates exceed 1.2 x the
measured HBM peak reports ``value: null`` with the reason.

``--gpus N`` started as a plain process starts the N ranks itself (torchrun on
127.0.0.1).  Ranks are independent replicas by default; ``--shard layers``
splits one model's layers over the ranks and adds the table exchange and the
selection to the step.

Prints one JSON line: ``value`` = scored bytes of all ranks / device time of the
step (CUDA events, max over ranks); ``roofline`` for the scoring kernel from
events the library records around that kernel; ``e2e`` through the same C-ABI
call with the tensors in pinned host memory (one block per step, copies inside
the timed region); ``cpu_baseline`` = the CPU oracle timed on a bounded sample
of the same workload.  ``--impl reference`` times only the oracle.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "sensitivity_pass_throughput_scored"
UNIT = "GB/s"
NUM_BLOCKS = 80
FALLBACK_HBM_GBS = 6650.0
# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) per scored byte of the
# scoring launches, from the ncu capture summarised in
# profiles/score_kernel_amax_kernel_llama70b_qkvo_ncu_full.md (a 1.98 GB case;
# traffic grows in proportion to the elements).  It holds only for the kernel
# source it was taken on: `kernels_sha256` is the digest of ampq_kernels.cu +
# ampq_device.h at capture time, and the bench reports traffic = null otherwise.
NCU_TRAFFIC = {
    "kernels_sha256": "504a1eb9e39bd496d4a1f1cbe80743bc420cea27dd48bcadf0ae52f374e98e0e",
    "dram_bytes_per_scored_byte": {"e4m3": 1.0059},
    "source": "profiles/score_kernel_amax_kernel_llama70b_qkvo_ncu_full.md",
}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--resident-blocks", type=int, default=8,
                    help="distinct 70B-shaped blocks held on the device (7.68 GB each)")
    ap.add_argument("--blocks", type=int, default=NUM_BLOCKS, help="blocks scored per step (the config has 80)")
    ap.add_argument("--formats", default="e4m3", choices=["e4m3", "e5m2", "both"])
    ap.add_argument("--workload", default="llama70b", choices=["llama70b", "llama7b", "attention"],
                    help="llama70b is the benchmark; llama7b (3.2 GB per block) and attention (the two BGEMMs of one "
                         "attention layer per block, 2.55 GB) are side measurements, never the headline")
    ap.add_argument("--model-only", action="store_true",
                    help="side measurement: score only the paper's model term S (no amax pass, no FP8 cast)")
    ap.add_argument("--causal", action="store_true",
                    help="attention workload: declare the softmax operand causal so that its zero triangle is not read")
    ap.add_argument("--shared-inputs", action="store_true",
                    help="side measurement (llama70b / llama7b): q,k,v bind one input tensor and gate,up another, as "
                         "in a real transformer block, each layer with gradients of its own; every block is resident "
                         "(no slot reuse), and the library reads each shared input once")
    ap.add_argument("--shard", default="replicas", choices=["replicas", "layers"],
                    help="several ranks: 'replicas' gives every rank its own copy of the workload (weak scaling, no "
                         "exchange); 'layers' splits ONE model's layers over the ranks, exchanges the per-layer table "
                         "and runs the sub-graph sums and the selection on every rank (strong scaling)")
    ap.add_argument("--layers", default="",
                    help="comma-separated subset of a block's layers (q,k,v,o,gate,up,down); a small case of the "
                         "same kernels for profiler captures, never the benchmark")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-threads", type=int, default=0)
    return ap.parse_args()


def hbm_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


def kernels_digest() -> str:
    import hashlib

    h = hashlib.sha256()
    for f in ("ampq_kernels.cu", "ampq_device.h"):
        with open(os.path.join(ROOT, "paper_2505_13060_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()


# --------------------------------------------------------------------------
# clocks: nvidia-smi sampled while the timed region runs
class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None

    def start(self):
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                       "--format=csv,noheader,nounits", "-lms", "100"],
                                      stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def stop(self) -> dict:
        if self.p is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        time.sleep(0.15)
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, reasons, power = [], [], set(), []
        for line in self.f.read().splitlines():
            c = [x.strip() for x in line.split(",")]
            if len(c) < 9:
                continue
            try:
                sm.append(float(c[1]))
                mx.append(float(c[2]))
                power.append(float(c[3]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), c[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        try:
            os.unlink(self.f.name)
        except OSError:
            pass
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "samples": len(sm), "power_w_max": max(power)}


# --------------------------------------------------------------------------
def oracle_sample(threads: int, low_fmts, device, whole_block: bool):
    """The oracle's bounded sample of the 70B-shaped workload: one whole block
    (7 linear layers, R = 2 samples; 7.68 GB of scored bytes, about 10 s on 16
    cores) or only its q, k, v, o layers (1.98 GB; the per-step sample of the
    reference arm, which repeats it `--steps` times).  Returns (host tensors per
    layer, scored bytes, description)."""
    from paper_2505_13060_b200 import synth

    specs = synth.llama70b_block() if whole_block else synth.llama70b_block()[:4]
    layers, nbytes = [], 0
    for i, s in enumerate(specs):
        lt = synth.make_layer(s, device, seed=1234, layer=i)
        layers.append((s, [synth.to_numpy(t) for t in lt.values], [synth.to_numpy(t) for t in lt.grads]))
        nbytes += s.scored_bytes()
        del lt
    what = "all 7 linear layers" if whole_block else "q,k,v,o linear layers"
    return layers, nbytes, what + " of one Llama-70B-shaped block (R=2 x 4096 tokens, bf16)"


def time_oracle(layers, threads: int, low_fmts):
    """One pass of the oracle (amax, scales, cast, error, weighting, sums, layer
    combine) over the sample; independent segments run on host threads."""
    from concurrent.futures import ThreadPoolExecutor

    from oracle import ampq_oracle as orc

    t0 = time.perf_counter()
    with ThreadPoolExecutor(max_workers=threads) as ex:
        amaxes = list(ex.map(lambda a: orc.amax(a), [v for _, vals, _ in layers for v in vals]))
        jobs = []
        for li, (spec, vals, grads) in enumerate(layers):
            for k, op in enumerate((spec.op0, spec.op1)):
                a = amaxes[2 * li + k]
                sc_iv = [orc.scales(f, a) for f in low_fmts]
                sc = [x[0] for x in sc_iv]
                iv = [x[1] for x in sc_iv]
                v = vals[k].reshape(spec.R, -1) if op.per_sample else vals[k].reshape(1, -1)
                g = grads[k].reshape(spec.R, -1)
                for r in range(spec.R):
                    jobs.append((li, k, r, v[r if op.per_sample else 0], g[r], sc, iv))
        segs = list(ex.map(lambda j: orc.score_segment(j[3], j[4], low_fmts, j[5], j[6]), jobs))
    import numpy as np

    out = []
    for li, (spec, _, _) in enumerate(layers):
        seg = [[None] * spec.R, [None] * spec.R]
        for j, s in zip(jobs, segs):
            if j[0] == li:
                seg[j[1]][j[2]] = s
        out.append(orc.layer_combine(np.stack(seg[0]), np.stack(seg[1]), [orc.FMT_BASE] + list(low_fmts)))
    return time.perf_counter() - t0, len(jobs), out


def usable_cores() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except Exception:
        return os.cpu_count() or 1


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import torch

    low = {"e4m3": [1], "e5m2": [2], "both": [1, 2]}[args.formats]
    threads = args.cpu_threads or usable_cores()
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    layers, nbytes, desc = oracle_sample(threads, low, dev, whole_block=False)
    for _ in range(max(0, min(args.warmup, 1))):  # a warm-up pass of a deterministic CPU loop buys nothing more
        time_oracle(layers, threads, low)
    times = []
    used = 0
    for _ in range(args.steps):
        dt, njobs, _ = time_oracle(layers, threads, low)
        used = min(threads, njobs)
        times.append(dt)
    total = sum(times)
    val = nbytes * len(times) / total / 1e9
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / len(times),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "llama70b_shaped", "sample": desc, "formats": args.formats},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": used, "kind": "oracle", "sample": desc},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------
def workload_specs(workload: str, layers: str = ""):
    """Layer specs of one block of the named workload (optionally a subset of its layers)."""
    from paper_2505_13060_b200 import synth

    specs = {"llama70b": synth.llama70b_block, "llama7b": synth.llama7b_block,
             "attention": synth.attention_bgemm}[workload]()
    if layers:
        keep = layers.split(",")
        specs = [sp for sp in specs if sp.name in keep]
        if not specs:
            raise SystemExit("--layers matched no layer of the block")
    return specs


def bind_workload(ctx, specs, blocks: int, nres: int, dev, seed: int, causal: bool = False,
                  shared_inputs: bool = False, only=None):
    """Registers `blocks` blocks of `specs` in ctx.  Block b is bound to device
    slot b mod nres; each slot is a full block of distinct random tensors.
    The slots stand for `blocks` different blocks, so the library is told NOT to
    treat equal pointers as one tensor (ampq_set_sharing off): every binding is
    measured and scored in full.  With `shared_inputs` (needs blocks == nres)
    q,k,v and gate,up of a block bind one input each and sharing stays on.
    With `causal`, causal-softmax operands are declared triangular and only the
    bytes on or left of the diagonal count as scored.  `only`: the set of global
    layer indices (block * len(specs) + i) this process registers.
    Returns (slots, layer ids, scored bytes of one score)."""
    import torch

    from paper_2505_13060_b200 import binding as ampq
    from paper_2505_13060_b200 import synth

    if shared_inputs and blocks != nres:
        raise SystemExit("--shared-inputs needs every block resident")
    ctx.set_sharing(shared_inputs)
    slots = []
    for s in range(nres):
        lts = [synth.make_layer(sp, dev, seed=seed, layer=len(specs) * s + i) for i, sp in enumerate(specs)]
        if shared_inputs:
            synth.share_block_inputs(lts)
        slots.append(lts)
    torch.cuda.synchronize()
    ids, scored_bytes = [], 0
    for b in range(blocks):
        for i, sp in enumerate(specs):
            if only is not None and b * len(specs) + i not in only:
                continue
            lid = ctx.register_layer(sp.kind, "blk%d.%s" % (b, sp.name), sp.R)
            ampq.bind_layer_tensors(ctx, lid, slots[b % nres][i])
            ids.append(lid)
            scored_bytes += sp.scored_bytes()
            for k, op in enumerate((sp.op0, sp.op1)):
                if causal and op.dist == "causal_softmax":
                    T = op.shape[-1]
                    ctx.set_causal(lid, k, T)
                    es = slots[b % nres][i].values[k].element_size()
                    scored_bytes -= 2 * es * (op.numel // (T * T)) * (T * (T - 1) // 2)   # the triangle not read
    return slots, ids, scored_bytes


def selection_groups(specs, blocks: int, seed: int = 0):
    """One sub-graph per block with two configurations, all layers in the
    baseline format or all in the low-precision one (the benchmark's per-block
    groups); gains drawn uniformly in [0.5, 2] ms.  Layer indices are global."""
    import numpy as np

    rng = np.random.default_rng(seed)
    n = len(specs)
    groups = []
    for b in range(blocks):
        Q = np.array([[0, 1]] * n, dtype=np.uint8)
        groups.append((list(range(b * n, (b + 1) * n)), Q, np.array([0.0, rng.uniform(0.5, 2.0)])))
    return groups


def run_b200(args):
    import torch

    from paper_2505_13060_b200 import binding as ampq
    from paper_2505_13060_b200 import shard, synth

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the scoring path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod

        dist = dist_mod
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    dev = torch.device("cuda", local_rank)
    fmts = {"e4m3": [0, 1], "e5m2": [0, 2], "both": [0, 1, 2]}[args.formats]
    F = len(fmts)
    shard_layers = args.shard == "layers"

    specs = workload_specs(args.workload, args.layers)
    block_gb = sum(sp.scored_bytes() for sp in specs) / 1e9
    nres = max(1, min(args.resident_blocks, args.blocks))
    if args.shared_inputs:
        args.blocks = nres
    stream = torch.cuda.Stream(device=dev)
    ctx = ampq.Context(local_rank, stream.cuda_stream)
    ctx.set_formats(fmts)
    if args.model_only:
        ctx.set_measured(False)
    n_layers_model = args.blocks * len(specs)
    only, owner = None, None
    if shard_layers:
        # ONE model: its layers are dealt to the ranks by scored bytes, the same way on every rank
        owner = shard.assign_layers([sp.scored_bytes() for _ in range(args.blocks) for sp in specs], world)
        only = {i for i in range(n_layers_model) if owner[i] == rank}
    slots, ids, scored_bytes = bind_workload(ctx, specs, args.blocks, nres, dev,
                                             seed=100 + (0 if shard_layers else rank), causal=args.causal,
                                             shared_inputs=args.shared_inputs, only=only)
    my_global = sorted(only) if only is not None else list(range(n_layers_model))
    groups = selection_groups(specs, args.blocks) if shard_layers else None
    ctx.set_timing(True)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    plan = None

    def step():
        """One pass of the hot path.  Layer-sharded: plus the exchange of the
        per-layer table and the sub-graph sums and selection on every rank."""
        nonlocal plan
        ctx.score()
        t = ctx.get_timing()  # synchronises the step; the per-kernel events are the library's own
        if shard_layers:
            rows = dict(zip(my_global, ctx.get_layer_table(ids)))
            table = shard.gather_layer_table(rows, n_layers_model, F, device=dev)
            all_low = float(table[:, 1 + F + 1].sum())
            plan = shard.select_from_table(ampq, table, F, groups, ampq.D_MEASURED, 0.2 * all_low)
        return t

    with torch.cuda.stream(stream):
        for _ in range(args.warmup):
            step()
    ctx.get_layer(ids[0])
    launches_per_step = ctx.last_launch_count()
    pass_bytes = ctx.get_pass_bytes()
    sampler = ClockSampler(local_rank) if rank == 0 else None
    ev0 = torch.cuda.Event(enable_timing=True)
    ev1 = torch.cuda.Event(enable_timing=True)
    score_ms, amax_ms = [], []
    barrier()
    if sampler:
        sampler.start()
    with torch.cuda.stream(stream):
        ev0.record(stream)
        for _ in range(args.steps):
            t = step()
            score_ms.append(t["score_ms"])
            amax_ms.append(t["amax_ms"])
        ev1.record(stream)
    barrier()
    clocks = sampler.stop() if sampler else None
    total_ms = ev0.elapsed_time(ev1)
    job_scored_bytes = world * scored_bytes
    if dist is not None:
        tt = torch.tensor([total_ms], device=dev, dtype=torch.float64)
        dist.all_reduce(tt, op=dist.ReduceOp.MAX)
        total_ms = float(tt.item())
        if shard_layers:
            sb = torch.tensor([float(scored_bytes)], device=dev, dtype=torch.float64)
            dist.all_reduce(sb, op=dist.ReduceOp.SUM)
            job_scored_bytes = int(sb.item())
    ms_per_step = total_ms / args.steps
    value = job_scored_bytes / (ms_per_step * 1e-3) / 1e9
    first = ctx.get_layer(ids[0])

    # ---- roofline of the dominant kernel (the fused scoring kernel) on this rank
    peak, peak_kind = hbm_peak()
    k_ms = sum(score_ms) / len(score_ms)
    a_ms = sum(amax_ms) / len(amax_ms)
    achieved = scored_bytes / (k_ms * 1e-3) / 1e9
    roofline = {
        "bound": "hbm", "kernel": "score_kernel", "achieved": achieved, "peak": peak, "unit": "GB/s",
        "frac": achieved / peak, "peak_source": peak_kind + " (MEASURED_PEAKS.json hbm_gbs)" if peak_kind == "measured" else "fallback 6650 GB/s",
        "traffic": None, "kernel_ms": k_ms, "algorithmic_bytes_per_launch": scored_bytes,
        "bytes_read_by_scoring_launches": pass_bytes["score"],
        "amax_kernel_ms": a_ms, "amax_bytes_read": pass_bytes["amax"],
        "amax_kernel_gbs": pass_bytes["amax"] / (a_ms * 1e-3) / 1e9 if a_ms > 0 else None,
        "frac_of_8000_datasheet": achieved / 8000.0,
    }
    ratio = NCU_TRAFFIC["dram_bytes_per_scored_byte"].get(args.formats)
    if ratio is not None and kernels_digest() == NCU_TRAFFIC["kernels_sha256"] and not args.shared_inputs and not args.causal:
        roofline["traffic"] = ratio * scored_bytes  # scaled from the small capture to this launch
        roofline["traffic_source"] = NCU_TRAFFIC["source"]

    # ---- end to end: tensors in pinned host memory, one block per step
    e2e = None
    if not args.no_e2e and rank == 0:
        ectx = ampq.Context(local_rank, stream.cuda_stream)
        ectx.set_formats(fmts)
        host_layers, eids, h2d = [], [], 0

        class H:
            pass

        for i, sp in enumerate(specs):
            h = H()
            h.spec = sp
            h.values = [t.cpu().pin_memory() for t in slots[0][i].values]
            h.grads = [t.cpu().pin_memory() for t in slots[0][i].grads]
            host_layers.append(h)
            lid = ectx.register_layer(sp.kind, sp.name, sp.R)
            ampq.bind_layer_tensors(ectx, lid, h, mem=ampq.MEM_HOST)
            eids.append(lid)
            h2d += sum(t.numel() * t.element_size() for t in h.values + h.grads)
        block_scored = sum(sp.scored_bytes() for sp in specs)
        ectx.score()
        ectx.get_layer(eids[0])
        a0 = torch.cuda.Event(enable_timing=True)
        a1 = torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        d2h = 0
        with torch.cuda.stream(stream):
            a0.record(stream)
            for _ in range(args.e2e_steps):
                ectx.score()
                res = [ectx.get_layer(l) for l in eids]  # device -> host read of the step's result
            a1.record(stream)
        torch.cuda.synchronize()
        for sp in specs:
            d2h += 8 * (sp.R + 1 + sp.R * len(fmts) + 2 * len(fmts)) + 2 * (4 + 16 + 4) + 2 * 8 * sp.R * len(fmts)
        e_ms = a0.elapsed_time(a1) / args.e2e_steps
        if my_global[0] == 0 and not args.causal:   # same tensors, another tiling: equal up to the order of the fp64 additions
            assert abs(res[0]["s_mean"] - first["s_mean"]) <= 1e-9 * abs(first["s_mean"])
        e2e = {"value": block_scored / (e_ms * 1e-3) / 1e9, "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "ms_per_step": e_ms,
               "workload": "one %s-shaped block per step from pinned host memory (AMPQ_MEM_HOST binding)" % args.workload}
        ectx.destroy()
        del host_layers

    check = {"s_mean_layer0": first["s_mean"], "d_meas_layer0": float(first["d_meas"][1])}
    if plan is not None:
        check["plan_low_precision_groups"] = int(plan[0].sum())
    ctx.destroy()
    del slots
    torch.cuda.empty_cache()

    # ---- CPU baseline: the oracle on a bounded sample, rank 0, N = 1 only
    cpu = None
    if not args.no_cpu_baseline and rank == 0 and world == 1:
        threads = args.cpu_threads or usable_cores()
        layers, nbytes, desc = oracle_sample(threads, fmts[1:], dev, whole_block=True)
        dt, njobs, out = time_oracle(layers, threads, fmts[1:])
        cpu = {"value": nbytes / dt / 1e9, "unit": UNIT, "cores": min(threads, njobs), "kind": "oracle",
               "sample": desc + ", %.2f GB scored in %.1f s" % (nbytes / 1e9, dt)}

    if rank == 0:
        read_bytes = pass_bytes["amax"] + pass_bytes["score"]   # what this rank's step reads from HBM
        whole_gbs = read_bytes / (ms_per_step * 1e-3) / 1e9
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "strong" if shard_layers else "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {
                "workload": args.workload + "_shaped" + ("[%s]" % args.layers if args.layers else "") + ("[causal]" if args.causal else "")
                            + ("[model term only]" if args.model_only else "") + ("[q,k,v and gate,up share their input]" if args.shared_inputs else ""),
                "blocks": args.blocks, "layers": n_layers_model, "layers_on_rank0": len(ids), "R": specs[0].R,
                "tokens_per_sample": specs[0].op0.shape[-2], "operand_dtype": "bf16", "formats": args.formats,
                "scored_bytes_per_step_per_gpu": scored_bytes, "resident_blocks": nres,
                "residency": "block b reads device slot b %% %d; each slot is a distinct %.2f GB block; the library "
                             "treats every binding as a tensor of its own (pointer sharing off)" % (nres, block_gb)
                             if not args.shared_inputs else "every block resident, pointer sharing on",
                "l2": "inputs larger than L2 (%.1f GB resident, 126 MB L2)" % (nres * block_gb),
                "parallelism": ("one model, layers dealt to %d ranks by scored bytes; per-layer table exchanged by one "
                                "all-reduce; sub-graph sums and selection on every rank" % world) if shard_layers
                               else "independent replicas per GPU, no data-path collective",
            },
            "clocks": clocks, "e2e": e2e, "gpu_launches": launches_per_step * args.steps,
            "roofline": roofline, "cpu_baseline": cpu,
            "check": check,
            "pct_of_hbm_peak": {"measured_%.0f" % peak: 100.0 * value / peak / world, "datasheet_8000": 100.0 * value / 8000.0 / world},
            # every byte the step reads on rank 0 (the amax pass reads each operand once more)
            "whole_pass_traffic": {"bytes_read_per_gpu": read_bytes, "gbs": whole_gbs, "frac_of_measured_peak": whole_gbs / peak},
        }
        reject_implausible(line, peak, {"whole_pass_traffic.gbs": whole_gbs,
                                        "roofline.amax_kernel_gbs": roofline["amax_kernel_gbs"],
                                        "scoring launches (bytes read / kernel time)": pass_bytes["score"] / (k_ms * 1e-3) / 1e9})
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def reject_implausible(line: dict, peak_gbs: float, rates: dict) -> bool:
    """A step cannot read HBM much faster than the measured copy peak: a byte rate
    above 1.2 x that peak means the timed region skipped work, and the line then
    carries ``value: null`` with the reason instead of a number."""
    limit = 1.2 * peak_gbs
    too_fast = [k for k, v in rates.items() if v is not None and v > limit]
    if too_fast:
        line["rejected_value"] = line["value"]
        line["value"] = None
        line["invalid"] = "implausible: %s above 1.2 x the measured HBM peak (%.0f GB/s)" % (", ".join(too_fast), limit)
    return bool(too_fast)


def relaunch_ranks(args):
    """`--gpus N` (N > 1) started as a plain process: start the N ranks with
    torchrun on this node and let them print the line."""
    import socket

    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(args.gpus),
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    raise SystemExit(subprocess.call(cmd))


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        relaunch_ranks(args)
    else:
        run_b200(args)


if __name__ == "__main__":
    main()
