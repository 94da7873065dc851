"""Seeded synthetic calibration tensors (inputs only; none of the method's arithmetic).

The paper calibrates on real Llama activations, weights and loss gradients
(Sec. 3.1); those are not available, so every test and the bench use random
tensors with the shapes, dtypes and value distributions of LLM layers:

  * toy MLP           4 linear layers, fp32, R = 8 samples of 128 tokens x 256,
                      X ~ N(0,1) with 1 % of the entries multiplied by 20,
                      W ~ N(0, 0.02), gradients ~ N(0, 1e-3);
  * Llama-7B block    q,k,v,o 4096->4096, gate,up 4096->11008, down 11008->4096,
                      bf16, R = 4 samples of 2048 tokens, 0.1 % of the input
                      channels of X multiplied by 50, W ~ N(0, 0.02), gradients
                      ~ N(0, 1e-4);
  * attention BGEMMs  (Q, K) and (P, V) with Q,K,V [R=4, 32 heads, 2048, 128]
                      ~ N(0,1) and P the causal softmax of N(0,1) logits
                      [4, 32, 2048, 2048]; gradients ~ N(0, 1e-4);
  * Llama-70B block   hidden 8192, KV 1024, FFN 28672, bf16, R = 2 samples of
                      4096 tokens, 0.1 % outlier channels x100, W ~ N(0, 0.01),
                      gradients ~ N(0, 1e-5).

The second parameter of N(.,.) is a standard deviation.  A weight has one
gradient per calibration sample (shape [R, K, C]), drawn independently.  Every
recipe takes ``shrink`` to divide the large dimensions for tests.  Numbers come
from ``torch.Generator`` seeded from (seed, layer, operand, kind), on the
device asked for; the tensors are rounded to their storage dtype here, before
either the CUDA library or the CPU oracle sees them.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import torch

LINEAR, BGEMM = 0, 1


@dataclass
class OperandSpec:
    shape: tuple            # shape of the values; leading dim is R when per_sample
    per_sample: bool        # True: sample r owns values[r]; False: shared (weights)
    std: float = 1.0
    grad_std: float = 1e-3
    dist: str = "normal"    # "normal" | "causal_softmax"
    outlier: tuple | None = None  # ("element"|"channel", probability, factor)

    @property
    def numel(self) -> int:
        n = 1
        for s in self.shape:
            n *= s
        return n


@dataclass
class LayerSpec:
    name: str
    kind: int
    R: int
    dtype: torch.dtype
    op0: OperandSpec
    op1: OperandSpec
    mac: int = 0  # multiply-accumulates of the layer, for theoretical time gain

    def scored_bytes(self) -> int:
        """Bytes of operand values and gradients the weighting step consumes:
        per-sample operands value+gradient once; shared operands value once and
        one gradient per sample."""
        es = torch.empty((), dtype=self.dtype).element_size()
        b = 0
        for op in (self.op0, self.op1):
            b += es * (2 * op.numel if op.per_sample else (1 + self.R) * op.numel)
        return b

    def value_bytes(self) -> int:
        es = torch.empty((), dtype=self.dtype).element_size()
        return es * (self.op0.numel + self.op1.numel)


def _linear(name, R, tokens, cin, cout, dtype, w_std, g_std, outlier) -> LayerSpec:
    return LayerSpec(
        name=name, kind=LINEAR, R=R, dtype=dtype,
        op0=OperandSpec((R, tokens, cin), True, 1.0, g_std, "normal", outlier),
        op1=OperandSpec((cout, cin), False, w_std, g_std, "normal", None),
        mac=R * tokens * cin * cout,
    )


def toy_mlp(R: int = 8, tokens: int = 128, width: int = 256, layers: int = 4) -> list[LayerSpec]:
    return [
        _linear("fc%d" % i, R, tokens, width, width, torch.float32, 0.02, 1e-3, ("element", 0.01, 20.0))
        for i in range(layers)
    ]


def llama_block(hidden: int, kv: int, ffn: int, R: int, tokens: int, w_std: float, g_std: float,
                outlier_factor: float, prefix: str = "", dtype=torch.bfloat16) -> list[LayerSpec]:
    out = ("channel", 0.001, outlier_factor)
    dims = [("q", hidden, hidden), ("k", hidden, kv), ("v", hidden, kv), ("o", hidden, hidden),
            ("gate", hidden, ffn), ("up", hidden, ffn), ("down", ffn, hidden)]
    return [_linear(prefix + n, R, tokens, cin, cout, dtype, w_std, g_std, out) for n, cin, cout in dims]


def llama7b_block(shrink: int = 1, prefix: str = "") -> list[LayerSpec]:
    return llama_block(4096 // shrink, 4096 // shrink, 11008 // shrink, 4, 2048 // shrink,
                       0.02, 1e-4, 50.0, prefix)


def llama70b_block(shrink: int = 1, prefix: str = "") -> list[LayerSpec]:
    return llama_block(8192 // shrink, 1024 // shrink, 28672 // shrink, 2, 4096 // shrink,
                       0.01, 1e-5, 100.0, prefix)


def attention_bgemm(shrink: int = 1, prefix: str = "", R: int = 4, heads: int = 32,
                    seq: int = 2048, hd: int = 128) -> list[LayerSpec]:
    heads, seq = max(1, heads // shrink), seq // shrink
    qk = lambda: OperandSpec((R, heads, seq, hd), True, 1.0, 1e-4)
    p = OperandSpec((R, heads, seq, seq), True, 1.0, 1e-4, "causal_softmax")
    return [
        LayerSpec(prefix + "qk_matmul", BGEMM, R, torch.bfloat16, qk(), qk(), R * heads * seq * seq * hd),
        LayerSpec(prefix + "av_matmul", BGEMM, R, torch.bfloat16, p, qk(), R * heads * seq * seq * hd),
    ]


def _gen(device, *key) -> torch.Generator:
    h = 0x9E3779B97F4A7C15
    for k in key:
        h = (h ^ (int(k) + 0x9E3779B97F4A7C15 + ((h << 6) & 0xFFFFFFFFFFFFFFFF) + (h >> 2))) & 0xFFFFFFFFFFFFFFFF
    g = torch.Generator(device=device)
    g.manual_seed(h & 0x7FFFFFFFFFFFFFFF)
    return g


def make_values(op: OperandSpec, dtype, device, seed: int, layer: int, operand: int) -> torch.Tensor:
    g = _gen(device, seed, layer, operand, 0)
    if op.dist == "causal_softmax":
        R = op.shape[0]
        out = torch.empty(op.shape, dtype=dtype, device=device)
        T = op.shape[-1]
        mask = torch.ones(T, T, dtype=torch.bool, device=device).triu(1)
        for r in range(R):  # one sample at a time bounds the fp32 temporary
            logits = torch.randn(op.shape[1:], generator=g, device=device, dtype=torch.float32)
            logits.masked_fill_(mask, float("-inf"))
            out[r] = torch.softmax(logits, dim=-1).to(dtype)
        return out
    v = torch.empty(op.shape, dtype=dtype, device=device)
    v.normal_(0.0, 1.0, generator=g)
    if op.std != 1.0:
        v.mul_(op.std)
    if op.outlier is not None:
        where, prob, factor = op.outlier
        go = _gen(device, seed, layer, operand, 2)
        if where == "element":
            m = torch.rand(op.shape, generator=go, device=device) < prob
            v[m] *= factor
        else:  # whole input channels (last dim) of X
            m = torch.rand(op.shape[-1], generator=go, device=device) < prob
            if not bool(m.any()):
                m[int(torch.randint(0, op.shape[-1], (1,), generator=go, device=device))] = True
            v[..., m] *= factor
    return v


def make_grads(op: OperandSpec, R: int, dtype, device, seed: int, layer: int, operand: int) -> torch.Tensor:
    g = _gen(device, seed, layer, operand, 1)
    shape = op.shape if op.per_sample else (R,) + tuple(op.shape)
    t = torch.empty(shape, dtype=dtype, device=device)
    t.normal_(0.0, 1.0, generator=g)
    t.mul_(op.grad_std)
    return t


@dataclass
class LayerTensors:
    spec: LayerSpec
    values: list = field(default_factory=list)  # [op0, op1]
    grads: list = field(default_factory=list)   # [op0, op1]; shared operands: [R, ...]


def make_layer(spec: LayerSpec, device, seed: int = 0, layer: int = 0) -> LayerTensors:
    lt = LayerTensors(spec)
    for i, op in enumerate((spec.op0, spec.op1)):
        lt.values.append(make_values(op, spec.dtype, device, seed, layer, i))
        lt.grads.append(make_grads(op, spec.R, spec.dtype, device, seed, layer, i))
    return lt


def share_block_inputs(lts: list) -> None:
    """Makes the layers of one transformer block that read the same activation
    bind the same tensor, as they do in a model: k and v take q's input, up takes
    gate's.  Every layer keeps the gradient with respect to its own input."""
    by_name = {lt.spec.name.split(".")[-1]: lt for lt in lts}
    for first, others in (("q", ("k", "v")), ("gate", ("up",))):
        if first not in by_name:
            continue
        for o in others:
            if o in by_name and by_name[o].values[0].shape == by_name[first].values[0].shape:
                by_name[o].values[0] = by_name[first].values[0]


def to_numpy(t: torch.Tensor):
    """Host copy for the oracle: fp32 as float32, bf16 as its uint16 bit pattern."""
    t = t.detach().contiguous().cpu()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view("uint16")
    return t.numpy()
