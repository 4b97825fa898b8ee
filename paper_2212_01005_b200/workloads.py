"""Seeded synthetic workloads: subgraph descriptions and their input tensors.

This module holds no operator arithmetic. It only (1) describes each benchmark
subgraph as a neutral ordered operator list with shapes and (2) draws the
seeded random inputs and weights. Both the CUDA path and the CPU checker are
fed from here so that they see the same bits.

The shapes stand in for subgraphs of the networks the paper evaluates
(Section VI: MobileNet-V2-style inverted-residual blocks, BERT-style attention
and feed-forward chains) plus a ResNet basic block; values are random, because
neither the trained models nor their datasets are available.

Recipe: ``numpy.random.default_rng(seed_seq)``; tensors are drawn in ABI order
(all inputs, then all weights), each as float64 draws, scaled, cast to float32
and -- for bf16 tensors -- rounded to bf16 (round to nearest even). Bias vectors
stay float32.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Sequence, Tuple

import numpy as np

Op = Tuple[str, dict]


# ---- bf16 <-> float32 bit conversions (data preparation only) ----------------


def bf16_round(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bf16 (ties to even); returns float32."""
    return bf16_bits_to_f32(f32_to_bf16_bits(x))


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> uint16 bf16 bit patterns, round to nearest even."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    rounded = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    return rounded.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """uint16 bf16 bit patterns -> float32 (exact)."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


# ---- workload description -----------------------------------------------------


@dataclass
class Workload:
    name: str
    seed_seq: Sequence[int]
    input_shapes: List[Tuple[int, ...]]
    ops: List[Op]
    samples: int                     # independent problem instances per launch
    input_dist: List[str] = field(default_factory=list)   # "uniform" | "normal" | "relu_normal"
    note: str = ""

    # Derived by shape inference below.
    weight_shapes: List[Tuple[int, ...]] = field(default_factory=list)
    weight_kinds: List[str] = field(default_factory=list)   # "conv" | "dw" | "gemm" | "bias"
    weight_fan_in: List[int] = field(default_factory=list)
    output_shape: Tuple[int, ...] = ()

    def __post_init__(self):
        if not self.input_dist:
            self.input_dist = ["normal"] * len(self.input_shapes)
        self._infer()

    def _infer(self):
        shp = tuple(self.input_shapes[0])
        ws, kinds, fans = [], [], []
        for kind, p in self.ops:
            if kind == "conv2d":
                N, H, W, C = shp
                R, S, st, pad = p["R"], p["S"], p["stride"], p["pad"]
                Ho = (H + 2 * pad - R) // st + 1
                Wo = (W + 2 * pad - S) // st + 1
                if p.get("groups", 1) == 1:
                    ws.append((p["O"], R, S, C)); kinds.append("conv"); fans.append(R * S * C)
                else:
                    ws.append((R, S, C)); kinds.append("dw"); fans.append(R * S)
                shp = (N, Ho, Wo, p["O"])
            elif kind == "gemm":
                K = shp[-1]
                ws.append((K, p["N"])); kinds.append("gemm"); fans.append(K)
                shp = shp[:-1] + (p["N"],)
            elif kind == "qkt":
                B, S_, E = shp
                shp = (B, p["heads"], S_, S_)
            elif kind == "pv":
                B, Hh, S_, _ = shp
                shp = (B, S_, p["heads"] * p["head_dim"])
            elif kind == "bias_add":
                ws.append((shp[-1],)); kinds.append("bias"); fans.append(1)
            elif kind == "reshape":
                shp = tuple(p["shape"])
            elif kind == "transpose":
                l = list(shp); l[p["a"]], l[p["b"]] = l[p["b"]], l[p["a"]]; shp = tuple(l)
        self.weight_shapes, self.weight_kinds, self.weight_fan_in = ws, kinds, fans
        self.output_shape = shp


def _mbv2_ops(c_exp: int, c_out: int, stride: int, residual: bool) -> List[Op]:
    ops: List[Op] = [
        ("conv2d", dict(O=c_exp, R=1, S=1, stride=1, pad=0, groups=1)),
        ("bias_add", {}), ("relu6", {}),
        ("conv2d", dict(O=c_exp, R=3, S=3, stride=stride, pad=1, groups=c_exp)),
        ("bias_add", {}), ("relu6", {}),
        ("conv2d", dict(O=c_out, R=1, S=1, stride=1, pad=0, groups=1)),
        ("bias_add", {}),
    ]
    if residual:
        ops.append(("add_input", dict(input=0)))
    return ops


def _ffn_ops(hidden: int, out: int) -> List[Op]:
    return [("gemm", dict(N=hidden)), ("bias_add", {}), ("gelu_tanh", {}),
            ("gemm", dict(N=out)), ("bias_add", {})]


def _resnet_ops(ch: int) -> List[Op]:
    return [
        ("conv2d", dict(O=ch, R=3, S=3, stride=1, pad=1, groups=1)), ("bias_add", {}), ("relu", {}),
        ("conv2d", dict(O=ch, R=3, S=3, stride=1, pad=1, groups=1)), ("bias_add", {}),
        ("add_input", dict(input=0)), ("relu", {}),
    ]


def _attn_ops(heads: int, head_dim: int) -> List[Op]:
    return [("qkt", dict(input=1, heads=heads, head_dim=head_dim)),
            ("scale", dict(f=1.0 / float(np.sqrt(head_dim)))),
            ("softmax_rows", {}),
            ("pv", dict(input=2, heads=heads, head_dim=head_dim))]


def mbv2_block(name, seed_seq, N, H, c_in, c_exp, c_out, stride, residual) -> Workload:
    return Workload(name, seed_seq, [(N, H, H, c_in)], _mbv2_ops(c_exp, c_out, stride, residual),
                    samples=N, input_dist=["uniform"])


def ffn(name, seed_seq, M, d_model, hidden, samples, d_out=None) -> Workload:
    return Workload(name, seed_seq, [(M, d_model)], _ffn_ops(hidden, d_out or d_model), samples=samples)


def resnet_block(name, seed_seq, N, H, ch) -> Workload:
    return Workload(name, seed_seq, [(N, H, H, ch)], _resnet_ops(ch), samples=N,
                    input_dist=["relu_normal"])


def attention(name, seed_seq, B, S, heads, head_dim) -> Workload:
    E = heads * head_dim
    return Workload(name, seed_seq, [(B, S, E)] * 3, _attn_ops(heads, head_dim), samples=B,
                    input_dist=["normal"] * 3)


# The two-complex-operator pairs of the fusion-strategy micro-benchmark (Section VI-B): pointwise and depthwise
# convolutions with their bias / ReLU6 as they follow each other in MobileNetV2-like blocks.
_PW = lambda o: ("conv2d", dict(O=o, R=1, S=1, stride=1, pad=0, groups=1))
_DW = lambda c, stride: ("conv2d", dict(O=c, R=3, S=3, stride=stride, pad=1, groups=c))


def pw_dw(name, seed_seq, N, H, c_in, c_exp, stride) -> Workload:
    ops = [_PW(c_exp), ("bias_add", {}), ("relu6", {}), _DW(c_exp, stride), ("bias_add", {}), ("relu6", {})]
    return Workload(name, seed_seq, [(N, H, H, c_in)], ops, samples=N, input_dist=["uniform"])


def dw_pw(name, seed_seq, N, H, c_exp, c_out, stride) -> Workload:
    ops = [_DW(c_exp, stride), ("bias_add", {}), ("relu6", {}), _PW(c_out), ("bias_add", {})]
    return Workload(name, seed_seq, [(N, H, H, c_exp)], ops, samples=N, input_dist=["relu_normal"])


def dw_dw(name, seed_seq, N, H, c) -> Workload:
    ops = [_DW(c, 1), ("bias_add", {}), ("relu6", {}), _DW(c, 1), ("bias_add", {}), ("relu6", {})]
    return Workload(name, seed_seq, [(N, H, H, c)], ops, samples=N, input_dist=["relu_normal"])


def pw_pw(name, seed_seq, N, H, c_in, c_mid, c_out, act1=False, act2=True) -> Workload:
    # default: the linear bottleneck of one block followed by the expansion of the next
    ops = [_PW(c_mid), ("bias_add", {})] + ([("relu6", {})] if act1 else []) + [_PW(c_out), ("bias_add", {})] + \
          ([("relu6", {})] if act2 else [])
    return Workload(name, seed_seq, [(N, H, H, c_in)], ops, samples=N, input_dist=["relu_normal"])


def unfold_chain(name, seed_seq, B, P, N, d, d_out) -> Workload:
    """Two projections of a patch-unfolded attention block (MobileViT-like: B images, P pixels per patch, N patches,
    d channels) with the layout operators between them: matrix multiplication, reshape, add, reshape, transpose,
    reshape, matrix multiplication, reshape (Section VI-B). Rows are (image, pixel, patch) before the transpose and
    (image, patch, pixel) after it."""
    M = B * P * N
    ops = [("gemm", dict(N=d)), ("reshape", dict(shape=(B * P, N, d))), ("add_input", dict(input=1)),
           ("reshape", dict(shape=(B, P, N, d))), ("transpose", dict(a=1, b=2)), ("reshape", dict(shape=(M, d))),
           ("gemm", dict(N=d_out)), ("reshape", dict(shape=(B, N, P, d_out)))]
    return Workload(name, seed_seq, [(M, d), (B * P, N, d)], ops, samples=B, input_dist=["normal", "normal"])


def get(name: str, batch: int | None = None) -> Workload:
    """The benchmark configurations. ``batch`` overrides the number of
    independent samples (images, sequences) while keeping per-sample shapes."""
    if name == "mbv2_14":        # config 0
        return mbv2_block(name, [0], batch or 1, 14, 32, 192, 32, 1, True)
    if name == "ffn_512":        # config 1
        return ffn(name, [1], 512 * (batch or 1), 768, 3072, samples=batch or 1)
    if name == "mbv2_56":        # config 2a
        return mbv2_block(name, [2, 0], batch or 32, 56, 24, 144, 24, 1, True)
    if name == "mbv2_28s2":      # config 2b
        return mbv2_block(name, [2, 1], batch or 32, 28, 32, 192, 64, 2, False)
    if name == "resnet_56":      # config 3
        return resnet_block(name, [3], batch or 32, 56, 64)
    if name == "attn_384":       # config 4a
        return attention(name, [4, 0], batch or 32, 384, 12, 64)
    if name == "ffn_12288":      # config 4b
        b = batch or 32
        return ffn(name, [4, 1], 384 * b, 768, 3072, samples=b)
    # pairs of the 56 x 56 block (24 -> 144 -> 24), batch 32
    if name == "pw_dw_56":
        return pw_dw(name, [5, 0], batch or 32, 56, 24, 144, 1)
    if name == "dw_pw_56":
        return dw_pw(name, [5, 1], batch or 32, 56, 144, 24, 1)
    if name == "dw_dw_56":
        return dw_dw(name, [5, 2], batch or 32, 56, 144)
    if name == "pw_pw_56":
        return pw_pw(name, [5, 3], batch or 32, 56, 144, 24, 144)
    if name == "unfold_96":      # d = 96, 2 x 2 patches of a 32 x 32 feature map, expansion to 2 d
        return unfold_chain(name, [6], batch or 32, 4, 256, 96, 192)
    raise KeyError(name)


PAIRS = ["pw_dw_56", "dw_pw_56", "dw_dw_56", "pw_pw_56"]
ALL = ["mbv2_14", "ffn_512", "mbv2_56", "mbv2_28s2", "resnet_56", "attn_384", "ffn_12288"] + PAIRS + ["unfold_96"]


# ---- seeded tensors ---------------------------------------------------------------


def generate(wl: Workload, seed_seq: Sequence[int] | None = None) -> Dict[str, list]:
    """Draw inputs and weights. Returns float32 arrays whose values are exactly
    bf16-representable for bf16 tensors (activations, conv/gemm weights) and
    plain float32 for biases: ``{"inputs": [...], "weights": [...]}``."""
    rng = np.random.default_rng(list(seed_seq if seed_seq is not None else wl.seed_seq))
    inputs = []
    for shp, dist in zip(wl.input_shapes, wl.input_dist):
        if dist == "uniform":
            a = rng.uniform(-1.0, 1.0, size=shp)
        elif dist == "normal":
            a = rng.standard_normal(size=shp)
        elif dist == "relu_normal":
            a = np.maximum(rng.standard_normal(size=shp), 0.0)
        else:
            raise ValueError(dist)
        inputs.append(bf16_round(a.astype(np.float32)))
    gain = 2.0 if wl.ops[0][0] == "conv2d" else 1.0     # N(0, 2/fan_in) for conv nets, N(0, 1/fan_in) for GEMMs
    weights = []
    for shp, kind, fan in zip(wl.weight_shapes, wl.weight_kinds, wl.weight_fan_in):
        if kind == "bias":
            weights.append(rng.uniform(-0.1, 0.1, size=shp).astype(np.float32))
        else:
            a = rng.standard_normal(size=shp) * np.sqrt(gain / fan)
            weights.append(bf16_round(a.astype(np.float32)))
    return {"inputs": inputs, "weights": weights}


def io_bytes(wl: Workload) -> int:
    """Algorithmic HBM bytes of one fused launch: inputs + weights + output,
    bf16 activations and weights, float32 biases; no intermediates."""
    b = sum(2 * int(np.prod(s)) for s in wl.input_shapes)
    for s, k in zip(wl.weight_shapes, wl.weight_kinds):
        b += (4 if k == "bias" else 2) * int(np.prod(s))
    b += 2 * int(np.prod(wl.output_shape))
    return b


def flops(wl: Workload) -> Dict[str, float]:
    """Algorithmic work of the operator definitions (2 flop per MAC; no halo
    recomputation, no padding): tensor-core contractions, CUDA-core FMAs
    (depthwise) and transcendental evaluations (exp / tanh)."""
    shp = tuple(wl.input_shapes[0])
    tensor = cuda = sfu = 0.0
    for kind, p in wl.ops:
        if kind == "conv2d":
            N, H, W, C = shp
            Ho = (H + 2 * p["pad"] - p["R"]) // p["stride"] + 1
            Wo = (W + 2 * p["pad"] - p["S"]) // p["stride"] + 1
            if p.get("groups", 1) == 1:
                tensor += 2.0 * N * Ho * Wo * p["O"] * p["R"] * p["S"] * C
            else:
                cuda += 2.0 * N * Ho * Wo * C * p["R"] * p["S"]
            shp = (N, Ho, Wo, p["O"])
        elif kind == "gemm":
            M = int(np.prod(shp[:-1]))
            tensor += 2.0 * M * shp[-1] * p["N"]
            shp = shp[:-1] + (p["N"],)
        elif kind == "qkt":
            B, S_, E = shp
            tensor += 2.0 * B * p["heads"] * S_ * S_ * p["head_dim"]
            shp = (B, p["heads"], S_, S_)
        elif kind == "pv":
            B, Hh, S_, _ = shp
            tensor += 2.0 * B * Hh * S_ * S_ * p["head_dim"]
            shp = (B, S_, p["heads"] * p["head_dim"])
        elif kind in ("gelu_tanh", "softmax_rows"):
            sfu += float(np.prod(shp))
        elif kind == "reshape":
            shp = tuple(p["shape"])
        elif kind == "transpose":
            l = list(shp); l[p["a"]], l[p["b"]] = l[p["b"]], l[p["a"]]; shp = tuple(l)
    return {"tensor": tensor, "cuda": cuda, "sfu": sfu}
