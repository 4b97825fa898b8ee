"""CPU oracle for the fused-subgraph executor -- TEST INFRASTRUCTURE ONLY.

A subgraph is an ordered list of operators (Section II: nodes are operators,
edges are tensors; Section III-A: the convolution / bias / ReLU mini-subgraph).
``run_chain`` applies the operators one after the other, each materialising
its complete output in fp64, which is the unfused program of Section III-A
(Fig. "Loop nest of a mini-subgraph without fusion"). Fusion and tiling are
loop transformations (Section III, first paragraph) and therefore must not
change this result.

The arithmetic lives in ``ago_oracle.c`` (plain loop nests, fp64, OpenMP on the
outermost independent loop only). Nothing here is shared with the CUDA path and
nothing here imports it. Only tests, the smoke check and the benchmark's CPU
baseline may import this module.

Operator list format (plain tuples, the same neutral description the workload
generators emit): ``(kind, params)`` with

  ("conv2d",       {"O","R","S","stride","pad","groups"})  groups == 1 or == C
  ("gemm",         {"N"})
  ("qkt",          {"input","heads","head_dim"})   second operand = inputs[input]
  ("pv",           {"input","heads","head_dim"})
  ("bias_add",     {})        consumes the next weight (a vector)
  ("relu"|"relu6"|"gelu_tanh"|"softmax_rows", {})
  ("scale",        {"f"})
  ("add_input",    {"input"})

Weights are consumed in order of appearance (conv2d / gemm weight, bias vector).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ago_oracle.c")
_LIB = os.path.join(_HERE, "libago_oracle.so")

_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (-O2, OpenMP) next to its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c99", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        dp = ctypes.POINTER(ctypes.c_double)
        i64 = ctypes.c_int64
        lib.ago_oracle_threads.restype = ctypes.c_int
        lib.ago_oracle_out_extent.restype = i64
        lib.ago_oracle_out_extent.argtypes = [i64] * 4
        lib.ago_oracle_conv2d.argtypes = [dp, i64, i64, i64, i64, dp, i64, i64, i64, i64, i64, dp]
        lib.ago_oracle_depthwise.argtypes = [dp, i64, i64, i64, i64, dp, i64, i64, i64, i64, dp]
        lib.ago_oracle_gemm.argtypes = [dp, i64, i64, dp, i64, dp]
        lib.ago_oracle_bias_add.argtypes = [dp, i64, i64, dp, dp]
        for name in ("relu", "relu6", "gelu_tanh"):
            getattr(lib, "ago_oracle_" + name).argtypes = [dp, i64, dp]
        lib.ago_oracle_scale.argtypes = [dp, i64, ctypes.c_double, dp]
        lib.ago_oracle_add.argtypes = [dp, dp, i64, dp]
        lib.ago_oracle_softmax_rows.argtypes = [dp, i64, i64, dp]
        lib.ago_oracle_batched_qkt.argtypes = [dp, dp, i64, i64, i64, i64, dp]
        lib.ago_oracle_batched_pv.argtypes = [dp, dp, i64, i64, i64, i64, dp]
        _lib = lib
    return _lib


def threads() -> int:
    """Number of OpenMP threads the oracle will use."""
    return int(_load().ago_oracle_threads())


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.float64))


# ---- single operators -------------------------------------------------------


def out_extent(H: int, R: int, stride: int, pad: int) -> int:
    return int(_load().ago_oracle_out_extent(H, R, stride, pad))


def conv2d(x, w, stride: int = 1, pad: int = 0) -> np.ndarray:
    """x [N,H,W,I], w [O,R,S,I] -> [N,Ho,Wo,O] (Section III-A loop nest)."""
    x, w = _f64(x), _f64(w)
    N, H, W, I = x.shape
    O, R, S, I2 = w.shape
    if I != I2:
        raise ValueError("conv2d: input channels of x and w differ")
    out = np.empty((N, out_extent(H, R, stride, pad), out_extent(W, S, stride, pad), O))
    _load().ago_oracle_conv2d(_p(x), N, H, W, I, _p(w), O, R, S, stride, pad, _p(out))
    return out


def depthwise(x, w, stride: int = 1, pad: int = 0) -> np.ndarray:
    """x [N,H,W,C], w [R,S,C] -> [N,Ho,Wo,C] (no reduction over channels)."""
    x, w = _f64(x), _f64(w)
    N, H, W, C = x.shape
    R, S, C2 = w.shape
    if C != C2:
        raise ValueError("depthwise: channels of x and w differ")
    out = np.empty((N, out_extent(H, R, stride, pad), out_extent(W, S, stride, pad), C))
    _load().ago_oracle_depthwise(_p(x), N, H, W, C, _p(w), R, S, stride, pad, _p(out))
    return out


def gemm(a, w) -> np.ndarray:
    """a [..., K] times w [K, N] over the last dimension."""
    a, w = _f64(a), _f64(w)
    K, Nn = w.shape
    if a.shape[-1] != K:
        raise ValueError("gemm: inner dimensions differ")
    M = a.size // K
    out = np.empty(a.shape[:-1] + (Nn,))
    _load().ago_oracle_gemm(_p(a), M, K, _p(w), Nn, _p(out))
    return out


def bias_add(x, b) -> np.ndarray:
    x, b = _f64(x), _f64(b)
    C = x.shape[-1]
    if b.shape != (C,):
        raise ValueError("bias_add: bias must have the size of the last dimension")
    out = np.empty_like(x)
    _load().ago_oracle_bias_add(_p(x), x.size // C, C, _p(b), _p(out))
    return out


def _unary(name):
    def f(x) -> np.ndarray:
        x = _f64(x)
        out = np.empty_like(x)
        getattr(_load(), "ago_oracle_" + name)(_p(x), x.size, _p(out))
        return out

    f.__name__ = name
    return f


relu = _unary("relu")
relu6 = _unary("relu6")
gelu_tanh = _unary("gelu_tanh")


def scale(x, f: float) -> np.ndarray:
    x = _f64(x)
    out = np.empty_like(x)
    _load().ago_oracle_scale(_p(x), x.size, float(f), _p(out))
    return out


def add(x, y) -> np.ndarray:
    x, y = _f64(x), _f64(y)
    if x.shape != y.shape:
        raise ValueError("add: shapes differ")
    out = np.empty_like(x)
    _load().ago_oracle_add(_p(x), _p(y), x.size, _p(out))
    return out


def softmax_rows(x) -> np.ndarray:
    x = _f64(x)
    out = np.empty_like(x)
    _load().ago_oracle_softmax_rows(_p(x), x.size // x.shape[-1], x.shape[-1], _p(out))
    return out


def batched_qkt(q, k, heads: int, head_dim: int) -> np.ndarray:
    """q, k [B,S,heads*head_dim] -> scores [B,heads,S,S]."""
    q, k = _f64(q), _f64(k)
    B, S, E = q.shape
    if E != heads * head_dim or k.shape != q.shape:
        raise ValueError("batched_qkt: shape mismatch")
    out = np.empty((B, heads, S, S))
    _load().ago_oracle_batched_qkt(_p(q), _p(k), B, S, heads, head_dim, _p(out))
    return out


def batched_pv(p, v, heads: int, head_dim: int) -> np.ndarray:
    """p [B,heads,S,S], v [B,S,heads*head_dim] -> [B,S,heads*head_dim]."""
    p, v = _f64(p), _f64(v)
    B, S, E = v.shape
    if E != heads * head_dim or p.shape != (B, heads, S, S):
        raise ValueError("batched_pv: shape mismatch")
    out = np.empty((B, S, E))
    _load().ago_oracle_batched_pv(_p(p), _p(v), B, S, heads, head_dim, _p(out))
    return out


# ---- a whole subgraph, operator after operator ------------------------------


def reshape(x: np.ndarray, shape) -> np.ndarray:
    """The same elements in row-major order under a new shape (the layout
    operators between the matrix multiplications of an attention block,
    Section VI-B): element i of the flattened tensor stays element i."""
    flat = np.ascontiguousarray(x).ravel()
    if int(np.prod(shape)) != flat.size:
        raise ValueError("reshape: element count changes")
    return flat.reshape(shape)


def transpose(x: np.ndarray, a: int, b: int) -> np.ndarray:
    """Swap axes a and b: out[..., i_a = u, ..., i_b = v, ...] = x[..., v, ..., u, ...]."""
    return np.ascontiguousarray(np.swapaxes(x, a, b))


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """fp64 -> nearest bfloat16 (ties to even) -> fp64. Used only by the
    diagnostic switch of ``run_chain``."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).astype(np.float64).reshape(np.shape(x))


_COMPLEX = ("conv2d", "gemm", "qkt", "pv")


def run_chain(ops: Sequence, inputs: Sequence, weights: Sequence,
              return_intermediates: bool = False, round_intermediates_to_bf16: bool = False):
    """Apply ``ops`` in order to ``inputs[0]``; every operator materialises its
    whole output in fp64 (no intermediate rounding).

    ``round_intermediates_to_bf16`` is a DIAGNOSTIC switch, never the pass/fail
    reference: it rounds the tensor each complex operator after the first reads
    to bfloat16, which is where a bf16 tensor-core pipeline must round (its
    operands are bf16). The difference between the two runs is rounding noise;
    what remains between the CUDA path and the rounded run is not."""
    ins = [_f64(t) for t in inputs]
    ws = [_f64(t) for t in weights]
    wi = 0
    x = ins[0]
    trace = []
    seen_complex = False
    for kind, prm in ops:
        if kind in _COMPLEX:
            if round_intermediates_to_bf16 and seen_complex:
                x = round_to_bf16(x)
            seen_complex = True
        if kind == "conv2d":
            w = ws[wi]; wi += 1
            C = x.shape[-1]
            g = int(prm.get("groups", 1))
            if g == 1:
                x = conv2d(x, w, int(prm["stride"]), int(prm["pad"]))
            elif g == C and int(prm["O"]) == C:
                x = depthwise(x, w, int(prm["stride"]), int(prm["pad"]))
            else:
                raise ValueError("conv2d: groups must be 1 or equal to the channel count")
        elif kind == "gemm":
            w = ws[wi]; wi += 1
            x = gemm(x, w)
        elif kind == "qkt":
            x = batched_qkt(x, ins[int(prm["input"])], int(prm["heads"]), int(prm["head_dim"]))
        elif kind == "pv":
            x = batched_pv(x, ins[int(prm["input"])], int(prm["heads"]), int(prm["head_dim"]))
        elif kind == "bias_add":
            b = ws[wi]; wi += 1
            x = bias_add(x, b)
        elif kind == "relu":
            x = relu(x)
        elif kind == "relu6":
            x = relu6(x)
        elif kind == "gelu_tanh":
            x = gelu_tanh(x)
        elif kind == "scale":
            x = scale(x, float(prm["f"]))
        elif kind == "softmax_rows":
            x = softmax_rows(x)
        elif kind == "add_input":
            x = add(x, ins[int(prm["input"])])
        elif kind == "reshape":
            x = reshape(x, tuple(int(v) for v in prm["shape"]))
        elif kind == "transpose":
            x = transpose(x, int(prm["a"]), int(prm["b"]))
        else:
            raise ValueError(f"unknown operator kind {kind!r}")
        if return_intermediates:
            trace.append(x)
    if wi != len(ws):
        raise ValueError(f"{len(ws)} weights given, {wi} consumed")
    return (x, trace) if return_intermediates else x
