"""Thin ctypes binding over libago.so: argument marshalling only.

Every function of ``include/ago.h`` is exposed under its C name
(``ago_subgraph_create`` ...). ``Subgraph`` is a convenience wrapper that builds
the descriptor from a neutral operator list and passes torch tensors' device
pointers and the current CUDA stream; all computation happens inside the
library's kernels. There is no CPU or PyTorch fallback: if the library cannot
be loaded, or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Sequence

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libago.so")

AGO_OK = 0
AGO_ERR_INVALID_ARG, AGO_ERR_UNSUPPORTED, AGO_ERR_SHAPE, AGO_ERR_ALIGNMENT = 1, 2, 3, 4
AGO_ERR_WORKSPACE, AGO_ERR_CUDA, AGO_ERR_TIMEOUT = 5, 6, 7
AGO_BF16, AGO_FP32 = 0, 1
AGO_MODE_FUSED, AGO_MODE_PER_MINI_SUBGRAPH, AGO_MODE_PER_OP, AGO_MODE_AUTO = 0, 1, 2, 3
MODES = {"fused": AGO_MODE_FUSED, "per_mini_subgraph": AGO_MODE_PER_MINI_SUBGRAPH, "per_op": AGO_MODE_PER_OP, "auto": AGO_MODE_AUTO}

(AGO_OP_CONV2D, AGO_OP_GEMM, AGO_OP_BATCHED_QKT, AGO_OP_BATCHED_PV, AGO_OP_BIAS_ADD, AGO_OP_RELU,
 AGO_OP_RELU6, AGO_OP_GELU_TANH, AGO_OP_SCALE, AGO_OP_SOFTMAX_ROWS, AGO_OP_ADD_INPUT, AGO_OP_RESHAPE,
 AGO_OP_TRANSPOSE) = range(13)

(AGO_Q_NUM_WEIGHTS, AGO_Q_WEIGHT_BYTES, AGO_Q_OUTPUT_RANK, AGO_Q_OUTPUT_DIM, AGO_Q_OUTPUT_BYTES,
 AGO_Q_FLOPS_TENSOR, AGO_Q_FLOPS_CUDA, AGO_Q_SFU_OPS, AGO_Q_IO_BYTES, AGO_Q_NUM_LINKS, AGO_Q_LINK_CATEGORY,
 AGO_Q_NUM_LAUNCHES, AGO_Q_FUSED_KERNEL, AGO_Q_INTERMEDIATE_BYTES, AGO_Q_TILE_ROWS, AGO_Q_SMEM_BYTES, AGO_Q_MODE,
 AGO_Q_WORKSPACE_TRAFFIC) = range(18)

AGO_LINK_DOWNSTREAM_DEPTHWISE, AGO_LINK_DOWNSTREAM_POINTWISE, AGO_LINK_GENERAL = 1, 2, 3
(AGO_KERNEL_NONE, AGO_KERNEL_DEPTHWISE, AGO_KERNEL_MBV2_BLOCK, AGO_KERNEL_FFN, AGO_KERNEL_CONV3X3_PAIR,
 AGO_KERNEL_ATTENTION, AGO_KERNEL_PW_DW, AGO_KERNEL_DW_PW, AGO_KERNEL_DW_DW, AGO_KERNEL_PW_PW,
 AGO_KERNEL_GEMM_PERMUTE_GEMM) = range(11)

AGO_MAX_INPUTS, AGO_MAX_RANK, AGO_MAX_OPS = 4, 4, 32
AGO_STATIC_SCRATCH_BYTES = 4 << 20

EXPORTS = [
    "ago_subgraph_create", "ago_subgraph_run", "ago_subgraph_run_host", "ago_subgraph_destroy", "ago_last_error",
    "ago_subgraph_workspace_bytes", "ago_subgraph_set_workspace", "ago_subgraph_query", "ago_subgraph_status",
    "ago_version", "ago_subgraph_run_static", "ago_fusion_redundancy", "ago_op_weight", "ago_graph_cluster",
    "ago_launch_empty", "ago_subgraph_debug",
]


class ago_redundancy_query_t(ctypes.Structure):
    _fields_ = [("struct_size", ctypes.c_uint32), ("depthwise2", ctypes.c_int32), ("N", ctypes.c_int64),
                ("O1", ctypes.c_int64), ("I1", ctypes.c_int64), ("R1", ctypes.c_int64), ("C1", ctypes.c_int64),
                ("O2", ctypes.c_int64), ("R2", ctypes.c_int64), ("C2", ctypes.c_int64), ("stride2", ctypes.c_int64),
                ("H2", ctypes.c_int64), ("W2", ctypes.c_int64),
                ("o2", ctypes.c_int64), ("h2", ctypes.c_int64), ("w2", ctypes.c_int64)]


class ago_redundancy_result_t(ctypes.Structure):
    _fields_ = [("num_tiles", ctypes.c_int64), ("upstream_elems_unfused", ctypes.c_int64),
                ("upstream_elems_fused", ctypes.c_int64), ("upstream_macs_unfused", ctypes.c_int64),
                ("upstream_macs_fused", ctypes.c_int64), ("factor", ctypes.c_double),
                ("category", ctypes.c_int32), ("reserved", ctypes.c_int32)]


class ago_graph_desc_t(ctypes.Structure):
    _fields_ = [("struct_size", ctypes.c_uint32), ("num_nodes", ctypes.c_int32), ("weights", ctypes.POINTER(ctypes.c_double)),
                ("num_edges", ctypes.c_int32), ("reserved", ctypes.c_int32), ("edges", ctypes.POINTER(ctypes.c_int32)),
                ("threshold", ctypes.c_double)]


class ago_op_t(ctypes.Structure):
    _fields_ = [("kind", ctypes.c_int32), ("p", ctypes.c_int32 * 8), ("f", ctypes.c_float)]


class ago_subgraph_desc_t(ctypes.Structure):
    _fields_ = [
        ("struct_size", ctypes.c_uint32),
        ("mode", ctypes.c_int32),
        ("num_inputs", ctypes.c_int32),
        ("input_rank", ctypes.c_int32 * AGO_MAX_INPUTS),
        ("input_shape", (ctypes.c_int64 * AGO_MAX_RANK) * AGO_MAX_INPUTS),
        ("input_dtype", ctypes.c_int32 * AGO_MAX_INPUTS),
        ("num_ops", ctypes.c_int32),
        ("ops", ctypes.POINTER(ago_op_t)),
        ("output_dtype", ctypes.c_int32),
    ]


class AgoError(RuntimeError):
    def __init__(self, status: int, msg: str):
        super().__init__(f"ago status {status}: {msg}")
        self.status = status


_lib = None


def load(build_if_missing: bool = True):
    """Load libago.so (building it in-tree first when asked). Fails loudly."""
    global _lib
    if _lib is not None:
        return _lib
    if build_if_missing:
        from . import build as _build
        _build.build()
    if not os.path.exists(LIB_PATH):
        raise FileNotFoundError(f"{LIB_PATH} is missing: run paper_2212_01005_b200/build.py (needs nvcc)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, vpp = ctypes.c_void_p, ctypes.POINTER(ctypes.c_void_p)
    lib.ago_subgraph_create.restype = vp
    lib.ago_subgraph_create.argtypes = [ctypes.POINTER(ago_subgraph_desc_t)]
    lib.ago_subgraph_run.restype = ctypes.c_int
    lib.ago_subgraph_run.argtypes = [vp, vpp, vpp, vpp, vp]
    lib.ago_subgraph_run_host.restype = ctypes.c_int
    lib.ago_subgraph_run_host.argtypes = [vp, vpp, vpp, vpp, vpp, vpp, vp]
    lib.ago_subgraph_destroy.restype = None
    lib.ago_subgraph_destroy.argtypes = [vp]
    lib.ago_last_error.restype = ctypes.c_int
    lib.ago_last_error.argtypes = [ctypes.POINTER(ctypes.c_char_p)]
    lib.ago_subgraph_workspace_bytes.restype = ctypes.c_size_t
    lib.ago_subgraph_workspace_bytes.argtypes = [vp]
    lib.ago_subgraph_set_workspace.restype = ctypes.c_int
    lib.ago_subgraph_set_workspace.argtypes = [vp, vp, ctypes.c_size_t]
    lib.ago_subgraph_query.restype = ctypes.c_int
    lib.ago_subgraph_query.argtypes = [vp, ctypes.c_int32, ctypes.POINTER(ctypes.c_int64)]
    lib.ago_subgraph_status.restype = ctypes.c_int
    lib.ago_subgraph_status.argtypes = [vp]
    lib.ago_version.restype = ctypes.c_char_p
    lib.ago_launch_empty.restype = ctypes.c_int
    lib.ago_launch_empty.argtypes = [ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, vp]
    lib.ago_op_weight.restype = ctypes.c_double
    lib.ago_op_weight.argtypes = [ctypes.POINTER(ctypes.c_int64), ctypes.c_int32, ctypes.c_double, ctypes.c_double]
    lib.ago_graph_cluster.restype = ctypes.c_int
    lib.ago_graph_cluster.argtypes = [ctypes.POINTER(ago_graph_desc_t), ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_int32)]
    lib.ago_fusion_redundancy.restype = ctypes.c_int
    lib.ago_fusion_redundancy.argtypes = [ctypes.POINTER(ago_redundancy_query_t), ctypes.POINTER(ago_redundancy_result_t)]
    lib.ago_subgraph_debug.restype = ctypes.c_int
    lib.ago_subgraph_debug.argtypes = [vp, ctypes.c_int32, ctypes.c_int64]
    lib.ago_subgraph_run_static.restype = ctypes.c_int
    lib.ago_subgraph_run_static.argtypes = [vp, vpp, vpp, vpp, vp]
    _lib = lib
    return lib


# ---- the C entry points under their own names ------------------------------------


def ago_last_error():
    msg = ctypes.c_char_p()
    st = load().ago_last_error(ctypes.byref(msg))
    return st, (msg.value or b"").decode()


def ago_subgraph_create(desc: ago_subgraph_desc_t):
    return load().ago_subgraph_create(ctypes.byref(desc))


def ago_subgraph_destroy(h):
    load().ago_subgraph_destroy(h)


def _ptr_array(ptrs: Sequence[int]):
    arr = (ctypes.c_void_p * max(1, len(ptrs)))()
    for i, p in enumerate(ptrs):
        arr[i] = p
    return arr


def ago_subgraph_run(h, inputs: Sequence[int], weights: Sequence[int], outputs: Sequence[int], stream: int = 0) -> int:
    return load().ago_subgraph_run(h, _ptr_array(inputs), _ptr_array(weights), _ptr_array(outputs), stream)


def ago_op_weight(loop_extents: Sequence[int], c: float = 1.0, b: float = 0.0) -> float:
    """Eq. 1: c * prod(log(extent)) + b."""
    arr = (ctypes.c_int64 * max(1, len(loop_extents)))(*[int(x) for x in loop_extents])
    return float(load().ago_op_weight(arr, len(loop_extents), float(c), float(b)))


def ago_graph_cluster(weights: Sequence[float], edges: Sequence[Sequence[int]], threshold: float):
    """Algorithm 1 on a DAG: returns the subgraph index of every node (numbered by smallest member)."""
    n = len(weights)
    w = (ctypes.c_double * max(1, n))(*[float(x) for x in weights])
    flat = [int(x) for e in edges for x in e]
    ed = (ctypes.c_int32 * max(1, len(flat)))(*flat)
    g = ago_graph_desc_t()
    g.struct_size = ctypes.sizeof(ago_graph_desc_t)
    g.num_nodes, g.weights, g.num_edges, g.edges, g.threshold = n, w, len(edges), ed, float(threshold)
    out = (ctypes.c_int32 * max(1, n))()
    cnt = ctypes.c_int32(0)
    st = load().ago_graph_cluster(ctypes.byref(g), out, ctypes.byref(cnt))
    if st != AGO_OK:
        raise ValueError(f"ago_graph_cluster: status {st}: {ago_last_error()[1]}")
    return list(out[:n]), int(cnt.value)


def ago_fusion_redundancy(**kw) -> dict:
    """Upstream work of two stacked convolutions with and without intensive fusion (Section III-B).

    Keyword arguments are the fields of ago_redundancy_query_t except struct_size (depthwise2 defaults to 0,
    stride2, N, I1, R1, C1 to 1). Returns the fields of ago_redundancy_result_t as a dict; raises ValueError
    with the library's message on a non-zero status.
    """
    q = ago_redundancy_query_t()
    q.struct_size = ctypes.sizeof(ago_redundancy_query_t)
    defaults = dict(depthwise2=0, N=1, I1=1, R1=1, C1=1, stride2=1)
    defaults.update(kw)
    for k, v in defaults.items():
        setattr(q, k, int(v))
    r = ago_redundancy_result_t()
    st = load().ago_fusion_redundancy(ctypes.byref(q), ctypes.byref(r))
    if st != AGO_OK:
        raise ValueError(f"ago_fusion_redundancy: status {st}: {ago_last_error()[1]}")
    return {name: getattr(r, name) for name, _ in ago_redundancy_result_t._fields_ if name != "reserved"}


def ago_subgraph_run_static(h, inputs: Sequence[int], weights: Sequence[int], outputs: Sequence[int], stream: int = 0) -> int:
    """Unfused run whose scratch is the array built into the library: for callers
    that may not allocate device memory. Marshals pointers only."""
    return load().ago_subgraph_run_static(h, _ptr_array(inputs), _ptr_array(weights), _ptr_array(outputs), stream)


def ago_subgraph_run_host(h, host_inputs, weights, host_outputs, dev_inputs, dev_outputs, stream: int = 0) -> int:
    return load().ago_subgraph_run_host(h, _ptr_array(host_inputs), _ptr_array(weights), _ptr_array(host_outputs),
                                        _ptr_array(dev_inputs), _ptr_array(dev_outputs), stream)


def ago_subgraph_workspace_bytes(h) -> int:
    return int(load().ago_subgraph_workspace_bytes(h))


def ago_subgraph_set_workspace(h, dev_ptr: int, nbytes: int) -> int:
    return load().ago_subgraph_set_workspace(h, dev_ptr, nbytes)


def ago_subgraph_query(h, what: int, index: int = 0) -> int:
    out = ctypes.c_int64()
    st = load().ago_subgraph_query(h, what | (index << 16), ctypes.byref(out))
    if st != AGO_OK:
        raise AgoError(*ago_last_error())
    return int(out.value)


def ago_subgraph_status(h) -> int:
    return load().ago_subgraph_status(h)


AGO_DEBUG_WAIT_BUDGET_US, AGO_DEBUG_SKIP_SIGNAL = 1, 2


def ago_subgraph_debug(h, what: int, value: int) -> int:
    """Test hook of the failure path: wait budget in microseconds / wait site whose producer skips its signal."""
    return load().ago_subgraph_debug(h, int(what), int(value))


def ago_launch_empty(grid: int, block: int, smem_bytes: int = 0, stream: int = 0) -> None:
    st = load().ago_launch_empty(int(grid), int(block), int(smem_bytes), ctypes.c_void_p(stream))
    if st != AGO_OK:
        raise AgoError(*ago_last_error())


def ago_version() -> str:
    return load().ago_version().decode()


# ---- descriptor marshalling ----------------------------------------------------------


_KIND = {"conv2d": AGO_OP_CONV2D, "gemm": AGO_OP_GEMM, "qkt": AGO_OP_BATCHED_QKT, "pv": AGO_OP_BATCHED_PV,
         "bias_add": AGO_OP_BIAS_ADD, "relu": AGO_OP_RELU, "relu6": AGO_OP_RELU6, "gelu_tanh": AGO_OP_GELU_TANH,
         "scale": AGO_OP_SCALE, "softmax_rows": AGO_OP_SOFTMAX_ROWS, "add_input": AGO_OP_ADD_INPUT,
         "reshape": AGO_OP_RESHAPE, "transpose": AGO_OP_TRANSPOSE}


def make_desc(ops, input_shapes, mode="fused", dtype=AGO_BF16):
    """(kind, params) tuples + input shapes -> (ago_subgraph_desc_t, keep-alive ops array)."""
    arr = (ago_op_t * len(ops))()
    for i, (kind, prm) in enumerate(ops):
        o = arr[i]
        o.kind = _KIND[kind]
        if kind == "conv2d":
            vals = [prm["O"], prm["R"], prm["S"], prm["stride"], prm["pad"], prm.get("groups", 1)]
        elif kind == "gemm":
            vals = [prm["N"]]
        elif kind in ("qkt", "pv"):
            vals = [prm["input"], prm["heads"], prm["head_dim"]]
        elif kind == "add_input":
            vals = [prm["input"]]
        elif kind == "reshape":
            vals = [len(prm["shape"])] + list(prm["shape"])
        elif kind == "transpose":
            vals = [prm["a"], prm["b"]]
        else:
            vals = []
        for k, v in enumerate(vals):
            o.p[k] = int(v)
        o.f = float(prm.get("f", 0.0))
    d = ago_subgraph_desc_t()
    d.struct_size = ctypes.sizeof(ago_subgraph_desc_t)
    d.mode = MODES[mode] if isinstance(mode, str) else int(mode)
    d.num_inputs = len(input_shapes)
    for i, shp in enumerate(input_shapes):
        d.input_rank[i] = len(shp)
        for k, v in enumerate(shp):
            d.input_shape[i][k] = int(v)
        d.input_dtype[i] = dtype
    d.num_ops = len(ops)
    d.ops = ctypes.cast(arr, ctypes.POINTER(ago_op_t))
    d.output_dtype = dtype
    return d, arr


class Subgraph:
    """Handle wrapper: create from an operator list, run on torch CUDA tensors."""

    def __init__(self, ops, input_shapes, mode="fused", dtype=AGO_BF16):
        desc, keep = make_desc(ops, input_shapes, mode, dtype)
        self._h = ago_subgraph_create(desc)
        if not self._h:
            raise AgoError(*ago_last_error())
        self.mode = mode
        self.dtype = dtype
        self._ws = None
        rank = self.query(AGO_Q_OUTPUT_RANK)
        self.output_shape = tuple(self.query(AGO_Q_OUTPUT_DIM, i) for i in range(rank))
        self.num_weights = self.query(AGO_Q_NUM_WEIGHTS)

    def query(self, what: int, index: int = 0) -> int:
        return ago_subgraph_query(self._h, what, index)

    @property
    def workspace_bytes(self) -> int:
        return ago_subgraph_workspace_bytes(self._h)

    def _check(self, st: int):
        if st != AGO_OK:
            raise AgoError(*ago_last_error())

    def ensure_workspace(self, device):
        """Allocate (through torch) and attach the workspace the handle asks for."""
        import torch
        need = self.workspace_bytes
        if need and (self._ws is None or self._ws.numel() < need or self._ws.device != torch.device(device)):
            self._ws = torch.empty(need + 256, dtype=torch.uint8, device=device)
            base = (self._ws.data_ptr() + 255) & ~255
            self._check(ago_subgraph_set_workspace(self._h, base, need))

    def empty_output(self, device):
        import torch
        dt = torch.float32 if self.dtype == AGO_FP32 else torch.bfloat16
        return torch.empty(self.output_shape, dtype=dt, device=device)

    def run(self, inputs, weights, out=None, stream=None):
        """inputs / weights: torch CUDA tensors (contiguous). Enqueues on the
        current torch stream (or ``stream``) and returns the output tensor."""
        import torch
        dev = inputs[0].device
        if dev.type != "cuda":
            raise AgoError(AGO_ERR_CUDA, "inputs must be CUDA tensors: this library has no CPU path")
        if out is None:
            out = self.empty_output(dev)
        self.ensure_workspace(dev)
        s = stream if stream is not None else torch.cuda.current_stream(dev).cuda_stream
        st = ago_subgraph_run(self._h, [t.data_ptr() for t in inputs], [t.data_ptr() for t in weights],
                              [out.data_ptr()], s)
        self._check(st)
        return out

    def run_host(self, host_inputs, weights, host_out, dev_inputs, dev_out, stream=None):
        """Pinned host tensors in and out, device staging tensors supplied by the caller."""
        import torch
        dev = dev_out.device
        self.ensure_workspace(dev)
        s = stream if stream is not None else torch.cuda.current_stream(dev).cuda_stream
        st = ago_subgraph_run_host(self._h, [t.data_ptr() for t in host_inputs], [t.data_ptr() for t in weights],
                                   [host_out.data_ptr()], [t.data_ptr() for t in dev_inputs], [dev_out.data_ptr()], s)
        self._check(st)
        return host_out

    def status(self) -> int:
        return ago_subgraph_status(self._h)

    def close(self):
        if getattr(self, "_h", None):
            ago_subgraph_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
