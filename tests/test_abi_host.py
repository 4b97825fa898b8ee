"""Host-side checks that need no GPU: the library loads, exports every symbol
the header declares, validates descriptors, classifies links and counts work."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2212_01005_b200 import binding as B
from paper_2212_01005_b200 import workloads as WL

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_workspace_traffic_query_names_the_split_reduction_only():
    # The feed-forward kernels split the hidden tiles of some row blocks over J clusters that add their output
    # shares into an fp32 buffer in device memory: J additions of the whole output, one read-back and one zeroing sweep
    # (config 1: 24 hidden tiles, clusters of 4, J = 6). Kernels whose intermediates stay on chip, and every unfused mode,
    # report 0.
    wl = WL.get("ffn_512")
    sg = B.Subgraph(wl.ops, wl.input_shapes, mode="fused")
    m, n2, hid = 512, 768, 3072
    assert sg.query(B.AGO_Q_WORKSPACE_TRAFFIC) == (6 + 2) * m * n2 * 4
    sg.close()
    # config 4b: 48 blocks of 256 rows on 33 resident clusters; the 15 blocks of the second round are split in two
    wl = WL.get("ffn_12288")
    sg = B.Subgraph(wl.ops, wl.input_shapes, mode="fused")
    assert sg.query(B.AGO_Q_WORKSPACE_TRAFFIC) == (2 + 2) * (15 * 256) * n2 * 4    # two planes written, two read back
    assert sg.query(B.AGO_Q_NUM_LAUNCHES) == 2
    sg.close()
    for name, mode in (("ffn_512", "per_mini_subgraph"), ("ffn_12288", "per_mini_subgraph"), ("mbv2_56", "fused"), ("attn_384", "fused")):
        wl = WL.get(name)
        sg = B.Subgraph(wl.ops, wl.input_shapes, mode=mode)
        assert sg.query(B.AGO_Q_WORKSPACE_TRAFFIC) == 0, (name, mode)
        sg.close()


def test_library_exports_every_declared_symbol():
    lib = B.load()
    hdr = open(os.path.join(ROOT, "include", "ago.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = set(re.findall(r"\b(ago_[a-z_]+)\s*\(", hdr))
    assert declared, "no declarations found"
    assert declared == set(B.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name
    assert B.ago_version() == "0.1"


def test_desc_struct_matches_header_layout():
    # int32 fields, then [4][4] int64, ...; the library checks struct_size itself
    d, _ = B.make_desc([("relu", {})], [(8, 8)], "per_op")
    h = B.ago_subgraph_create(d)
    assert h, B.ago_last_error()
    B.ago_subgraph_destroy(h)
    d.struct_size = 12
    assert not B.ago_subgraph_create(d)
    st, msg = B.ago_last_error()
    assert st == B.AGO_ERR_INVALID_ARG and "struct_size" in msg


@pytest.mark.parametrize("name", WL.ALL)
def test_plan_counters_match_workload_arithmetic(name):
    wl = WL.get(name)
    sg = B.Subgraph(wl.ops, wl.input_shapes, mode="per_mini_subgraph")
    assert sg.output_shape == tuple(wl.output_shape)
    assert sg.num_weights == len(wl.weight_shapes)
    fl = WL.flops(wl)
    assert sg.query(B.AGO_Q_FLOPS_TENSOR) == int(fl["tensor"])
    assert sg.query(B.AGO_Q_FLOPS_CUDA) == int(fl["cuda"])
    assert sg.query(B.AGO_Q_SFU_OPS) == int(fl["sfu"])
    assert sg.query(B.AGO_Q_IO_BYTES) == WL.io_bytes(wl)
    for i, (shp, kind) in enumerate(zip(wl.weight_shapes, wl.weight_kinds)):
        assert sg.query(B.AGO_Q_WEIGHT_BYTES, i) == int(np.prod(shp)) * (4 if kind == "bias" else 2)
    sg.close()


def test_link_categories_follow_the_downstream_operator():
    # Section III-B: downstream depthwise / downstream pointwise (or matmul) / anything else
    cases = {
        "mbv2_56": [B.AGO_LINK_DOWNSTREAM_DEPTHWISE, B.AGO_LINK_DOWNSTREAM_POINTWISE],
        "ffn_512": [B.AGO_LINK_DOWNSTREAM_POINTWISE],
        "resnet_56": [B.AGO_LINK_GENERAL],
        "attn_384": [B.AGO_LINK_DOWNSTREAM_POINTWISE],
    }
    for name, want in cases.items():
        wl = WL.get(name)
        sg = B.Subgraph(wl.ops, wl.input_shapes, mode="per_op")
        n = sg.query(B.AGO_Q_NUM_LINKS)
        assert [sg.query(B.AGO_Q_LINK_CATEGORY, i) for i in range(n)] == want
        sg.close()


def test_launch_counts_per_mode():
    wl = WL.get("mbv2_14")
    per_op = B.Subgraph(wl.ops, wl.input_shapes, mode="per_op")
    mini = B.Subgraph(wl.ops, wl.input_shapes, mode="per_mini_subgraph")
    assert per_op.query(B.AGO_Q_NUM_LAUNCHES) == len(wl.ops) == 9
    assert mini.query(B.AGO_Q_NUM_LAUNCHES) == 3
    assert per_op.workspace_bytes >= 2 * 196 * 192 * 2
    wl = WL.get("attn_384", batch=1)
    mini = B.Subgraph(wl.ops, wl.input_shapes, mode="per_mini_subgraph")
    assert mini.query(B.AGO_Q_NUM_LAUNCHES) == 3          # QK^T+scale | softmax | PV
    # intermediates of the attention chain: scores and probabilities, written and read once each
    assert mini.query(B.AGO_Q_INTERMEDIATE_BYTES) == 2 * 2 * 12 * 384 * 384 * 2


def test_fused_planner_matches_every_chain_family_and_its_limits():
    # plan-time only: which kernel the fused mode picks, and what it refuses (no silent fallback)
    want = {"mbv2_56": B.AGO_KERNEL_MBV2_BLOCK, "mbv2_28s2": B.AGO_KERNEL_MBV2_BLOCK, "ffn_512": B.AGO_KERNEL_FFN,
            "resnet_56": B.AGO_KERNEL_CONV3X3_PAIR, "attn_384": B.AGO_KERNEL_ATTENTION, "pw_dw_56": B.AGO_KERNEL_PW_DW,
            "dw_pw_56": B.AGO_KERNEL_DW_PW, "dw_dw_56": B.AGO_KERNEL_DW_DW, "pw_pw_56": B.AGO_KERNEL_PW_PW,
            "unfold_96": B.AGO_KERNEL_GEMM_PERMUTE_GEMM}
    for name, kernel in want.items():
        wl = WL.get(name)
        sg = B.Subgraph(wl.ops, wl.input_shapes, mode="fused")
        assert sg.query(B.AGO_Q_FUSED_KERNEL) == kernel, name
        # one kernel, except where a row block's hidden tiles are split over clusters (config 1: few rows): a second,
        # small launch turns the fp32 sums into the output
        assert sg.query(B.AGO_Q_NUM_LAUNCHES) == (2 if name == "ffn_512" else 1), name
        assert 0 < sg.query(B.AGO_Q_SMEM_BYTES) <= 227 * 1024 and sg.query(B.AGO_Q_TILE_ROWS) >= 1
        sg.close()
    # the two depthwise convolutions of the pair kernel are stride 1; a strided pair has no kernel
    wl = WL.dw_dw("x", [1], 1, 8, 16)
    ops = list(wl.ops); ops[3] = ("conv2d", dict(O=16, R=3, S=3, stride=2, pad=1, groups=16))
    _expect_fail(ops, wl.input_shapes, B.AGO_ERR_UNSUPPORTED, mode="fused", needle="family")
    # pointwise pair: more middle channels than tensor memory holds
    wl = WL.pw_pw("x", [1], 1, 8, 64, 512, 64)
    _expect_fail(wl.ops, wl.input_shapes, B.AGO_ERR_UNSUPPORTED, mode="fused", needle="256")
    # the attention kernel takes the row maximum of the raw scores: a non-positive scale is left to the unfused modes
    wl = WL.attention("x", [1], 1, 64, 1, 64)
    ops = list(wl.ops); ops[1] = ("scale", dict(f=-0.125))
    _expect_fail(ops, wl.input_shapes, B.AGO_ERR_UNSUPPORTED, mode="fused", needle="positive")
    B.Subgraph(ops, wl.input_shapes, mode="per_mini_subgraph").close()
    # a transpose of other axes than the two middle ones is not a row permutation the chain kernel knows
    wl = WL.unfold_chain("x", [1], 2, 4, 8, 16, 32)
    ops = list(wl.ops); ops[4] = ("transpose", dict(a=0, b=1)); ops[5] = ("reshape", dict(shape=(64, 16))); ops[7] = ("reshape", dict(shape=(4, 2, 8, 32)))
    _expect_fail(ops, wl.input_shapes, B.AGO_ERR_UNSUPPORTED, mode="fused", needle="family")


def test_feed_forward_planner_picks_the_cluster_kernel_where_the_shape_splits():
    # cluster kernels on many row blocks: no workspace (nothing is reduced through device memory) as long as the blocks
    # fill whole rounds of resident clusters; the blocks of a last, partial round are split over two or more clusters that
    # write an fp32 plane each; few row blocks (their hidden tiles split over several clusters) and the kernel without
    # clusters: an fp32 buffer over all rows
    def ws(M, K, hid, out):
        wl = WL.ffn("x", [1], M, K, hid, 1, d_out=out)
        sg = B.Subgraph(wl.ops, wl.input_shapes, mode="fused")
        w = sg.workspace_bytes
        sg.close()
        return w
    assert ws(33 * 256, 768, 3072, 768) == 0       # paired clusters: 33 blocks of 256 rows = one whole round of 33 resident clusters
    assert ws(12288, 768, 3072, 768) == 2 * 15 * 256 * 768 * 4   # 48 blocks: one whole round, the other 15 split in two parts, an fp32 plane each
    assert ws(40 * 256 - 100, 64, 512, 256) == 2 * (40 * 256 - 100 - 33 * 256) * 256 * 4   # 7 blocks (the last ragged) in two parts
    assert ws(36 * 256, 128, 768, 512) == 3 * (3 * 256) * 512 * 4     # 3 blocks in three parts of one step
    assert ws(9637, 64, 256, 384) == 0             # clusters of 2, ragged last row block
    assert ws(512, 768, 3072, 768) >= 512 * 768 * 4    # four row blocks: six clusters each
    assert ws(12800, 256, 384, 256) >= 12800 * 256 * 4  # three hidden tiles, 256 columns: no cluster size divides both


def test_layout_operators_in_the_planner():
    wl = WL.get("unfold_96", batch=2)
    per_op = B.Subgraph(wl.ops, wl.input_shapes, mode="per_op")
    mini = B.Subgraph(wl.ops, wl.input_shapes, mode="per_mini_subgraph")
    assert per_op.output_shape == (2, 256, 4, 192)
    assert per_op.query(B.AGO_Q_NUM_LAUNCHES) == 4        # GEMM | add | transpose | GEMM: reshapes are views
    assert mini.query(B.AGO_Q_NUM_LAUNCHES) == 3          # GEMM + add | transpose | GEMM
    # intermediates of that mode: the middle tensor before and after the transpose, written and read once each
    assert mini.query(B.AGO_Q_INTERMEDIATE_BYTES) == 2 * 2 * (2 * 4 * 256 * 96) * 2
    n = per_op.query(B.AGO_Q_NUM_LINKS)
    assert [per_op.query(B.AGO_Q_LINK_CATEGORY, i) for i in range(n)] == [B.AGO_LINK_DOWNSTREAM_POINTWISE]
    rs = lambda *shape: ("reshape", dict(shape=shape))
    _expect_fail([("relu", {}), rs(4, 16)], [(8, 8)], B.AGO_ERR_SHAPE, needle="last dimension")
    _expect_fail([("relu", {}), rs(3, 8)], [(8, 8)], B.AGO_ERR_SHAPE, needle="element count")
    _expect_fail([rs(4, 2, 8)], [(8, 8)], B.AGO_ERR_UNSUPPORTED, needle="follow")
    _expect_fail([("relu", {}), ("transpose", dict(a=0, b=2))], [(2, 4, 8)], B.AGO_ERR_SHAPE, needle="axes")
    _expect_fail([("relu", {}), ("transpose", dict(a=1, b=1))], [(2, 4, 8, 8)], B.AGO_ERR_SHAPE, needle="axes")


def _expect_fail(ops, shapes, status, mode="per_op", dtype=B.AGO_BF16, needle=""):
    with pytest.raises(B.AgoError) as e:
        B.Subgraph(ops, shapes, mode=mode, dtype=dtype)
    assert e.value.status == status, str(e.value)
    assert needle in str(e.value)


def test_create_rejects_bad_descriptors():
    conv = lambda **k: ("conv2d", dict(dict(O=8, R=3, S=3, stride=1, pad=1, groups=1), **k))
    _expect_fail([conv()], [(4, 8)], B.AGO_ERR_SHAPE, needle="NHWC")
    _expect_fail([conv(O=12)], [(1, 4, 4, 8)], B.AGO_ERR_SHAPE, needle="multiple")
    _expect_fail([conv(groups=4)], [(1, 4, 4, 8)], B.AGO_ERR_SHAPE, needle="groups")
    _expect_fail([conv(R=7, pad=0)], [(1, 4, 4, 8)], B.AGO_ERR_SHAPE, needle="empty")
    _expect_fail([("gemm", dict(N=0))], [(4, 8)], B.AGO_ERR_SHAPE)
    _expect_fail([("add_input", dict(input=3))], [(4, 8)], B.AGO_ERR_SHAPE)
    _expect_fail([("qkt", dict(input=1, heads=3, head_dim=8))], [(1, 8, 16), (1, 8, 16)], B.AGO_ERR_SHAPE)
    _expect_fail([("relu", {})], [(4, 7)], B.AGO_ERR_SHAPE, needle="16-byte")
    _expect_fail([("gemm", dict(N=8))], [(4, 8)], B.AGO_ERR_UNSUPPORTED, dtype=B.AGO_FP32)
    # a chain that is valid but matches no fused family
    _expect_fail([("gemm", dict(N=8)), ("relu", {})], [(4, 8)], B.AGO_ERR_UNSUPPORTED, mode="fused", needle="family")
    d, _ = B.make_desc([("relu", {})], [(8, 8)], "per_op")
    d.ops[0].kind = 99
    assert not B.ago_subgraph_create(d) and B.ago_last_error()[0] == B.AGO_ERR_INVALID_ARG
    d, _ = B.make_desc([("relu", {})], [(8, 8)], "per_op")
    d.mode = 7
    assert not B.ago_subgraph_create(d) and B.ago_last_error()[0] == B.AGO_ERR_INVALID_ARG


def test_null_and_misaligned_arguments_are_rejected_before_any_cuda_call():
    wl = WL.get("mbv2_14")
    sg = B.Subgraph(wl.ops, wl.input_shapes, mode="per_op")
    lib = B.load()
    assert lib.ago_subgraph_run(None, None, None, None, None) == B.AGO_ERR_INVALID_ARG
    assert lib.ago_subgraph_run(sg._h, None, None, None, None) == B.AGO_ERR_INVALID_ARG
    good = [0x1000] * 8
    assert B.ago_subgraph_run(sg._h, [0], good, good) == B.AGO_ERR_INVALID_ARG
    assert B.ago_subgraph_run(sg._h, [0x1004], good, good) == B.AGO_ERR_ALIGNMENT
    assert B.ago_subgraph_run(sg._h, good, [0x1000, 0x1008] + good, good) == B.AGO_ERR_ALIGNMENT
    assert B.ago_subgraph_set_workspace(sg._h, 0x1010, 1 << 30) == B.AGO_ERR_ALIGNMENT
    assert B.ago_subgraph_set_workspace(sg._h, 0x1000, 16) == B.AGO_ERR_WORKSPACE
    assert B.ago_subgraph_workspace_bytes(None) == 0
    B.ago_subgraph_destroy(None)
    sg.close()


def test_launch_floor_entry_validates_its_sizes_before_any_cuda_call():
    lib = B.load()
    for grid, block, smem in ((0, 128, 0), (70000, 128, 0), (1, 0, 0), (1, 2048, 0), (1, 128, -1), (1, 128, 300 * 1024)):
        assert lib.ago_launch_empty(grid, block, smem, None) == B.AGO_ERR_INVALID_ARG
        assert "ago_launch_empty" in B.ago_last_error()[1]


def test_bf16_helpers_round_to_nearest_even():
    x = np.array([1.0, 1.00390625, 1.001953125, 1.005859375, -2.5, 3.0e38], dtype=np.float32)
    r = WL.bf16_round(x)
    # 1 + 2^-8 is a tie between 1 and 1 + 2^-7 -> even (1.0); 1 + 3*2^-9 rounds up to 1 + 2^-7
    assert r[0] == 1.0 and r[1] == 1.0 and r[2] == 1.0 and r[3] == np.float32(1.0078125) and r[4] == -2.5
    import torch
    t = torch.from_numpy(x).to(torch.bfloat16).float().numpy()
    assert np.array_equal(r, t)


def test_auto_mode_fuses_unless_the_contractions_bound_both_modes():
    # AGO_MODE_AUTO resolves at create time (host only): chains whose intermediates dominate the traffic are fused;
    # the feed-forward chain on many rows (two large GEMMs, Section VI-B's pointwise -> pointwise observation) and chains
    # without a fused kernel run per mini-subgraph; the feed-forward chain on few rows is fused (its unfused GEMMs
    # cannot fill the SMs, the fused kernel splits the hidden dimension over clusters)
    from paper_2212_01005_b200 import workloads as WL
    want = {"attn_384": B.AGO_MODE_FUSED, "mbv2_56": B.AGO_MODE_FUSED, "mbv2_28s2": B.AGO_MODE_FUSED, "resnet_56": B.AGO_MODE_FUSED,
            "pw_pw_56": B.AGO_MODE_FUSED, "dw_dw_56": B.AGO_MODE_FUSED, "unfold_96": B.AGO_MODE_FUSED,
            "ffn_12288": B.AGO_MODE_PER_MINI_SUBGRAPH, "ffn_512": B.AGO_MODE_FUSED}
    for name, mode in want.items():
        wl = WL.get(name)
        sg = B.Subgraph(wl.ops, wl.input_shapes, mode="auto")
        assert sg.query(B.AGO_Q_MODE) == mode, name
        same = B.Subgraph(wl.ops, wl.input_shapes, mode="fused" if mode == B.AGO_MODE_FUSED else "per_mini_subgraph")
        assert sg.query(B.AGO_Q_NUM_LAUNCHES) == same.query(B.AGO_Q_NUM_LAUNCHES)
        same.close()
        sg.close()
    lone = B.Subgraph([("gemm", {"N": 64}), ("relu", {})], [(256, 64)], mode="auto")     # no fused family: not an error in AUTO
    assert lone.query(B.AGO_Q_MODE) == B.AGO_MODE_PER_MINI_SUBGRAPH
    lone.close()
    with pytest.raises(B.AgoError):
        B.Subgraph([("gemm", {"N": 0})], [(256, 64)], mode="auto")                        # malformed in every mode
