"""Parity of the CUDA path (through the C-ABI) against the fp64 CPU oracle on
the same seeded inputs. Tolerance (bf16 in, fp32 accumulate):
max|gpu - ref| <= 1e-2 * max|ref| + 1e-3 over the whole output tensor; the
fp32-I/O depthwise check uses 1e-5 * max|ref|."""
import numpy as np
import pytest

from oracle import oracle as O
from paper_2212_01005_b200 import workloads as WL
from helpers import assert_close, rounding_share, run_gpu

pytestmark = pytest.mark.gpu

UNFUSED = ["per_op", "per_mini_subgraph"]


def small_workloads():
    """Small instances of every chain family: several tiles plus ragged tails."""
    return {
        "mbv2_14": WL.get("mbv2_14"),
        "mbv2_s1_odd": WL.mbv2_block("mbv2_s1_odd", [21], 3, 13, 24, 144, 24, 1, True),
        "mbv2_s2": WL.mbv2_block("mbv2_s2", [22], 2, 14, 32, 192, 64, 2, False),
        "mbv2_s2_odd": WL.mbv2_block("mbv2_s2_odd", [23], 2, 9, 16, 96, 32, 2, False),
        "ffn_small": WL.ffn("ffn_small", [24], 200, 128, 512, 1),
        "ffn_ragged": WL.ffn("ffn_ragged", [25], 77, 96, 264, 1),
        "ffn_rows_ragged": WL.ffn("ffn_rows_ragged", [30], 333, 256, 384, 1),
        # tall enough that the fused kernel keeps 2 / 3 hidden tiles per CTA (100 row blocks x 6 / 9 hidden tiles)
        "ffn_g2": WL.ffn("ffn_g2", [31], 12800, 128, 768, 1),
        "ffn_g3": WL.ffn("ffn_g3", [32], 12800, 128, 1152, 1),
        # enough row blocks for the thread-block-cluster kernel: clusters of 2, 3 and 4 CTAs, one and two steps,
        # 64 to 256 output columns per CTA, a ragged last row block
        "ffn_c2": WL.ffn("ffn_c2", [33], 9637, 64, 256, 1, d_out=384),
        "ffn_c3": WL.ffn("ffn_c3", [34], 6400, 128, 768, 1, d_out=192),
        "ffn_c4": WL.ffn("ffn_c4", [35], 4864, 64, 512, 1, d_out=1024),
        # the paired-cluster kernel (two CTA pairs on 256 rows): 128 / 256 / 384 output columns per pair, one to three steps
        # per row block, one and two row blocks per cluster, ragged last block
        "ffn_p1": WL.ffn("ffn_p1", [38], 8349, 64, 512, 1, d_out=256),
        "ffn_p2": WL.ffn("ffn_p2", [39], 7680, 128, 256, 1, d_out=512),
        "ffn_p3": WL.ffn("ffn_p3", [40], 12000, 192, 768, 1, d_out=768),
        # few row blocks: the hidden tiles of a row block are split over several clusters (ragged rows; clusters of 2 / 4)
        "ffn_s3": WL.ffn("ffn_s3", [41], 700, 128, 1536, 1, d_out=384),
        "ffn_s4": WL.ffn("ffn_s4", [42], 1024, 256, 1024, 1, d_out=512),
        # many rows on the paired-cluster kernel with a last, partial round of resident clusters (33 on a B200): 40 blocks of 256
        # rows, the last ragged, 7 of them split in two parts of one step; 36 blocks, 3 of them split in three parts
        "ffn_r2": WL.ffn("ffn_r2", [46], 40 * 256 - 100, 64, 512, 1, d_out=256),
        "ffn_r3": WL.ffn("ffn_r3", [47], 36 * 256, 128, 768, 1, d_out=512),
        "resnet_small": WL.resnet_block("resnet_small", [26], 2, 12, 64),
        "resnet_odd": WL.resnet_block("resnet_odd", [27], 1, 9, 32),
        "resnet_16ch": WL.resnet_block("resnet_16ch", [32], 2, 20, 16),
        # widths around the 28-column segments of the conv3x3 kernels: exactly one segment, a second segment of one
        # column, two full segments and one column of a third; heights that leave ragged last strips and tile rows
        "resnet_w28": WL.resnet_block("resnet_w28", [43], 1, 28, 64),
        "resnet_w29": WL.resnet_block("resnet_w29", [44], 2, 29, 32),
        "resnet_w57": WL.resnet_block("resnet_w57", [45], 1, 57, 16),
        "attn_small": WL.attention("attn_small", [28], 2, 128, 2, 64),
        "attn_ragged": WL.attention("attn_ragged", [29], 1, 200, 3, 64),
        # more query tiles than SMs: the persistent CTAs' runs of 1-2 and of 3-4 items cross from one head (and batch) into the next
        # at every position of a run; ragged last tiles
        "attn_runs2": WL.attention("attn_runs2", [36], 5, 200, 16, 64),
        "attn_runs4": WL.attention("attn_runs4", [37], 8, 296, 20, 64),
    }


_ref_cache = {}


def reference(name, wl, data):
    if name not in _ref_cache:
        _ref_cache[name] = O.run_chain(wl.ops, data["inputs"], data["weights"])
    return _ref_cache[name]


_full_cache = {}


def full_size_case(name):
    """A benchmark workload at the size bench.py times it: (workload, seeded data, oracle result of the WHOLE batch)."""
    if name not in _full_cache:
        wl = WL.get(name)
        data = WL.generate(wl)
        _full_cache.clear()          # one bench-sized fp64 reference at a time
        _full_cache[name] = (wl, data, O.run_chain(wl.ops, data["inputs"], data["weights"]))
    return _full_cache[name]


def check_whole_tensor(ago, name, mode):
    """Every element of the bench-sized output against the oracle, same tolerance as everywhere. On failure the message
    carries the diagnostic share of bf16 rounding of the intermediates (never the reference)."""
    wl, data, ref = full_size_case(name)
    gpu = run_gpu(ago, wl, data, mode)
    err = float(np.max(np.abs(gpu - ref)))
    bound = 1e-2 * float(np.max(np.abs(ref))) + 1e-3
    if not (np.isfinite(gpu).all() and err <= bound):
        worst = np.unravel_index(int(np.argmax(np.abs(gpu - ref))), ref.shape)
        raise AssertionError(f"{name}/{mode}: max abs err {err:.4g} > bound {bound:.4g} at {worst}; "
                             f"bf16 rounding of intermediates alone: {rounding_share(O, wl, data, ref):.4g}")
    return gpu


@pytest.mark.parametrize("mode", UNFUSED)
@pytest.mark.parametrize("name", list(small_workloads().keys()))
def test_unfused_modes_match_oracle(ago, name, mode):
    wl = small_workloads()[name]
    data = WL.generate(wl)
    ref = reference(name, wl, data)
    gpu = run_gpu(ago, wl, data, mode)
    assert_close(gpu, ref, what=f"{name}/{mode}")


def test_depthwise_fp32_io_matches_oracle_to_1e5(ago):
    # the 14x14x192 depthwise stage of the N=1 block, fp32 in / fp32 out, fused and per-op
    wl = WL.Workload("dw14", [0, 99], [(1, 14, 14, 192)],
                     [("conv2d", dict(O=192, R=3, S=3, stride=1, pad=1, groups=192)), ("bias_add", {}), ("relu6", {})],
                     samples=1, input_dist=["uniform"])
    rng = np.random.default_rng([0, 99])
    data = {"inputs": [rng.uniform(0, 6, size=(1, 14, 14, 192)).astype(np.float32)],
            "weights": [(rng.standard_normal((3, 3, 192)) * np.sqrt(2 / 9)).astype(np.float32),
                        rng.uniform(-0.1, 0.1, 192).astype(np.float32)]}
    ref = O.run_chain(wl.ops, data["inputs"], data["weights"])
    for mode in ("fused", "per_op", "per_mini_subgraph"):
        gpu = run_gpu(ago, wl, data, mode, fp32=True)
        err = np.max(np.abs(gpu - ref))
        assert err <= 1e-5 * np.max(np.abs(ref)), (mode, err)


@pytest.mark.parametrize("stride", [1, 2])
def test_depthwise_bf16_fused_mini_subgraph(ago, stride):
    wl = WL.Workload("dwb", [31, stride], [(2, 11, 13, 48)],
                     [("conv2d", dict(O=48, R=3, S=3, stride=stride, pad=1, groups=48)), ("bias_add", {}), ("relu6", {})],
                     samples=2, input_dist=["uniform"])
    data = WL.generate(wl)
    ref = O.run_chain(wl.ops, data["inputs"], data["weights"])
    assert_close(run_gpu(ago, wl, data, "fused"), ref, what="dw fused")


@pytest.mark.parametrize("tail", ["bias_relu", "bias", "none", "relu", "bias_add_relu"])
@pytest.mark.parametrize("shape", [(2, 23, 17, 16), (1, 40, 56, 64), (3, 9, 30, 32)])
def test_single_conv3x3_stage_epilogues(ago, shape, tail):
    # one 3x3 convolution of equal width with each simple-operator tail the tensor-core stage kernel accepts,
    # on images of several strips with ragged last strips and non-square extents
    ch = shape[3]
    ops = [("conv2d", dict(O=ch, R=3, S=3, stride=1, pad=1, groups=1))]
    for t in tail.split("_"):
        if t == "bias":
            ops.append(("bias_add", {}))
        elif t == "add":
            ops.append(("add_input", dict(input=0)))
        elif t == "relu":
            ops.append(("relu", {}))
    wl = WL.Workload("conv1", [71, ch, len(ops)], [shape], ops, samples=shape[0])
    data = WL.generate(wl)
    ref = O.run_chain(wl.ops, data["inputs"], data["weights"])
    for mode in UNFUSED:
        assert_close(run_gpu(ago, wl, data, mode), ref, what=f"conv1 {shape} {tail}/{mode}")


@pytest.mark.parametrize("shape", [(1, 1, 1, 16), (1, 2, 3, 32), (2, 5, 31, 64), (1, 33, 30, 16), (3, 17, 59, 32), (1, 40, 85, 16), (2, 3, 113, 16)])
def test_conv3x3_pair_odd_shapes_every_mode(ago, shape):
    # the residual block on non-square images from a single pixel to four and five 28-column segments, heights that are
    # not multiples of the four-row tiles, every channel count the tensor-core kernels take; fused and both unfused modes
    n, h, w, ch = shape
    ops = [("conv2d", dict(O=ch, R=3, S=3, stride=1, pad=1, groups=1)), ("bias_add", {}), ("relu", {}),
           ("conv2d", dict(O=ch, R=3, S=3, stride=1, pad=1, groups=1)), ("bias_add", {}), ("add_input", dict(input=0)), ("relu", {})]
    wl = WL.Workload("conv_pair_odd", [72, h, w, ch], [shape], ops, samples=n, input_dist=["relu_normal"])
    data = WL.generate(wl)
    ref = O.run_chain(wl.ops, data["inputs"], data["weights"])
    for mode in ("fused",) + tuple(UNFUSED):
        assert_close(run_gpu(ago, wl, data, mode), ref, what=f"conv pair {shape}/{mode}")


def test_padding_of_the_intermediate_with_large_bias(ago):
    # the halo of the depthwise / second conv input is zero, not act(bias)
    wl = WL.mbv2_block("pad", [33], 1, 6, 8, 16, 8, 1, True)
    data = WL.generate(wl)
    data["weights"][1] = np.full(16, 3.0, dtype=np.float32)      # expand bias: ReLU6(b1) = 3 in the halo if mishandled
    ref = O.run_chain(wl.ops, data["inputs"], data["weights"])
    for mode in UNFUSED:
        assert_close(run_gpu(ago, wl, data, mode), ref, what=f"pad/{mode}")


# ---- fused kernels -------------------------------------------------------------------

FUSED_SMALL = ["mbv2_14", "mbv2_s1_odd", "mbv2_s2", "mbv2_s2_odd", "attn_small", "attn_ragged", "attn_runs2", "attn_runs4", "ffn_small", "ffn_rows_ragged", "ffn_g2", "ffn_g3",
               "ffn_c2", "ffn_c3", "ffn_c4", "ffn_p1", "ffn_p2", "ffn_p3", "ffn_s3", "ffn_s4", "ffn_r2", "ffn_r3", "resnet_small", "resnet_odd", "resnet_16ch", "resnet_w28", "resnet_w29", "resnet_w57"]


@pytest.mark.parametrize("name", FUSED_SMALL)
def test_fused_matches_oracle(ago, name):
    wl = small_workloads()[name]
    data = WL.generate(wl)
    ref = reference(name, wl, data)
    gpu = run_gpu(ago, wl, data, "fused")
    assert_close(gpu, ref, what=f"{name}/fused")


@pytest.mark.parametrize("name", FUSED_SMALL)
def test_fused_agrees_with_unfused_chain(ago, name):
    # fusion is a loop transformation: same result as the library's own unfused chain, up to bf16 rounding
    wl = small_workloads()[name]
    data = WL.generate(wl)
    fused = run_gpu(ago, wl, data, "fused")
    mini = run_gpu(ago, wl, data, "per_mini_subgraph")
    scale = float(np.max(np.abs(mini)))
    assert float(np.max(np.abs(fused - mini))) <= 2e-2 * scale + 1e-3


UNFOLD_SMALL = {
    "unfold_small": lambda: WL.unfold_chain("unfold_small", [101], 2, 4, 64, 96, 192),      # 512 rows
    "unfold_ragged": lambda: WL.unfold_chain("unfold_ragged", [102], 3, 4, 25, 64, 128),    # 300 rows: ragged last tile
    "unfold_narrow": lambda: WL.unfold_chain("unfold_narrow", [103], 1, 9, 49, 24, 40),     # channel counts 8 mod 16
    "unfold_wide": lambda: WL.unfold_chain("unfold_wide", [104], 2, 4, 16, 128, 256),
}


@pytest.mark.parametrize("mode", UNFUSED)
@pytest.mark.parametrize("name", list(UNFOLD_SMALL.keys()))
def test_unfold_chain_unfused_modes_match_oracle(ago, name, mode):
    wl = UNFOLD_SMALL[name]()
    data = WL.generate(wl)
    ref = O.run_chain(wl.ops, data["inputs"], data["weights"])
    assert_close(run_gpu(ago, wl, data, mode), ref, what=f"{name}/{mode}")


@pytest.mark.parametrize("name", list(UNFOLD_SMALL.keys()))
def test_unfold_chain_fused_matches_oracle(ago, name):
    # one kernel: the transpose only permutes the rows between the two products
    wl = UNFOLD_SMALL[name]()
    data = WL.generate(wl)
    ref = O.run_chain(wl.ops, data["inputs"], data["weights"])
    assert_close(run_gpu(ago, wl, data, "fused"), ref, what=f"{name}/fused")


def test_unfold_chain_full_size_whole_tensor(ago):
    check_whole_tensor(ago, "unfold_96", "fused")


PAIR_SMALL = {
    "pw_dw_s1": lambda: WL.pw_dw("pw_dw_s1", [81], 2, 14, 32, 192, 1),
    "pw_dw_s1_odd": lambda: WL.pw_dw("pw_dw_s1_odd", [82], 3, 13, 24, 144, 1),
    "pw_dw_s2": lambda: WL.pw_dw("pw_dw_s2", [83], 2, 14, 32, 192, 2),
    "pw_dw_s2_odd": lambda: WL.pw_dw("pw_dw_s2_odd", [84], 2, 9, 16, 96, 2),
    "pw_dw_tall": lambda: WL.pw_dw("pw_dw_tall", [85], 1, 40, 24, 48, 1),
    "dw_pw_s1": lambda: WL.dw_pw("dw_pw_s1", [86], 2, 14, 192, 32, 1),
    "dw_pw_s1_odd": lambda: WL.dw_pw("dw_pw_s1_odd", [87], 3, 13, 144, 24, 1),
    "dw_pw_s2": lambda: WL.dw_pw("dw_pw_s2", [88], 2, 14, 192, 64, 2),
    "dw_pw_s2_odd": lambda: WL.dw_pw("dw_pw_s2_odd", [89], 2, 9, 96, 32, 2),
    "dw_pw_tall": lambda: WL.dw_pw("dw_pw_tall", [90], 1, 40, 48, 24, 1),
    "dw_pw_one_chunk": lambda: WL.dw_pw("dw_pw_one_chunk", [91], 1, 11, 16, 8, 1),
    "dw_dw_14": lambda: WL.dw_dw("dw_dw_14", [92], 2, 14, 192),
    "dw_dw_odd": lambda: WL.dw_dw("dw_dw_odd", [93], 3, 13, 48),
    "dw_dw_tall": lambda: WL.dw_dw("dw_dw_tall", [94], 1, 45, 32),
    "dw_dw_tiny": lambda: WL.dw_dw("dw_dw_tiny", [95], 1, 3, 16),
    "pw_pw_14": lambda: WL.pw_pw("pw_pw_14", [96], 2, 14, 192, 32, 192),
    "pw_pw_ragged": lambda: WL.pw_pw("pw_pw_ragged", [97], 3, 13, 144, 24, 144),          # 507 rows, channel counts 8 mod 16
    "pw_pw_act_first": lambda: WL.pw_pw("pw_pw_act_first", [98], 1, 20, 64, 128, 40, act1=True, act2=False),
    "pw_pw_act_both": lambda: WL.pw_pw("pw_pw_act_both", [99], 1, 9, 8, 8, 8, act1=True, act2=True),
    "pw_pw_linear": lambda: WL.pw_pw("pw_pw_linear", [100], 2, 16, 160, 128, 256, act1=False, act2=False),
}


@pytest.mark.parametrize("name", list(PAIR_SMALL.keys()))
def test_fused_pairs_match_oracle(ago, name):
    # the two-complex-operator pairs: stride 1 and 2, ragged strips, one to twelve channel chunks
    wl = PAIR_SMALL[name]()
    data = WL.generate(wl)
    ref = O.run_chain(wl.ops, data["inputs"], data["weights"])
    assert_close(run_gpu(ago, wl, data, "fused"), ref, what=f"{name}/fused")
    for mode in UNFUSED:
        assert_close(run_gpu(ago, wl, data, mode), ref, what=f"{name}/{mode}")


@pytest.mark.parametrize("name", ["pw_dw_56", "dw_pw_56", "dw_dw_56", "pw_pw_56"])
def test_fused_pairs_full_size_whole_tensor(ago, name):
    check_whole_tensor(ago, name, "fused")


def test_fused_mbv2_pads_the_intermediate_not_the_input(ago):
    wl = WL.mbv2_block("pad", [33], 1, 6, 8, 16, 8, 1, True)
    data = WL.generate(wl)
    data["weights"][1] = np.full(16, 3.0, dtype=np.float32)
    ref = O.run_chain(wl.ops, data["inputs"], data["weights"])
    assert_close(run_gpu(ago, wl, data, "fused"), ref, what="pad/fused")


@pytest.mark.parametrize("shape", [
    dict(N=2, H=7, c_in=16, c_exp=32, c_out=16, stride=1, residual=True),     # 32-byte input rows (Cin 16)
    dict(N=1, H=20, c_in=64, c_exp=64, c_out=40, stride=1, residual=False),   # 128-byte input rows, Cout not a multiple of 16
    dict(N=3, H=5, c_in=8, c_exp=16, c_out=8, stride=2, residual=False),      # one chunk, tiny image, odd size
    dict(N=1, H=30, c_in=40, c_exp=240, c_out=80, stride=2, residual=False),  # Cin padded 40 -> 64
    dict(N=1, H=32, c_in=64, c_exp=64, c_out=64, stride=1, residual=True),    # large 128-byte-row tile: more input slots than one staging pass
    dict(N=2, H=24, c_in=64, c_exp=384, c_out=64, stride=1, residual=True),   # many weight slots, 24 chunks
    dict(N=2, H=6, c_in=8, c_exp=16, c_out=8, stride=1, residual=True),       # one column segment per row
    dict(N=4, H=3, c_in=16, c_exp=32, c_out=24, stride=1, residual=False),    # images of one strip
    dict(N=2, H=2, c_in=16, c_exp=16, c_out=16, stride=2, residual=False),    # one output pixel per image
])
def test_fused_mbv2_shape_sweep(ago, shape):
    wl = WL.mbv2_block("sweep", [41, shape["H"], shape["c_in"]], shape["N"], shape["H"], shape["c_in"], shape["c_exp"],
                       shape["c_out"], shape["stride"], shape["residual"])
    data = WL.generate(wl)
    ref = O.run_chain(wl.ops, data["inputs"], data["weights"])
    assert_close(run_gpu(ago, wl, data, "fused"), ref, what=f"sweep {shape}")


@pytest.mark.parametrize("name", ["mbv2_56", "mbv2_28s2"])
def test_fused_full_size_whole_tensor(ago, name):
    # the benchmark's launch configuration, every element of every image against the oracle
    check_whole_tensor(ago, name, "fused")


def test_fused_attention_full_size_whole_tensor(ago):
    check_whole_tensor(ago, "attn_384", "fused")


def test_fused_attention_dominant_key_and_uniform_rows(ago):
    # one key dominates every query of head 0; head 1 has equal scores (uniform average of V)
    wl = WL.attention("attn_probe", [51], 1, 144, 2, 64)
    data = WL.generate(wl)
    q, k, v = (a.copy() for a in data["inputs"])
    q[:] = 0; k[:] = 0
    q[0, :, 0] = 1.0; k[0, 77, 0] = 640.0         # head 0: score 640 / 8 = 80 at key 77, 0 elsewhere
    data["inputs"] = [q, k, v]
    gpu = run_gpu(ago, wl, data, "fused")
    ref = O.run_chain(wl.ops, data["inputs"], data["weights"])
    assert_close(gpu, ref, what="attn probe")
    np.testing.assert_allclose(gpu[0, :, :64], np.broadcast_to(v[0, 77, :64].astype(np.float64), (144, 64)), atol=2e-2)


@pytest.mark.parametrize("S", [200, 384])
def test_fused_attention_scores_far_above_the_first_keys(ago, S):
    # The kernel takes a row's exponentials relative to the maximum of its first 32 scores of each half and repeats the
    # pass with the true row maximum when that reference turns out too low. Here the scores grow along the keys: row r
    # scores g_r * 8 * (k // 8) on key k, with g_r = 1 for rows that need the exact pass (at S = 200 the last keys of the
    # second half lie 80 powers of two above its first 32) and g_r = 1/4 for rows that, at S = 200, do not; both kinds
    # sit in every warp.
    wl = WL.attention("attn_growing", [53], 1, S, 2, 64)
    data = WL.generate(wl)
    q, k, v = (a.copy() for a in data["inputs"])
    q[:] = 0; k[:] = 0
    for head in range(2):
        q[0, 0::2, head * 64] = 1.0
        q[0, 1::2, head * 64] = 0.25
        k[0, :, head * 64] = 64.0 * (np.arange(S) // 8)
    data["inputs"] = [q, k, v]
    gpu = run_gpu(ago, wl, data, "fused")
    ref = O.run_chain(wl.ops, data["inputs"], data["weights"])
    assert np.isfinite(gpu).all()
    assert_close(gpu, ref, what=f"attn growing scores S={S}")


@pytest.mark.parametrize("S", [128, 200, 256, 384])
def test_fused_attention_each_query_selects_its_keys(ago, S):
    # Query row r scores 32 on the keys j with j = r + 5 (mod 64) and 0 elsewhere, so its probabilities are (almost) one-hot
    # per 64-key block; V row k carries k + 1 in the column of its block. The output names, per query and key block, the V
    # row that met the probability: a product that pairs a 16-key step of P with the wrong rows of V shows up as a wrong
    # integer. Key counts of one, two and three 128-key loads, with and without a ragged last tile.
    wl = WL.attention("attn_select", [52], 1, S, 1, 64)
    q = np.zeros((1, S, 64), np.float32); k = np.zeros_like(q); v = np.zeros_like(q)
    for r in range(S):
        q[0, r, (r + 5) % 64] = 16.0
        k[0, r, r % 64] = 16.0
        v[0, r, r // 64] = (r % 64) + 1
    data = {"inputs": [q, k, v], "weights": []}
    gpu = run_gpu(ago, wl, data, "fused")
    ref = O.run_chain(wl.ops, data["inputs"], data["weights"])
    assert_close(gpu, ref, what=f"attn_select S={S}")
    nb = (S + 63) // 64
    for blk in range(nb):
        rows = np.arange(64)
        want = (rows + 5) % 64
        present = blk * 64 + want < S                       # the last block of a ragged S lacks some keys
        hits = np.array([sum(1 for b2 in range(nb) if b2 * 64 + w < S) for w in want])
        got = gpu[0, :64, blk].astype(np.float64) * hits - 1
        np.testing.assert_allclose(got[present], want[present], atol=0.26, err_msg=f"S={S} key block {blk}")


@pytest.mark.parametrize("name", ["resnet_56", "attn_384", "ffn_12288", "pw_dw_56", "dw_dw_56", "pw_pw_56", "unfold_96"])
def test_fused_kernels_repeat_bit_for_bit(ago, name):
    # These kernels have no atomics and a fixed accumulation order: back-to-back launches at the bench's sizes, with other
    # launches of the same kernel still in flight on the GPU, must reproduce the first result exactly. A race between the
    # asynchronous copies, the tensor core and the CUDA-core stages shows up as a difference in some launch.
    # (Not in the list: the kernels with a project GEMM fed by two thread groups -- the inverted-residual block and the
    # depthwise -> pointwise pair -- add the channel chunks in the order the groups finish them, and the split-reduction
    # feed-forward kernel adds with atomics: their last bit may differ from launch to launch.)
    import torch
    wl = WL.get(name)
    data = WL.generate(wl)
    sg = ago.Subgraph(wl.ops, wl.input_shapes, mode="fused")
    from helpers import to_device
    ins, ws = to_device(wl, data)
    outs = [torch.empty(wl.output_shape, dtype=torch.bfloat16, device="cuda:0") for _ in range(6)]
    for o in outs:
        sg.run(ins, ws, out=o)
    torch.cuda.synchronize()
    assert sg.status() == ago.AGO_OK, ago.ago_last_error()
    first = outs[0].view(torch.int16)
    for k, o in enumerate(outs[1:], 1):
        assert torch.equal(first, o.view(torch.int16)), f"{name}: launch {k} differs from launch 0"
    sg.close()


def test_fused_attention_full_size_constant_values_come_back(ago):
    # Any-size property, every element of the bench's output checked: when all keys of a (batch, head) carry the same value
    # vector, the softmax-weighted mean returns that vector whatever the scores are. The kernel divides a sum of bf16-rounded
    # probabilities times the constant by the fp32 sum of the unrounded ones: within 2^-9 relative.
    wl = WL.get("attn_384")
    data = WL.generate(wl)
    q, k, v = data["inputs"]
    B_, S, E = v.shape
    const = ((np.arange(B_)[:, None] * 7 + np.arange(E)[None, :] * 3) % 33 - 16).astype(np.float32) / 8.0   # bf16-exact
    v = np.broadcast_to(const[:, None, :], (B_, S, E)).copy()
    data["inputs"] = [q, k, v]
    gpu = run_gpu(ago, wl, data, "fused")
    err = np.abs(gpu - const[:, None, :].astype(np.float64))
    assert err.max() <= 2.0 * 2.0 ** -8, f"max deviation {err.max():.4g} at {np.unravel_index(err.argmax(), err.shape)}"


@pytest.mark.parametrize("name", ["mbv2_56", "mbv2_28s2"])
def test_fused_inverted_residual_full_size_with_zero_expand_weights(ago, name):
    # Any-size property at the bench's size, every output element checked against a closed form: with zero expand
    # weights the expanded tensor is relu6(b1) inside the image and 0 in the padding ring the depthwise convolution sees,
    # so the depthwise output depends on a pixel's position only through the taps that fall inside the image. A strip
    # halo that is padded, dropped or taken from the wrong row changes the border rows of some strip.
    wl = WL.get(name)
    data = WL.generate(wl)
    w1, b1, wd, bd, w3, b3 = (a.astype(np.float64) for a in data["weights"])
    data["weights"][0] = np.zeros_like(data["weights"][0])
    x = data["inputs"][0].astype(np.float64)
    N, H, W, _ = x.shape
    stride = wl.ops[3][1]["stride"]
    Ho, Wo = wl.output_shape[1], wl.output_shape[2]
    e = np.clip(b1, 0.0, 6.0)                                    # [Cexp]
    ho, wo = np.arange(Ho) * stride, np.arange(Wo) * stride
    acc = np.zeros((Ho, Wo, e.size))
    for r in range(3):
        for c in range(3):
            inside = ((ho + r - 1 >= 0) & (ho + r - 1 < H))[:, None] & ((wo + c - 1 >= 0) & (wo + c - 1 < W))[None, :]
            acc += inside[:, :, None] * (wd[r, c] * e)[None, None, :]
    d = np.clip(acc + bd, 0.0, 6.0)                              # [Ho, Wo, Cexp], the same for every image
    out = d @ w3.reshape(w3.shape[0], -1).T + b3                 # [Ho, Wo, Cout]
    ref = np.broadcast_to(out, (N,) + out.shape).copy()
    if len(wl.ops) == 9:
        ref += x
    gpu = run_gpu(ago, wl, data, "fused")
    assert_close(gpu, ref, what=f"{name} with zero expand weights")


def _taps_inside(H, W):
    """inside[r][c]: [H, W] mask of the output pixels whose tap (r, c) of a 3x3 window, pad 1, stride 1 lies in the image."""
    h, w = np.arange(H), np.arange(W)
    return [[((h + r - 1 >= 0) & (h + r - 1 < H))[:, None] & ((w + c - 1 >= 0) & (w + c - 1 < W))[None, :] for c in range(3)]
            for r in range(3)]


@pytest.mark.parametrize("name", ["resnet_56", "dw_dw_56", "pw_dw_56", "ffn_12288", "pw_pw_56", "dw_pw_56"])
def test_fused_pairs_full_size_with_zero_first_weights(ago, name):
    # The first complex operator gets zero weights, so its output is act(b1) everywhere inside the image (and 0 in the
    # padding ring a 3x3 second operator sees). The result then has a closed form by pixel position, the same for every
    # image or row: every element of the bench-sized output is checked, whichever CTA, strip or cluster wrote it.
    wl = WL.get(name)
    data = WL.generate(wl)
    data["weights"][0] = np.zeros_like(data["weights"][0])
    x = data["inputs"][0].astype(np.float64)
    w2, b2 = data["weights"][2].astype(np.float64), data["weights"][3].astype(np.float64)
    b1 = data["weights"][1].astype(np.float64)
    if name == "resnet_56":
        N, H, W, _ = x.shape
        mid = np.maximum(b1, 0.0)
        ins = _taps_inside(H, W)
        out = np.zeros((H, W, w2.shape[0]))
        for r in range(3):
            for c in range(3):
                out += ins[r][c][:, :, None] * (w2[:, r, c, :] @ mid)[None, None, :]
        ref = np.maximum(out[None] + b2 + x, 0.0)
    elif name in ("dw_dw_56", "pw_dw_56"):
        N, H, W, _ = x.shape
        mid = np.clip(b1, 0.0, 6.0)
        ins = _taps_inside(H, W)
        out = np.zeros((H, W, mid.size))
        for r in range(3):
            for c in range(3):
                out += ins[r][c][:, :, None] * (w2[r, c] * mid)[None, None, :]
        ref = np.broadcast_to(np.clip(out + b2, 0.0, 6.0), x.shape[:3] + (mid.size,))
    elif name == "dw_pw_56":
        # zero depthwise weights: relu6(b1) at every pixel, padding or not; the pointwise product of that vector
        ref = np.broadcast_to(w2.reshape(w2.shape[0], -1) @ np.clip(b1, 0.0, 6.0) + b2, wl.output_shape)
    else:
        # no window: every row / pixel gives the same vector; the oracle computes it for one row / pixel
        one = [x[:1]] if name == "ffn_12288" else [x[:1, :1, :1]]
        row = O.run_chain(wl.ops, one, data["weights"])
        ref = np.broadcast_to(row.reshape(-1), wl.output_shape)
    gpu = run_gpu(ago, wl, data, "fused")
    assert_close(gpu, np.asarray(ref, np.float64), what=f"{name} with zero first weights")


def test_fused_ffn_512_full(ago):
    wl = WL.get("ffn_512")
    data = WL.generate(wl)
    ref = O.run_chain(wl.ops, data["inputs"], data["weights"])
    gpu = run_gpu(ago, wl, data, "fused")
    assert_close(gpu, ref, what="ffn_512 fused")
    # the accumulation buffer must be left clean: a second and third run give the same bits
    import torch
    from helpers import to_device
    sg = ago.Subgraph(wl.ops, wl.input_shapes, mode="fused")
    ins, ws = to_device(wl, data)
    a = sg.run(ins, ws).clone(); b = sg.run(ins, ws).clone(); c = sg.run(ins, ws).clone()
    torch.cuda.synchronize()
    for t in (a, b, c):
        assert_close(t.float().cpu().numpy().astype(np.float64), ref, what="ffn_512 repeated run")
    sg.close()


def test_fused_ffn_12288_rows_of_every_block(ago):
    # Rows are independent samples of the chain. The oracle needs ~2.4 G fp64 MACs per 512 rows, so it checks nine rows
    # of EVERY block of 128 rows (first, last and seven seeded ones: every row block, cluster and CTA of the launch is
    # covered), and the library's own per-mini-subgraph chain -- checked against the oracle the same way -- covers
    # every element.
    wl = WL.get("ffn_12288")
    data = WL.generate(wl)
    x = data["inputs"][0]
    rng = np.random.default_rng([4, 1, 7])
    rows = np.concatenate([np.sort(np.concatenate([[0, 127], rng.choice(np.arange(1, 127), 7, replace=False)])) + b * 128
                           for b in range(x.shape[0] // 128)])
    ref = O.run_chain(wl.ops, [x[rows]], data["weights"])
    fused = run_gpu(ago, wl, data, "fused")
    assert_close(fused[rows], ref, what="ffn_12288 fused, rows of every block")
    mini = run_gpu(ago, wl, data, "per_mini_subgraph")
    assert_close(mini[rows], ref, what="ffn_12288 per_mini_subgraph, rows of every block")
    # every element: fusion is a loop transformation, both modes round H to bf16 at the same point
    scale = float(np.max(np.abs(mini)))
    diff = np.abs(fused - mini)
    assert float(diff.max()) <= 1e-2 * scale + 1e-3, f"fused vs per-mini-subgraph: {diff.max():.4g} at {np.unravel_index(diff.argmax(), diff.shape)}"


def test_fused_conv3x3_pads_the_intermediate_not_the_input(ago):
    # with a large positive first bias, ReLU(b1) in the halo of the intermediate would leak into the border
    wl = WL.resnet_block("respad", [61], 1, 10, 16)
    data = WL.generate(wl)
    data["weights"][1] = np.full(16, 2.0, dtype=np.float32)
    ref = O.run_chain(wl.ops, data["inputs"], data["weights"])
    assert_close(run_gpu(ago, wl, data, "fused"), ref, what="resnet pad/fused")


@pytest.mark.parametrize("name", ["mbv2_56", "mbv2_28s2", "resnet_56", "pw_pw_56", "attn_384"])
def test_unfused_baseline_full_size_whole_tensor(ago, name):
    # the per-mini-subgraph baseline at the size the bench times it (tensor-core stage kernels, their tile choices)
    check_whole_tensor(ago, name, "per_mini_subgraph")


def test_fused_resnet_full_size_whole_tensor(ago):
    check_whole_tensor(ago, "resnet_56", "fused")


def test_fused_ffn_workspace_lent_to_another_handle(ago):
    # The split-reduction feed-forward kernel relies on a zeroed workspace that it leaves zeroed. A caller that lends the
    # buffer to another handle in between re-attaches it (ago_subgraph_set_workspace), which makes the next run zero it
    # again: fused and unfused handles alternate on ONE buffer and every fused result stays correct.
    import torch
    from helpers import to_device
    wl = WL.get("ffn_512")
    data = WL.generate(wl)
    ref = O.run_chain(wl.ops, data["inputs"], data["weights"])
    fused = ago.Subgraph(wl.ops, wl.input_shapes, mode="fused")
    mini = ago.Subgraph(wl.ops, wl.input_shapes, mode="per_mini_subgraph")
    need = max(fused.workspace_bytes, mini.workspace_bytes)
    assert fused.workspace_bytes > 0
    buf = torch.empty(need + 256, dtype=torch.uint8, device="cuda:0")
    base = (buf.data_ptr() + 255) & ~255
    ins, ws = to_device(wl, data)
    for h in (fused, mini):
        h._ws = buf
    for rnd in range(3):
        assert ago.ago_subgraph_set_workspace(mini._h, base, need) == ago.AGO_OK
        m = mini.run(ins, ws)                      # fills the shared buffer with the hidden activations
        assert ago.ago_subgraph_set_workspace(fused._h, base, need) == ago.AGO_OK
        f = fused.run(ins, ws)
        torch.cuda.synchronize()
        assert fused.status() == ago.AGO_OK and mini.status() == ago.AGO_OK, ago.ago_last_error()
        assert_close(f.float().cpu().numpy().astype(np.float64), ref, what=f"ffn_512 fused after lending, round {rnd}")
        assert_close(m.float().cpu().numpy().astype(np.float64), ref, what=f"ffn_512 unfused, round {rnd}")
    fused.close(); mini.close()


@pytest.mark.parametrize("name", ["ffn_small", "ffn_c3", "mbv2_14", "attn_small", "resnet_small"])
def test_auto_mode_matches_oracle(ago, name):
    # AGO_MODE_AUTO resolves to the fused kernel or to the per-mini-subgraph chain; either way the result is the chain's
    wl = small_workloads()[name]
    data = WL.generate(wl)
    assert_close(run_gpu(ago, wl, data, "auto"), reference(name, wl, data), what=f"{name}/auto")
