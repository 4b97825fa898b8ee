"""Redundancy calculator of the C ABI (host-only) against brute-force counting and the paper's figures."""
import itertools

import pytest

from oracle import redundancy as R
from paper_2212_01005_b200 import binding as B


def query(**kw):
    return B.ago_fusion_redundancy(**kw)


CASES = [
    # (N, O1, O2, R2, C2, s, H2, W2, o2, h2, w2, depthwise2)
    (1, 3, 4, 3, 3, 1, 6, 7, 1, 1, 4, False),
    (2, 2, 5, 3, 3, 1, 5, 9, 2, 2, 3, False),      # ragged in every dimension
    (1, 4, 4, 3, 3, 1, 6, 6, 2, 6, 6, True),       # depthwise, spatial dims untiled
    (1, 4, 4, 3, 3, 1, 6, 6, 4, 2, 3, True),       # depthwise, spatial dims tiled: halo recomputation
    (1, 3, 6, 1, 1, 1, 5, 8, 6, 2, 3, False),      # pointwise, all output channels in the tile
    (1, 3, 6, 1, 1, 1, 5, 8, 2, 5, 8, False),      # pointwise, output channels tiled: recomputed per channel tile
    (1, 2, 3, 3, 3, 2, 4, 5, 3, 2, 2, False),      # stride 2
    (1, 2, 2, 5, 1, 1, 4, 4, 1, 3, 3, True),       # 5 x 1 window
    (1, 2, 3, 3, 3, 1, 4, 4, 99, 99, 99, False),   # tile larger than the tensor: one tile
]


@pytest.mark.parametrize("case", CASES)
def test_matches_brute_force(case):
    N, O1, O2, R2, C2, s, H2, W2, o2, h2, w2, dw = case
    got = query(N=N, O1=O1, I1=3, R1=3, C1=3, O2=O2, R2=R2, C2=C2, stride2=s, H2=H2, W2=W2, o2=o2, h2=h2, w2=w2,
                depthwise2=int(dw))
    fused, tiles = R.upstream_elems_fused(N, O1, O2, R2, C2, s, H2, W2, o2, h2, w2, dw)
    unfused = R.upstream_elems_unfused(N, O1, O2, R2, C2, s, H2, W2)
    assert got["upstream_elems_fused"] == fused
    assert got["upstream_elems_unfused"] == unfused
    assert got["num_tiles"] == tiles
    assert got["upstream_macs_fused"] == fused * 27 and got["upstream_macs_unfused"] == unfused * 27
    assert got["factor"] == pytest.approx(fused / unfused)


def test_paper_conv_conv_example():
    # Section III-B, the conv -> conv listing: downstream tile 1 x 1 x 16 on O2 x H2 x W2. The upstream reduction
    # body runs N O2 H2 (W2/16) O1 R2 (15 + C2) times after fusion against N O1 (H2 + R2 - 1)(W2 + C2 - 1) before.
    N, O1, O2, H2, W2, R2, C2 = 2, 5, 7, 6, 32, 3, 3
    got = query(N=N, O1=O1, O2=O2, R2=R2, C2=C2, H2=H2, W2=W2, o2=1, h2=1, w2=16)
    assert got["upstream_elems_fused"] == N * O2 * H2 * (W2 // 16) * O1 * R2 * (15 + C2)
    assert got["upstream_elems_unfused"] == N * O1 * (H2 + R2 - 1) * (W2 + C2 - 1)
    assert got["category"] == B.AGO_LINK_GENERAL
    # the two sources of redundancy named there: O2-fold over the channel tiles, and the window overlap
    assert got["factor"] == pytest.approx(O2 * (H2 * W2 * R2 * (15 + C2)) / ((H2 + R2 - 1) * (W2 + C2 - 1) * 16))


def test_recommended_tilings_have_no_recomputation():
    # downstream depthwise: tile H2 W2 o2 (spatial dims untiled, channels tiled) -> factor 1
    got = query(O1=32, O2=32, R2=3, C2=3, H2=14, W2=14, o2=8, h2=14, w2=14, depthwise2=1)
    assert got["factor"] == 1.0 and got["category"] == B.AGO_LINK_DOWNSTREAM_DEPTHWISE
    # downstream pointwise: tile h2 w2 O2 (all output channels, rows tiled) -> factor 1
    got = query(O1=144, O2=24, R2=1, C2=1, H2=56, W2=56, o2=24, h2=14, w2=56)
    assert got["factor"] == 1.0 and got["category"] == B.AGO_LINK_DOWNSTREAM_POINTWISE
    # general 3x3 with row strips of 14 over 56 rows (the conv3x3 pair kernel's tiling): (14 + 2) / 14 per strip
    got = query(O1=64, O2=64, R2=3, C2=3, H2=56, W2=56, o2=64, h2=14, w2=56)
    assert got["factor"] == pytest.approx(4 * 16 / 58.0)


def test_argument_errors():
    with pytest.raises(ValueError):
        query(O1=4, O2=5, R2=3, C2=3, H2=4, W2=4, o2=1, h2=1, w2=1, depthwise2=1)   # depthwise needs O2 == O1
    with pytest.raises(ValueError):
        query(O1=4, O2=4, R2=0, C2=3, H2=4, W2=4, o2=1, h2=1, w2=1)
    lib = B.load()
    assert lib.ago_fusion_redundancy(None, None) == B.AGO_ERR_INVALID_ARG
