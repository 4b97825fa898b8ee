"""Brute-force count of upstream work under intensive fusion (Section III-B).

TEST INFRASTRUCTURE ONLY: imported by tests/ (and by nothing in the product path).

Two stacked convolutions: the upstream one produces [N, O1, H1, W1]; the downstream one has an
R2 x C2 window, stride s and no padding and produces [N, O2, H2, W2], so H1 = (H2 - 1) s + R2 and
W1 = (W2 - 1) s + C2. The downstream output is cut into tiles of (o2, h2, w2); after fusion every
tile computes, inside its own loops, the set of upstream elements that its outputs read. The
functions below enumerate these sets element by element -- no closed form, no per-dimension
factorisation -- exactly as the fused loop nest of the section's conv -> conv listing would touch them.
"""
from __future__ import annotations

import itertools


def upstream_elems_unfused(N, O1, O2, R2, C2, s, H2, W2):
    """|GS1| in output elements: every upstream element once."""
    H1, W1 = (H2 - 1) * s + R2, (W2 - 1) * s + C2
    return N * O1 * H1 * W1


def upstream_elems_fused(N, O1, O2, R2, C2, s, H2, W2, o2, h2, w2, depthwise2=False):
    """Sum over the downstream tiles of the number of distinct upstream elements the tile reads."""
    o2, h2, w2 = min(o2, O2), min(h2, H2), min(w2, W2)
    total = 0
    tiles = 0
    for n in range(N):
        for c0, r0, q0 in itertools.product(range(0, O2, o2), range(0, H2, h2), range(0, W2, w2)):
            tiles += 1
            needed = set()
            for c in range(c0, min(c0 + o2, O2)):
                chans = [c] if depthwise2 else range(O1)   # depthwise: channel c reads upstream channel c
                for r in range(r0, min(r0 + h2, H2)):
                    for q in range(q0, min(q0 + w2, W2)):
                        for dr in range(R2):
                            for dc in range(C2):
                                for u in chans:
                                    needed.add((u, r * s + dr, q * s + dc))
            total += len(needed)
    return total, tiles
