"""Frontend graph partitioning (Eq. 1, Algorithm 1) of the C ABI against the Python restatement, the paper's
definitions and hand-worked graphs. Host only."""
import math

import numpy as np
import pytest

from oracle import cluster as C
from paper_2212_01005_b200 import binding as B
from paper_2212_01005_b200 import workloads as WL


def test_op_weight_is_eq1():
    # a 2-d convolution has seven loops (Section IV): N, O, H, W, I, R, S
    loops = [1, 64, 56, 56, 64, 3, 3]
    expect = 2.0 * math.prod(math.log(s) for s in loops) + 0.5
    assert B.ago_op_weight(loops, 2.0, 0.5) == pytest.approx(expect, rel=1e-12)
    assert C.op_weight(loops, 2.0, 0.5) == pytest.approx(expect, rel=1e-12)
    assert B.ago_op_weight([7], 1.0, 0.0) == pytest.approx(math.log(7))


def test_topological_stage_and_affix_set_definitions():
    # diamond with a long side: 0 -> 1 -> 3, 0 -> 2 -> 4 -> 3
    edges = [(0, 1), (1, 3), (0, 2), (2, 4), (4, 3)]
    ts = C.topological_stage(range(5), edges)
    assert ts == {0: 1, 1: 2, 2: 2, 4: 3, 3: 4}          # longest path from the root
    assert C.affix_set(1, range(5), edges, ts) == {0}    # 3 is adjacent but two stages below
    assert C.affix_set(4, range(5), edges, ts) == {2, 3}


def test_cyclic_dependency_example_is_never_produced():
    # Section IV's figure: Conv1 -> Conv2 -> Conv3 and Conv1 -> Conv3. Conv1 and Conv3 alone in one subgraph
    # would make the two subgraphs depend on each other; they are two stages apart, so never an affix pair.
    edges = [(0, 1), (1, 2), (0, 2)]
    weights = [5.0, 1.0, 5.0]
    for td in (6.5, 10.5, 100.0):
        got, cnt = B.ago_graph_cluster(weights, edges, td)
        assert got == C.cluster(weights, edges, td)
        assert C.is_acyclic_partition(got, edges)
        assert not (got[0] == got[2] and got[1] != got[0])
    assert B.ago_graph_cluster(weights, edges, 100.0)[0] == [0, 0, 0]   # a large threshold takes all three
    assert B.ago_graph_cluster(weights, edges, 1.0)[1] == 3             # a small one merges nothing


def test_hand_worked_chain():
    # chain 0-1-2-3 with weights 4, 1, 1, 4 and Td = 6: the heaviest (node 0) takes its lightest affix node 1
    # (weight 5 < 6), cannot take 2 (6 is not < 6) and leaves; then node 3 takes node 2.
    got, cnt = B.ago_graph_cluster([4.0, 1.0, 1.0, 4.0], [(0, 1), (1, 2), (2, 3)], 6.0)
    assert (got, cnt) == ([0, 0, 1, 1], 2)


def random_dag(rng, n, p):
    edges = [(i, j) for i in range(n) for j in range(i + 1, n) if rng.random() < p]
    perm = rng.permutation(n)                      # node ids not in topological order
    return [(int(perm[a]), int(perm[b])) for a, b in edges]


@pytest.mark.parametrize("seed", range(12))
def test_random_dags_match_restatement_and_are_acyclic(seed):
    rng = np.random.default_rng([91, seed])
    n = int(rng.integers(2, 13))
    edges = random_dag(rng, n, float(rng.uniform(0.15, 0.5)))
    weights = [float(x) for x in rng.integers(1, 9, size=n)]    # integer weights: ties do occur
    td = float(rng.integers(4, 20))
    got, cnt = B.ago_graph_cluster(weights, edges, td)
    assert got == C.cluster(weights, edges, td)
    assert cnt == len(set(got))
    assert C.is_acyclic_partition(got, edges)                   # Definition 1 / Theorem 1
    for s in set(got):                                          # merged subgraphs stay below the threshold
        members = [i for i in range(n) if got[i] == s]
        if len(members) > 1:
            assert sum(weights[i] for i in members) < td


def test_clustered_chain_feeds_subgraph_create():
    # The inverted-residual block as a 9-node chain with Eq. 1 weights: one subgraph under a large threshold, whose
    # nodes in topological order are exactly the op list ago_subgraph_create takes.
    wl = WL.get("mbv2_14")
    n_ops = len(wl.ops)
    weights = [B.ago_op_weight([14, 14, 32 + i], 1.0, 0.1) for i in range(n_ops)]
    edges = [(i, i + 1) for i in range(n_ops - 1)]
    got, cnt = B.ago_graph_cluster(weights, edges, 1e9)
    assert cnt == 1 and got == [0] * n_ops
    order = [i for i in range(n_ops) if got[i] == 0]
    sg = B.Subgraph([wl.ops[i] for i in order], wl.input_shapes, mode="fused")   # host-side create: plans the fused kernel
    assert sg.query(B.AGO_Q_FUSED_KERNEL) != 0
    sg.close()


def test_argument_errors():
    with pytest.raises(ValueError):
        B.ago_graph_cluster([1.0, 1.0], [(0, 1), (1, 0)], 5.0)      # cyclic input
    with pytest.raises(ValueError):
        B.ago_graph_cluster([1.0, 1.0], [(0, 2)], 5.0)              # edge names no node
    assert B.load().ago_graph_cluster(None, None, None) == B.AGO_ERR_INVALID_ARG
