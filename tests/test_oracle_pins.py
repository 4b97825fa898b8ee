"""Pins for the CPU oracle: every operator is checked against something other
than itself -- closed forms, invariants, brute force written a second way, and
torch's float64 CPU library routines. A dropped term, a flipped kernel, a
transposed operand or a wrong pad/stride index fails at least one of these."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import oracle as O

rng = np.random.default_rng(1234)
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def t64(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float64))


# ---- convolution: orientation, padding, stride (Section III-A loop nest) --------


def test_conv_centre_delta_reproduces_input():
    x = rng.standard_normal((2, 5, 7, 3))
    w = np.zeros((3, 3, 3, 3))
    for c in range(3):
        w[c, 1, 1, c] = 1.0
    assert np.array_equal(O.conv2d(x, w, 1, 1), x)


def test_conv_shifted_tap_is_cross_correlation_not_flipped():
    # tap (r=0, s=1) with pad 1: out[h,w] = in[h-1, w]; first row is zero padding.
    x = rng.standard_normal((1, 4, 5, 1))
    w = np.zeros((1, 3, 3, 1)); w[0, 0, 1, 0] = 1.0
    y = O.conv2d(x, w, 1, 1)
    assert np.array_equal(y[0, 0], np.zeros((5, 1)))
    assert np.array_equal(y[0, 1:], x[0, :-1])
    # tap (r=1, s=2): out[h,w] = in[h, w+1]; last column is zero padding.
    w = np.zeros((1, 3, 3, 1)); w[0, 1, 2, 0] = 1.0
    y = O.conv2d(x, w, 1, 1)
    assert np.array_equal(y[0, :, -1], np.zeros((4, 1)))
    assert np.array_equal(y[0, :, :-1], x[0, :, 1:])


def test_conv_stride2_centre_delta_subsamples():
    x = rng.standard_normal((1, 8, 6, 2))
    w = np.zeros((2, 3, 3, 2)); w[0, 1, 1, 0] = 1.0; w[1, 1, 1, 1] = 1.0
    y = O.conv2d(x, w, 2, 1)
    assert y.shape == (1, 4, 3, 2)
    assert np.array_equal(y, x[:, ::2, ::2, :])


def test_valid_mode_extent_matches_paper_relation():
    # H1 = H2 + (R2 - 1), W1 = W2 + (C2 - 1)  (Section III-B)
    with open(os.path.join(GOLDEN, "valid_extent.txt")) as f:
        rows = [tuple(int(v) for v in ln.split()) for ln in f if ln.strip() and not ln.startswith("#")]
    for H1, R2, H2 in rows:
        assert O.out_extent(H1, R2, 1, 0) == H2 == H1 - (R2 - 1)
    x = rng.standard_normal((1, 9, 11, 2)); w = rng.standard_normal((3, 3, 5, 2))
    assert O.conv2d(x, w, 1, 0).shape == (1, 7, 7, 3)


def test_conv_weight_layout_is_OHWI_against_triple_loop():
    x = rng.standard_normal((1, 4, 4, 3)); w = rng.standard_normal((2, 3, 2, 3))
    y = O.conv2d(x, w, 1, 0)
    ref = np.zeros((1, 2, 3, 2))
    for o in range(2):
        for h in range(2):
            for ww in range(3):
                for r in range(3):
                    for s in range(2):
                        for i in range(3):
                            ref[0, h, ww, o] += x[0, h + r, ww + s, i] * w[o, r, s, i]
    np.testing.assert_allclose(y, ref, rtol=0, atol=1e-13)


@pytest.mark.parametrize("stride,pad,R", [(1, 1, 3), (2, 1, 3), (1, 0, 1), (2, 2, 5), (3, 0, 2)])
def test_conv_matches_torch_float64(stride, pad, R):
    x = rng.standard_normal((2, 9, 10, 4)); w = rng.standard_normal((6, R, R, 4))
    y = O.conv2d(x, w, stride, pad)
    ref = torch.nn.functional.conv2d(t64(x).permute(0, 3, 1, 2), t64(w).permute(0, 3, 1, 2),
                                     stride=stride, padding=pad).permute(0, 2, 3, 1).numpy()
    np.testing.assert_allclose(y, ref, rtol=0, atol=1e-12)


# ---- pointwise conv == matmul (Section III-B, last paragraph) ---------------------


def test_pointwise_conv_equals_gemm_and_triple_loop():
    x = rng.standard_normal((2, 3, 4, 5)); w = rng.standard_normal((7, 1, 1, 5))
    y = O.conv2d(x, w, 1, 0)
    g = O.gemm(x.reshape(-1, 5), w.reshape(7, 5).T.copy()).reshape(2, 3, 4, 7)
    np.testing.assert_allclose(y, g, rtol=0, atol=1e-13)
    ref = np.zeros((24, 7)); xf = x.reshape(24, 5)
    for m in range(24):
        for n in range(7):
            for k in range(5):
                ref[m, n] += xf[m, k] * w[n, 0, 0, k]
    np.testing.assert_allclose(y.reshape(24, 7), ref, rtol=0, atol=1e-13)


def test_gemm_identity_linearity_and_orientation():
    a = rng.standard_normal((6, 4))
    assert np.array_equal(O.gemm(a, np.eye(4)), a)
    w = rng.standard_normal((4, 3))
    np.testing.assert_allclose(O.gemm(2.5 * a, w), 2.5 * O.gemm(a, w), rtol=1e-14)
    # w is [K][N]: a one-hot row k of the weight routes column k of a to output n.
    w1 = np.zeros((4, 3)); w1[2, 1] = 1.0
    y = O.gemm(a, w1)
    assert np.array_equal(y[:, 1], a[:, 2]) and not y[:, [0, 2]].any()
    np.testing.assert_allclose(O.gemm(a, w), (t64(a) @ t64(w)).numpy(), rtol=0, atol=1e-13)


# ---- depthwise -------------------------------------------------------------------


def test_depthwise_equals_block_diagonal_dense_conv():
    C = 4
    x = rng.standard_normal((2, 6, 5, C)); w = rng.standard_normal((3, 3, C))
    dense = np.zeros((C, 3, 3, C))
    for c in range(C):
        dense[c, :, :, c] = w[:, :, c]
    for stride in (1, 2):
        np.testing.assert_allclose(O.depthwise(x, w, stride, 1), O.conv2d(x, dense, stride, 1),
                                   rtol=0, atol=1e-13)


def test_depthwise_ones_counts_in_image_neighbours():
    with open(os.path.join(GOLDEN, "ones3x3_counts.txt")) as f:
        vals = {k: float(v) for k, v in (ln.split() for ln in f if ln.strip() and not ln.startswith("#"))}
    y = O.depthwise(np.ones((1, 5, 6, 2)), np.ones((3, 3, 2)), 1, 1)
    assert y[0, 2, 3, 0] == vals["interior"]
    assert y[0, 0, 3, 1] == vals["edge"] and y[0, 2, 0, 0] == vals["edge"]
    assert y[0, 0, 0, 0] == vals["corner"] and y[0, 4, 5, 1] == vals["corner"]


def test_depthwise_matches_torch_grouped_conv():
    C = 6
    x = rng.standard_normal((2, 7, 8, C)); w = rng.standard_normal((3, 3, C))
    for stride in (1, 2):
        ref = torch.nn.functional.conv2d(t64(x).permute(0, 3, 1, 2), t64(w).permute(2, 0, 1).unsqueeze(1),
                                         stride=stride, padding=1, groups=C).permute(0, 2, 3, 1).numpy()
        np.testing.assert_allclose(O.depthwise(x, w, stride, 1), ref, rtol=0, atol=1e-12)


# ---- simple operators ----------------------------------------------------------------


def test_bias_broadcasts_over_last_dim_only():
    x = np.zeros((2, 3, 4)); b = np.array([1.0, 2.0, 3.0, 4.0])
    y = O.bias_add(x, b)
    assert np.array_equal(y, np.broadcast_to(b, (2, 3, 4)))


def test_relu_relu6_saturate():
    x = np.array([-3.0, -0.0, 0.0, 0.5, 5.999, 6.0, 6.5, 100.0])
    assert np.array_equal(O.relu(x), np.array([0, 0, 0, 0.5, 5.999, 6.0, 6.5, 100.0]))
    assert np.array_equal(O.relu6(x), np.array([0, 0, 0, 0.5, 5.999, 6.0, 6.0, 6.0]))


def test_gelu_tanh_invariants_and_library():
    x = np.linspace(-8, 8, 1001)
    g = O.gelu_tanh(x)
    assert O.gelu_tanh(np.zeros(1))[0] == 0.0
    np.testing.assert_allclose(g - O.gelu_tanh(-x), x, rtol=0, atol=1e-14)      # g(x) - g(-x) = x
    big = np.array([6.0, 7.5, 20.0])
    np.testing.assert_allclose(O.gelu_tanh(big), big, rtol=0, atol=1e-9)          # g(x) -> x
    np.testing.assert_allclose(g, torch.nn.functional.gelu(t64(x), approximate="tanh").numpy(),
                               rtol=0, atol=1e-14)
    # the tanh form differs measurably from the erf form: a mix-up fails here
    erf_form = np.array([0.5 * v * (1 + math.erf(v / math.sqrt(2))) for v in (1.0, -1.5)])
    assert np.max(np.abs(O.gelu_tanh(np.array([1.0, -1.5])) - erf_form)) > 1e-4


def test_scale_and_add():
    x = rng.standard_normal(17); y = rng.standard_normal(17)
    assert np.array_equal(O.scale(x, 0.125), x * 0.125)
    assert np.array_equal(O.add(x, y), x + y)


# ---- softmax / attention ----------------------------------------------------------------


def test_softmax_rows_properties():
    s = rng.standard_normal((5, 9)) * 3
    p = O.softmax_rows(s)
    np.testing.assert_allclose(p.sum(-1), np.ones(5), rtol=0, atol=1e-14)
    np.testing.assert_allclose(O.softmax_rows(s + 7.25), p, rtol=0, atol=1e-14)    # shift invariance
    np.testing.assert_allclose(O.softmax_rows(np.full((2, 4), 3.0)), np.full((2, 4), 0.25), atol=1e-15)
    np.testing.assert_allclose(p, torch.softmax(t64(s), -1).numpy(), rtol=0, atol=1e-14)
    # rows are independent and the reduction runs over the LAST dimension
    two = np.array([[0.0, math.log(3.0)], [5.0, 5.0]])
    np.testing.assert_allclose(O.softmax_rows(two), [[0.25, 0.75], [0.5, 0.5]], atol=1e-15)
    assert np.isfinite(O.softmax_rows(np.array([[1000.0, 999.0]]))).all()           # max subtraction


def _attn(q, k, v, heads, hd):
    s = O.scale(O.batched_qkt(q, k, heads, hd), 1.0 / math.sqrt(hd))
    return O.batched_pv(O.softmax_rows(s), v, heads, hd)


def test_attention_equal_scores_give_column_mean_of_v():
    B, S, Hh, D = 1, 6, 2, 4
    q = np.zeros((B, S, Hh * D)); k = rng.standard_normal((B, S, Hh * D)); v = rng.standard_normal((B, S, Hh * D))
    o = _attn(q, k, v, Hh, D)
    np.testing.assert_allclose(o, np.broadcast_to(v.mean(1, keepdims=True), o.shape), atol=1e-14)


def test_attention_dominant_score_selects_that_v_row_per_head():
    B, S, Hh, D = 1, 5, 2, 4
    q = np.zeros((B, S, Hh * D)); k = np.zeros((B, S, Hh * D)); v = rng.standard_normal((B, S, Hh * D))
    # head 0: every query points at key 3; head 1: every query points at key 1 (score +100 after 1/sqrt(D))
    q[0, :, 0] = 1.0; k[0, 3, 0] = 200.0
    q[0, :, D] = 1.0; k[0, 1, D] = 200.0
    o = _attn(q, k, v, Hh, D)
    np.testing.assert_allclose(o[0, :, :D], np.broadcast_to(v[0, 3, :D], (S, D)), atol=1e-12)
    np.testing.assert_allclose(o[0, :, D:], np.broadcast_to(v[0, 1, D:], (S, D)), atol=1e-12)


def test_attention_each_query_selects_its_own_key():
    # query r points at key (r + 2) mod S only (score 50 after the scale, 0 elsewhere): a permutation of the rows of V --
    # a transposed score matrix or a softmax over the wrong axis gives the inverse permutation or a blend
    B, S, Hh, D = 1, 8, 1, 8
    q = np.zeros((B, S, D)); k = np.zeros((B, S, D)); v = rng.standard_normal((B, S, D))
    for r in range(S):
        q[0, r, (r + 2) % S] = 10.0
        k[0, r, r] = 5.0 * np.sqrt(D)
    o = _attn(q, k, v, Hh, D)
    np.testing.assert_allclose(o[0], v[0, (np.arange(S) + 2) % S], atol=1e-12)


def test_attention_matches_torch_float64_per_head():
    B, S, Hh, D = 2, 7, 3, 4
    q, k, v = (rng.standard_normal((B, S, Hh * D)) for _ in range(3))
    o = _attn(q, k, v, Hh, D)
    tq, tk, tv = (t64(a).reshape(B, S, Hh, D).permute(0, 2, 1, 3) for a in (q, k, v))
    ref = (torch.softmax(tq @ tk.transpose(-1, -2) / math.sqrt(D), -1) @ tv).permute(0, 2, 1, 3).reshape(B, S, Hh * D)
    np.testing.assert_allclose(o, ref.numpy(), rtol=0, atol=1e-13)
    # q and k are not interchangeable: scores[b,h,i,j] = q_i . k_j
    s = O.batched_qkt(q, k, Hh, D)
    np.testing.assert_allclose(s[1, 2, 3, 5], q[1, 3, 2 * D:3 * D] @ k[1, 5, 2 * D:3 * D], atol=1e-14)


# ---- whole chains ---------------------------------------------------------------------------


def test_padding_applies_to_the_intermediate_not_the_input():
    # conv1 = centre delta with a large positive bias, ReLU, then an all-ones 3x3 with pad 1:
    # every output must count only the in-image neighbours of the post-activation tensor
    # (zero padding of conv2's own input), never ReLU(bias) in the halo.
    x = np.zeros((1, 4, 4, 1))
    w1 = np.zeros((1, 3, 3, 1)); w1[0, 1, 1, 0] = 1.0
    ops = [("conv2d", dict(O=1, R=3, S=3, stride=1, pad=1, groups=1)), ("bias_add", {}), ("relu", {}),
           ("conv2d", dict(O=1, R=3, S=3, stride=1, pad=1, groups=1))]
    y = O.run_chain(ops, [x], [w1, np.array([5.0]), np.ones((1, 3, 3, 1))])
    assert y[0, 0, 0, 0] == 20.0 and y[0, 0, 1, 0] == 30.0 and y[0, 1, 1, 0] == 45.0


def _im2col_conv(x, w, stride, pad):
    """Second, independently written path: explicit padding + im2col + matmul."""
    N, H, W, I = x.shape
    O_, R, S, _ = w.shape
    xp = np.zeros((N, H + 2 * pad, W + 2 * pad, I)); xp[:, pad:pad + H, pad:pad + W] = x
    Ho = (H + 2 * pad - R) // stride + 1; Wo = (W + 2 * pad - S) // stride + 1
    cols = np.zeros((N, Ho, Wo, R * S * I))
    for ho in range(Ho):
        for wo in range(Wo):
            cols[:, ho, wo] = xp[:, ho * stride:ho * stride + R, wo * stride:wo * stride + S].reshape(N, -1)
    return cols @ w.reshape(O_, -1).T


def test_mbv2_chain_against_second_path_and_torch():
    from paper_2212_01005_b200 import workloads as WL
    for stride, residual, cin, cout in ((1, True, 8, 8), (2, False, 8, 16)):
        wl = WL.mbv2_block("t", [7, stride], 2, 6, cin, 24, cout, stride, residual)
        d = WL.generate(wl)
        x = d["inputs"][0].astype(np.float64)
        w1, b1, wd, bd, w3, b3 = (a.astype(np.float64) for a in d["weights"])
        y = O.run_chain(wl.ops, d["inputs"], d["weights"])
        e = np.clip(_im2col_conv(x, w1, 1, 0) + b1, 0, 6)
        dense = np.zeros((24, 3, 3, 24))
        for c in range(24):
            dense[c, :, :, c] = wd[:, :, c]
        m = np.clip(_im2col_conv(e, dense, stride, 1) + bd, 0, 6)
        ref = _im2col_conv(m, w3, 1, 0) + b3
        if residual:
            ref = ref + x
        assert y.shape == wl.output_shape
        np.testing.assert_allclose(y, ref, rtol=0, atol=1e-12)


@pytest.mark.parametrize("stride,residual", [(1, True), (2, False)])
def test_mbv2_chain_with_zero_expand_weights_has_a_closed_form(stride, residual):
    # With zero expand weights the expanded tensor is relu6(b1) inside the image and 0 in the padding ring of the
    # depthwise convolution: its output depends on the position only through the taps inside the image. This pins the
    # order "bias and ReLU6 first, padding afterwards" and the stride / padding geometry of the chain.
    from paper_2212_01005_b200 import workloads as WL
    wl = WL.mbv2_block("pin", [77, stride], 2, 9 + stride, 8, 32, 8 if residual else 16, stride, residual)
    data = WL.generate(wl)
    w1, b1, wd, bd, w3, b3 = (a.astype(np.float64) for a in data["weights"])
    data["weights"][0] = np.zeros_like(data["weights"][0])
    x = data["inputs"][0].astype(np.float64)
    N, H, W, _ = x.shape
    Ho, Wo = wl.output_shape[1], wl.output_shape[2]
    e = np.clip(b1, 0.0, 6.0)
    ho, wo = np.arange(Ho) * stride, np.arange(Wo) * stride
    acc = np.zeros((Ho, Wo, e.size))
    for r in range(3):
        for c in range(3):
            inside = ((ho + r - 1 >= 0) & (ho + r - 1 < H))[:, None] & ((wo + c - 1 >= 0) & (wo + c - 1 < W))[None, :]
            acc += inside[:, :, None] * (wd[r, c] * e)[None, None, :]
    out = np.clip(acc + bd, 0.0, 6.0) @ w3.reshape(w3.shape[0], -1).T + b3
    ref = np.broadcast_to(out, (N,) + out.shape).copy()
    if residual:
        ref += x
    got = O.run_chain(wl.ops, data["inputs"], data["weights"])
    np.testing.assert_allclose(got, ref, atol=1e-12)


def test_ffn_chain_against_torch():
    from paper_2212_01005_b200 import workloads as WL
    wl = WL.ffn("t", [9], 10, 16, 40, 1)
    d = WL.generate(wl)
    y = O.run_chain(wl.ops, d["inputs"], d["weights"])
    x, w1, b1, w2, b2 = (t64(a) for a in (d["inputs"][0], *d["weights"]))
    ref = torch.nn.functional.gelu(x @ w1 + b1, approximate="tanh") @ w2 + b2
    np.testing.assert_allclose(y, ref.numpy(), rtol=0, atol=1e-12)


def test_resnet_chain_against_torch():
    from paper_2212_01005_b200 import workloads as WL
    wl = WL.resnet_block("t", [11], 2, 7, 8)
    d = WL.generate(wl)
    y = O.run_chain(wl.ops, d["inputs"], d["weights"])
    x = t64(d["inputs"][0]).permute(0, 3, 1, 2)
    w1, b1, w2, b2 = (t64(a) for a in d["weights"])
    F = torch.nn.functional
    h = F.relu(F.conv2d(x, w1.permute(0, 3, 1, 2), b1, padding=1))
    ref = F.relu(F.conv2d(h, w2.permute(0, 3, 1, 2), b2, padding=1) + x).permute(0, 2, 3, 1)
    np.testing.assert_allclose(y, ref.numpy(), rtol=0, atol=1e-12)


def test_attention_chain_against_torch():
    from paper_2212_01005_b200 import workloads as WL
    wl = WL.attention("t", [13], 2, 9, 2, 8)
    d = WL.generate(wl)
    y = O.run_chain(wl.ops, d["inputs"], d["weights"])
    q, k, v = (t64(a).reshape(2, 9, 2, 8).permute(0, 2, 1, 3) for a in d["inputs"])
    ref = (torch.softmax(q @ k.transpose(-1, -2) / math.sqrt(8), -1) @ v).permute(0, 2, 1, 3).reshape(2, 9, 16)
    np.testing.assert_allclose(y, ref.numpy(), rtol=0, atol=1e-13)


# ---- layout operators and the chain around them (Section VI-B) ---------------------


def test_transpose_matches_hand_written_example_and_is_an_involution():
    x = np.arange(12, dtype=np.float64).reshape(2, 3, 2)
    want = np.loadtxt(os.path.join(GOLDEN, "transpose_2x3x2.txt")).reshape(3, 2, 2)
    got = O.transpose(x, 0, 1)
    assert got.shape == (3, 2, 2) and np.array_equal(got, want)
    y = rng.standard_normal((2, 3, 4, 5))
    assert np.array_equal(O.transpose(O.transpose(y, 1, 2), 1, 2), y)
    assert O.transpose(y, 1, 2)[1, 3, 2, 4] == y[1, 2, 3, 4]
    assert O.transpose(y, 0, 2)[3, 1, 0, 2] == y[0, 1, 3, 2]


def test_reshape_keeps_row_major_order():
    x = rng.standard_normal((4, 6, 5))
    r = O.reshape(x, (2, 2, 6, 5))
    assert r[1, 0, 3, 2] == x[2, 3, 2] and r[0, 1, 5, 4] == x[1, 5, 4]
    assert np.array_equal(O.reshape(r, (24, 5)).ravel(), x.ravel())
    with pytest.raises(ValueError):
        O.reshape(x, (4, 6, 4))


def test_unfold_chain_against_element_by_element_definition():
    # matmul, reshape, add, reshape, transpose, reshape, matmul, reshape: rows are (image, pixel, patch) before the
    # transpose and (image, patch, pixel) after it; written out with explicit indices, no reshape or transpose
    B, P, N, d, d2 = 2, 3, 4, 5, 6
    M = B * P * N
    x = rng.standard_normal((M, d)); r = rng.standard_normal((B * P, N, d))
    w1 = rng.standard_normal((d, d)); w2 = rng.standard_normal((d, d2))
    ops = [("gemm", dict(N=d)), ("reshape", dict(shape=(B * P, N, d))), ("add_input", dict(input=1)),
           ("reshape", dict(shape=(B, P, N, d))), ("transpose", dict(a=1, b=2)), ("reshape", dict(shape=(M, d))),
           ("gemm", dict(N=d2)), ("reshape", dict(shape=(B, N, P, d2)))]
    got = O.run_chain(ops, [x, r], [w1, w2])
    assert got.shape == (B, N, P, d2)
    for b in range(B):
        for p in range(P):
            for n in range(N):
                row = (b * P + p) * N + n
                mid = [sum(x[row, k] * w1[k, j] for k in range(d)) + r[b * P + p, n, j] for j in range(d)]
                for o in range(d2):
                    want = sum(mid[j] * w2[j, o] for j in range(d))
                    assert abs(got[b, n, p, o] - want) <= 1e-12 * max(1.0, abs(want))


def test_run_chain_rejects_unconsumed_weights():
    with pytest.raises(ValueError):
        O.run_chain([("relu", {})], [np.zeros(3)], [np.zeros(3)])
