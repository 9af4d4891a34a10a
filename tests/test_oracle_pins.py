"""Pins for the CPU oracle: closed forms, brute force through a second formulation,
library routines on special cases, and the paper's worked examples.  No GPU."""
import math
import os

import numpy as np
import pytest
import scipy.signal
import scipy.special

from oracle import oracle as orc
from paper_2201_05587_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def im2col_conv(x, w, bias, stride, pad):
    """Second, independent formulation: explicit padding, patch matrix, fp64 matmul."""
    x = x.astype(np.float64)
    w = w.astype(np.float64)
    n, c, h, wd = x.shape
    k, _, r, s = w.shape
    xp = np.zeros((n, c, h + 2 * pad[0], wd + 2 * pad[1]))
    xp[:, :, pad[0]:pad[0] + h, pad[1]:pad[1] + wd] = x
    p = (h + 2 * pad[0] - r) // stride[0] + 1
    q = (wd + 2 * pad[1] - s) // stride[1] + 1
    cols = np.zeros((n, c * r * s, p * q))
    for ci in range(c):
        for ri in range(r):
            for si in range(s):
                patch = xp[:, ci, ri:ri + stride[0] * p:stride[0], si:si + stride[1] * q:stride[1]]
                cols[:, (ci * r + ri) * s + si, :] = patch.reshape(n, -1)
    y = np.einsum("kj,njp->nkp", w.reshape(k, -1), cols).reshape(n, k, p, q)
    if bias is not None:
        y = y + bias.astype(np.float64)[None, :, None, None]
    return y


@pytest.mark.parametrize("stride", [(1, 1), (2, 2), (1, 2)])
@pytest.mark.parametrize("pad", [(0, 0), (1, 1), (2, 1)])
@pytest.mark.parametrize("rs", [(3, 3), (1, 1), (2, 3)])
def test_conv_brute_force_second_formulation(stride, pad, rs):
    x = inputs.uniform((2, 2, 5, 4), 11, 0)
    w = inputs.uniform((3, 2) + rs, 11, 1)
    b = inputs.uniform((3,), 11, 2)
    if 5 + 2 * pad[0] < rs[0] or 4 + 2 * pad[1] < rs[1]:
        pytest.skip("filter larger than padded input")
    y = orc.conv2d(x, w, b, stride=stride, pad=pad)
    ref = im2col_conv(x, w, b, stride, pad)
    assert y.shape == ref.shape
    np.testing.assert_allclose(y, ref.astype(np.float32), rtol=0, atol=1e-6)


def test_conv_is_cross_correlation_scipy():
    """One channel, one filter, no padding: the library's 'valid' correlation (no flip)."""
    x = inputs.uniform((1, 1, 9, 8), 12, 0)
    w = inputs.uniform((1, 1, 3, 3), 12, 1)
    y = orc.conv2d(x, w)
    ref = scipy.signal.correlate2d(x[0, 0].astype(np.float64), w[0, 0].astype(np.float64), mode="valid")
    np.testing.assert_allclose(y[0, 0], ref.astype(np.float32), atol=1e-6)
    flipped = scipy.signal.convolve2d(x[0, 0].astype(np.float64), w[0, 0].astype(np.float64), mode="valid")
    assert np.abs(y[0, 0] - flipped).max() > 1e-3


@pytest.mark.parametrize("c0,r0,s0", [(0, 0, 0), (1, 1, 1), (2, 2, 0), (1, 0, 2)])
def test_conv_delta_filter_is_shift(c0, r0, s0):
    """A filter with a single 1 at (c0,r0,s0) copies input channel c0 shifted by (r0-1, s0-1), zeros outside."""
    x = inputs.uniform((1, 3, 6, 7), 13, 0)
    w = np.zeros((2, 3, 3, 3), np.float32)
    w[1, c0, r0, s0] = 1.0
    y = orc.conv2d(x, w, pad=(1, 1))
    assert np.all(y[0, 0] == 0)
    exp = np.zeros((6, 7), np.float32)
    for p in range(6):
        for q in range(7):
            ih, iw = p + r0 - 1, q + s0 - 1
            if 0 <= ih < 6 and 0 <= iw < 7:
                exp[p, q] = x[0, c0, ih, iw]
    np.testing.assert_array_equal(y[0, 1], exp)


def test_conv_all_ones_filter_is_window_sum():
    x = inputs.uniform((1, 2, 8, 9), 14, 0)
    w = np.ones((1, 2, 3, 3), np.float32)
    y = orc.conv2d(x, w, pad=(1, 1))
    # summed-area table over the zero-padded channel sum
    cs = x.astype(np.float64).sum(axis=1)[0]
    padded = np.zeros((8 + 2, 9 + 2))
    padded[1:-1, 1:-1] = cs
    sat = np.zeros((11, 12))
    sat[1:, 1:] = padded.cumsum(0).cumsum(1)
    exp = sat[3:, 3:] - sat[:-3, 3:] - sat[3:, :-3] + sat[:-3, :-3]
    np.testing.assert_allclose(y[0, 0], exp.astype(np.float32), atol=1e-5)


def test_conv_1x1_equals_dense_on_reshaped_tensor():
    x = inputs.uniform((1, 5, 4, 3), 15, 0)
    w = inputs.uniform((6, 5, 1, 1), 15, 1)
    b = inputs.uniform((6,), 15, 2)
    y = orc.conv2d(x, w, b)
    pix = x[0].reshape(5, 12).T.copy()                 # [pixels, C]
    d = orc.dense(pix, w.reshape(6, 5), b)             # [pixels, K]
    np.testing.assert_array_equal(y[0].reshape(6, 12), d.T)


def test_conv_stride2_is_subsampled_stride1():
    x = inputs.uniform((1, 3, 9, 9), 16, 0)
    w = inputs.uniform((4, 3, 3, 3), 16, 1)
    y1 = orc.conv2d(x, w, pad=(1, 1))
    y2 = orc.conv2d(x, w, stride=(2, 2), pad=(1, 1))
    np.testing.assert_array_equal(y2, y1[:, :, ::2, ::2])


def test_conv_bias_only_and_activations():
    x = inputs.uniform((1, 2, 4, 4), 17, 0)
    w = np.zeros((3, 2, 3, 3), np.float32)
    b = np.array([-1.5, 2.0, 7.25], np.float32)
    y = orc.conv2d(x, w, b, pad=(1, 1), act=orc.ACT_RELU)
    assert np.all(y[0, 0] == 0) and np.all(y[0, 1] == 2.0) and np.all(y[0, 2] == 7.25)
    y6 = orc.conv2d(x, w, b, pad=(1, 1), act=orc.ACT_RELU6)
    assert np.all(y6[0, 0] == 0) and np.all(y6[0, 1] == 2.0) and np.all(y6[0, 2] == 6.0)
    yn = orc.conv2d(x, w, b, pad=(1, 1))
    assert np.all(yn[0, 0] == -1.5)


def test_conv_linearity_and_residual():
    x1 = inputs.uniform((1, 2, 5, 5), 18, 0)
    x2 = inputs.uniform((1, 2, 5, 5), 18, 1)
    w = inputs.uniform((3, 2, 3, 3), 18, 2)
    ya = orc.conv2d(x1, w, pad=(1, 1)).astype(np.float64)
    yb = orc.conv2d(x2, w, pad=(1, 1)).astype(np.float64)
    ys = orc.conv2d((x1 + 2 * x2), w, pad=(1, 1)).astype(np.float64)
    np.testing.assert_allclose(ys, ya + 2 * yb, atol=2e-5)
    res = inputs.uniform((1, 3, 5, 5), 18, 3)
    yr = orc.conv2d(x1, w, pad=(1, 1), residual=res, act=orc.ACT_RELU)
    np.testing.assert_allclose(yr, np.maximum(ya + res, 0).astype(np.float32), atol=1e-6)


def test_conv_residual_with_stride_and_asymmetric_padding():
    """The residual has the OUTPUT's shape and is added before the activation, also when stride > 1 and the two
    paddings differ (an index error between the strided output and the residual shows here, not at stride 1)."""
    x = inputs.uniform((2, 3, 9, 7), 24, 0)
    w = inputs.uniform((4, 3, 3, 2), 24, 1)
    b = inputs.uniform((4,), 24, 2)
    for stride, pad in (((2, 2), (1, 1)), ((2, 1), (0, 1)), ((1, 2), (2, 0))):
        pre = im2col_conv(x, w, b, stride, pad)
        res = inputs.uniform(pre.shape, 24, 3)
        y = orc.conv2d(x, w, b, stride=stride, pad=pad, residual=res, act=orc.ACT_RELU)
        np.testing.assert_allclose(y, np.maximum(pre + res, 0).astype(np.float32), rtol=0, atol=1e-6)


def window_products_dw(x, w, bias, stride, pad):
    """Depthwise convolution through a formulation that shares nothing with the loops of the oracle: explicit zero
    padding, then one strided view of the padded image per filter tap, multiplied by that tap and summed in fp64."""
    x = x.astype(np.float64)
    n, c, h, wd = x.shape
    r, s = w.shape[2], w.shape[3]
    xp = np.zeros((n, c, h + 2 * pad[0], wd + 2 * pad[1]))
    xp[:, :, pad[0]:pad[0] + h, pad[1]:pad[1] + wd] = x
    p = (h + 2 * pad[0] - r) // stride[0] + 1
    q = (wd + 2 * pad[1] - s) // stride[1] + 1
    y = np.zeros((n, c, p, q))
    for ri in range(r):
        for si in range(s):
            view = xp[:, :, ri:ri + stride[0] * (p - 1) + 1:stride[0], si:si + stride[1] * (q - 1) + 1:stride[1]]
            y += view * w[:, 0, ri, si].astype(np.float64)[None, :, None, None]
    if bias is not None:
        y += bias.astype(np.float64)[None, :, None, None]
    return y


@pytest.mark.parametrize("stride", [(1, 1), (2, 2), (1, 2), (2, 1)])
@pytest.mark.parametrize("pad", [(1, 1), (1, 0), (0, 2), (2, 2)])
@pytest.mark.parametrize("rs", [(3, 3), (5, 5), (3, 5)])
def test_depthwise_brute_force_and_block_diagonal_full_conv(stride, pad, rs):
    """Depthwise against (a) the tap-by-tap window products above and (b) the full convolution with block-diagonal
    weights, over asymmetric strides, paddings and filters: a swapped stride or padding axis, or a slip that only a
    5-wide filter shows, fails here."""
    c = 4
    x = inputs.uniform((2, c, 9, 8), 19, 0)
    w = inputs.uniform((c, 1) + rs, 19, 1)
    b = inputs.uniform((c,), 19, 2)
    if 9 + 2 * pad[0] < rs[0] or 8 + 2 * pad[1] < rs[1]:
        pytest.skip("filter larger than padded input")
    y = orc.dwconv2d(x, w, b, stride=stride, pad=pad, act=orc.ACT_RELU6)
    pre = window_products_dw(x, w, b, stride, pad)
    assert y.shape == pre.shape
    np.testing.assert_allclose(y, np.clip(pre, 0.0, 6.0).astype(np.float32), rtol=0, atol=1e-6)
    full = np.zeros((c, c) + rs, np.float32)
    for i in range(c):
        full[i, i] = w[i, 0]
    ref = orc.conv2d(x, full, b, stride=stride, pad=pad, act=orc.ACT_RELU6)
    np.testing.assert_array_equal(y, ref)


def test_depthwise_delta_and_ones():
    x = inputs.uniform((1, 3, 5, 5), 20, 0)
    w = np.zeros((3, 1, 3, 3), np.float32)
    w[:, 0, 1, 1] = 1.0
    np.testing.assert_array_equal(orc.dwconv2d(x, w, pad=(1, 1)), x)
    w[:] = 1.0
    y = orc.dwconv2d(x, w, pad=(0, 0))
    exp = sum(x[:, :, r:r + 3, s:s + 3].astype(np.float64) for r in range(3) for s in range(3))
    np.testing.assert_allclose(y, exp.astype(np.float32), atol=1e-6)


def test_matmul_algorithm1_against_numpy_and_closed_forms():
    a = inputs.uniform((1, 7, 5), 21, 0)
    b = inputs.uniform((1, 5, 6), 21, 1)
    c = orc.batch_matmul(a, b)
    ref = a[0].astype(np.float64) @ b[0].astype(np.float64)
    np.testing.assert_allclose(c[0], ref.astype(np.float32), atol=1e-6)
    # identity weight copies, ones give row sums
    x = inputs.uniform((4, 6), 21, 2)
    np.testing.assert_array_equal(orc.dense(x, np.eye(6, dtype=np.float32)), x)
    rs = orc.dense(x, np.ones((3, 6), np.float32))
    np.testing.assert_allclose(rs, np.repeat(x.astype(np.float64).sum(1, keepdims=True), 3, 1).astype(np.float32),
                               atol=1e-6)
    # a non-symmetric case separates a transposed operand from the right one
    w = inputs.uniform((3, 6), 21, 3)
    bias = inputs.uniform((3,), 21, 4)
    d = orc.dense(x, w, bias)
    np.testing.assert_allclose(d, (x.astype(np.float64) @ w.astype(np.float64).T + bias).astype(np.float32),
                               atol=1e-6)


def test_batch_matmul_nt_nn_consistency_and_batch1_dense():
    a = inputs.uniform((3, 4, 5), 22, 0)
    b = inputs.uniform((3, 6, 5), 22, 1)            # [B, M, K]
    nt = orc.batch_matmul(a, b, trans_b=True)
    nn = orc.batch_matmul(a, np.ascontiguousarray(b.transpose(0, 2, 1)), trans_b=False)
    np.testing.assert_array_equal(nt, nn)
    for i in range(3):
        np.testing.assert_array_equal(nt[i], orc.dense(a[i], b[i]))
    ident = np.broadcast_to(np.eye(5, dtype=np.float32), (3, 5, 5)).copy()
    np.testing.assert_array_equal(orc.batch_matmul(a, ident), a)


def test_softmax_pins():
    s = inputs.normal((3, 4, 17), 23, 0, std=3.0)
    p = orc.softmax(s, scale=0.125)
    np.testing.assert_allclose(p.astype(np.float64).sum(-1), 1.0, atol=1e-6)
    np.testing.assert_allclose(p, scipy.special.softmax(0.125 * s.astype(np.float64), axis=-1).astype(np.float32),
                               atol=1e-7)
    shifted = orc.softmax(s + np.float32(8.0), scale=0.125)
    np.testing.assert_allclose(shifted, p, atol=1e-6)
    u = orc.softmax(np.full((2, 8), 3.5, np.float32))
    np.testing.assert_array_equal(u, np.full((2, 8), 0.125, np.float32))
    # large magnitudes must not overflow
    big = orc.softmax(np.array([[1000.0, 1000.0, -1000.0]], np.float32))
    np.testing.assert_allclose(big, [[0.5, 0.5, 0.0]], atol=1e-7)


def test_activation_pins():
    x = np.array([[-3.0, -1.0, 0.0, 0.5, 1.0, 6.0, 7.5]], np.float32)
    eye = np.eye(7, dtype=np.float32)
    r6 = orc.dense(x, eye, act=orc.ACT_RELU6)
    np.testing.assert_array_equal(r6, [[0, 0, 0, 0.5, 1.0, 6.0, 6.0]])
    r = orc.dense(x, eye, act=orc.ACT_RELU)
    np.testing.assert_array_equal(r, [[0, 0, 0, 0.5, 1.0, 6.0, 7.5]])
    g = orc.dense(x, eye, act=orc.ACT_GELU_ERF).astype(np.float64)
    gm = orc.dense(-x, eye, act=orc.ACT_GELU_ERF).astype(np.float64)
    assert g[0, 2] == 0.0
    np.testing.assert_allclose(g - gm, x, atol=1e-6)             # GELU(x) - GELU(-x) = x
    assert abs(g[0, 4] - 0.8413447460685429) < 1e-7              # GELU(1) = Phi(1)
    assert abs(g[0, 4] - 0.5 * (1 + math.tanh(math.sqrt(2 / math.pi) * (1 + 0.044715)))) > 1e-5  # not the tanh form


def test_tf32_modes_are_diagnostics_close_to_exact():
    x = inputs.uniform((8, 64), 24, 0)
    w = inputs.uniform((16, 64), 24, 1)
    exact = orc.dense(x, w)
    for mode in (orc.MODE_TF32_TRUNC, orc.MODE_TF32_ROUND):
        e = orc.rel_l2(orc.dense(x, w, mode=mode), exact)
        assert 1e-6 < e < 2e-3
    # values already representable with 10 mantissa bits are unchanged by either mode
    xi = np.round(x * 64) / 64
    wi = np.round(w * 64) / 64
    np.testing.assert_array_equal(orc.dense(xi, wi, mode=orc.MODE_TF32_TRUNC), orc.dense(xi, wi))
    np.testing.assert_array_equal(orc.dense(xi, wi, mode=orc.MODE_TF32_ROUND), orc.dense(xi, wi))


def test_thread_count_does_not_change_results():
    x = inputs.uniform((1, 8, 12, 12), 25, 0)
    w = inputs.uniform((8, 8, 3, 3), 25, 1)
    y1 = orc.conv2d(x, w, pad=(1, 1), threads=1)
    yn, used = orc.conv2d(x, w, pad=(1, 1), threads=0, return_threads=True)
    assert used >= 1
    np.testing.assert_array_equal(y1, yn)


def test_split_rules_match_paper_examples():
    with open(os.path.join(GOLDEN, "split_validity.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            extent, form, factors, valid = line.split()
            extent, valid = int(extent), bool(int(valid))
            fs = [int(v) for v in factors.split(",")]
            if form == "fixed":
                assert orc.split_covers(extent, fs) == valid, line
            elif form == "reform":
                assert orc.split_reformulated_valid(extent, fs[0]) == valid, line
            else:
                assert orc.factor_fits(extent, fs[0]) == valid, line
    assert not orc.same_class(("conv2d", "bias", "relu"), ("dense", "add"))
    assert orc.same_class(("conv2d", "bias", "relu"), ("conv2d", "bias", "relu"))


def test_select_hand_tables():
    t = [5.0, 3.0, -1.0, 3.0,     # tie between 1 and 3 -> lowest index
         -1.0, -1.0, -1.0, -1.0,  # nothing valid
         2.0, -1.0, 1.5, 9.0]
    assert orc.select(t, 3, 4) == [1, -1, 2]
    assert orc.model_latency([2, 1, 3], t, [1, -1, 2], 4) == pytest.approx(2 * 3.0 + 3 * 1.5)


def _load_tables():
    """Tables 2 and 3 of the paper as stored under tests/golden/."""
    feats = {}
    with open(os.path.join(GOLDEN, "table2_model_features.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            mid, _name, cls, n, pct = line.split()
            feats.setdefault(mid, {})[cls] = (int(n), int(pct))
    choices = {}
    with open(os.path.join(GOLDEN, "table3_heuristic_choices.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            t, c1, c2, c3 = line.split()
            choices[t] = [c for c in (c1, c2, c3) if c != "-"]
    return feats, choices


def test_selection_heuristic_reproduces_the_papers_top3_choices():
    """Equation 1 evaluated on Table 2 must rank the candidate models as Table 3 lists them (all ten targets)."""
    feats, choices = _load_tables()
    assert len(feats) == 10 and len(choices) == 10
    for target, want in choices.items():
        cands = [m for m in feats if m != target]
        share = {c: pct / 100.0 for c, (_, pct) in feats[target].items()}
        counts = [{c: n for c, (n, _) in feats[m].items()} for m in cands]
        scores, order = orc.rank_pools(share, counts)
        got = [cands[i] for i in order[:len(want)]]
        assert got == want, (target, got, want, sorted(scores, reverse=True)[:4])
        if len(want) == 1:        # BERT / MobileBERT: every other model scores zero
            assert all(scores[i] == 0.0 for i in order[1:])
    # a dropped square or square root changes the ranking somewhere: GoogLeNet's second and third choice differ by 2e-4
    share = {c: pct / 100.0 for c, (_, pct) in feats["M7"].items()}
    s_vgg = sum(share.get(c, 0) ** 2 * math.sqrt(n) for c, (n, _) in feats["M3"].items())
    s_mnas = sum(share.get(c, 0) ** 2 * math.sqrt(n) for c, (n, _) in feats["M8"].items())
    assert 0 < s_vgg - s_mnas < 1e-3


def test_selection_heuristic_special_cases():
    # one class, one candidate kernel: score = P^2
    assert orc.rank_pools({"E": 0.5}, [{"E": 1}])[0] == [0.25]
    # four times the kernels doubles the score; a class the target lacks adds nothing
    s, order = orc.rank_pools({"E": 1.0}, [{"E": 4, "Z": 100}, {"E": 16}, {"Q": 9}])
    assert s == [2.0, 4.0, 0.0] and order == [1, 0, 2]
    # ties keep the lower index
    assert orc.rank_pools({"A": 0.3}, [{"A": 2}, {"A": 2}])[1] == [0, 1]


# ---- refining a transferred schedule: greedy one-parameter-at-a-time descent (Section 7, future work) ----
def test_ladder_steps_are_the_adjacent_rungs():
    lad = [1, 2, 4, 7, 8, 14]
    assert orc.ladder_steps(4, lad) == [2, 7]
    assert orc.ladder_steps(1, lad) == [2]
    assert orc.ladder_steps(14, lad) == [8]
    assert orc.ladder_steps(5, lad) == [4, 7]            # a value between two rungs
    assert orc.ladder_steps(100, lad) == [14] and orc.ladder_steps(0, lad) == [1]
    assert orc.ladder_steps(0, [0, 1]) == [1] and orc.ladder_steps(1, [0, 1]) == [0]


def test_raw_neighbours_change_exactly_one_parameter_by_one_rung():
    rec = {"block_x": 8, "block_y": 4, "vec_width": 2}
    nb = orc.raw_neighbours(rec, "row_simt")
    assert nb == [{"block_x": 4, "block_y": 4, "vec_width": 2}, {"block_x": 16, "block_y": 4, "vec_width": 2},
                  {"block_x": 8, "block_y": 2, "vec_width": 2}, {"block_x": 8, "block_y": 8, "vec_width": 2},
                  {"block_x": 8, "block_y": 4, "vec_width": 1}, {"block_x": 8, "block_y": 4, "vec_width": 4}]
    for fam in orc.LADDERS:
        start = {name: lad[len(lad) // 2] for name, lad in orc.LADDERS[fam]}
        for r in orc.raw_neighbours(start, fam):
            changed = [k for k in r if r[k] != start[k]]
            assert len(changed) == 1
            lad = dict(orc.LADDERS[fam])[changed[0]]
            assert abs(lad.index(r[changed[0]]) - lad.index(start[changed[0]])) == 1


def _row_space():
    lads = orc.LADDERS["row_simt"]
    names = [n for n, _ in lads]
    return names, [dict(zip(names, vals)) for vals in __import__("itertools").product(*[l for _, l in lads])]


def test_refine_reaches_the_exhaustive_minimum_of_a_separable_convex_cost():
    # cost = sum of per-parameter convex bowls: a one-parameter-at-a-time descent cannot get stuck, so it must end at
    # the minimum that exhaustive search over the whole space finds
    names, space = _row_space()
    target = {"block_x": 16, "block_y": 2, "vec_width": 4}
    cost = lambda d: 10.0 + sum((np.log2(d[k]) - np.log2(target[k])) ** 2 * (i + 1) for i, k in enumerate(names))
    key = lambda d: tuple(d[k] for k in names)
    unkey = lambda t: dict(zip(names, t))
    best_exh = min(space, key=cost)
    for start in ({"block_x": 1, "block_y": 16, "vec_width": 1}, {"block_x": 32, "block_y": 1, "vec_width": 2}, dict(target)):
        best, best_us, start_us, timed = orc.refine(key(start), lambda s: [key(r) for r in orc.raw_neighbours(unkey(s), "row_simt")],
                                                    lambda s: cost(unkey(s)), max_rounds=50)
        assert unkey(best) == best_exh == target
        assert best_us == pytest.approx(10.0) and start_us == pytest.approx(cost(start))
        assert timed <= len(space)                       # nothing is timed twice
    # from the optimum: one round, every neighbour timed once, no move
    _, _, _, timed = orc.refine(key(target), lambda s: [key(r) for r in orc.raw_neighbours(unkey(s), "row_simt")],
                                lambda s: cost(unkey(s)), max_rounds=50)
    assert timed == 1 + len(orc.raw_neighbours(target, "row_simt"))


def test_refine_round_limit_gain_threshold_invalid_and_ties():
    chain = {0: [1], 1: [2], 2: [3], 3: []}
    t = {0: 10.0, 1: 9.0, 2: 8.0, 3: 7.0}
    assert orc.refine(0, chain.__getitem__, t.__getitem__, max_rounds=2)[0] == 2           # two moves, no more
    assert orc.refine(0, chain.__getitem__, t.__getitem__, max_rounds=0) == (0, 10.0, 10.0, 1)
    t2 = {0: 10.0, 1: 8.5, 2: 8.0, 3: 1.0}
    assert orc.refine(0, chain.__getitem__, t2.__getitem__, max_rounds=9, min_gain=0.10)[0] == 1   # 15 % moves, the next 5.9 % does not
    assert orc.refine(0, chain.__getitem__, t.__getitem__, max_rounds=9, min_gain=0.10)[0] == 0    # a gain must EXCEED the threshold
    # a neighbour that cannot run (negative time) is never chosen, however "fast"; ties keep the earlier neighbour
    star = {0: [1, 2, 3], 1: [], 2: [], 3: []}
    assert orc.refine(0, star.__getitem__, {0: 5.0, 1: -1.0, 2: 4.0, 3: 4.0}.__getitem__, 3)[0] == 2
    with pytest.raises(ValueError):
        orc.refine(0, star.__getitem__, {0: -1.0, 1: 1.0, 2: 1.0, 3: 1.0}.__getitem__, 3)


def test_splitmix64_published_vector_and_subsample_is_a_shuffle_prefix():
    """The generator against the test vector published with its reference implementation (seed 1234567), and the
    subset against what a shuffle must satisfy: distinct indices in range, a prefix property (asking for more records
    extends the list, never reorders it), the full count is a permutation, another seed gives another order."""
    state, outs = 1234567, []
    for _ in range(5):
        state, v = orc.splitmix64(state)
        outs.append(v)
    assert outs == [6457827717110365317, 3203168211198807973, 9817491932198370423, 4593380528125082431, 16408922859458223821]
    for n in (1, 2, 7, 50, 111):
        full = orc.pool_subsample(n, n, 42)
        assert sorted(full) == list(range(n))
        for c in (0, 1, n // 3, n):
            assert orc.pool_subsample(n, c, 42) == full[:c]
    assert orc.pool_subsample(50, 50, 42) != orc.pool_subsample(50, 50, 43)
    # every index leads the list for some seed: no position is favoured out of existence
    assert {orc.pool_subsample(5, 1, s)[0] for s in range(200)} == set(range(5))
    with pytest.raises(ValueError):
        orc.pool_subsample(3, 4, 0)


def test_subsampled_evaluation_rule():
    row = [10.0, 12.0, 7.0, -1.0, 9.5, 4.0]          # default, then five pool records (one invalid)
    # the subset {1, 2} holds a record 30 % faster than the default: with a 20 % bar the search stops there
    assert orc.evaluate_subsampled(row, [1, 2], 20.0) == {0, 2, 3}
    # with a 40 % bar it does not, and every record is evaluated
    assert orc.evaluate_subsampled(row, [1, 2], 40.0) == set(range(6))
    # a subset without a valid record never ends the search
    assert orc.evaluate_subsampled(row, [2], 0.0) == set(range(6))
