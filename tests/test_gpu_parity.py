"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same seeded inputs."""
import ctypes
import itertools

import numpy as np
import pytest

from oracle import oracle as orc
from paper_2201_05587_b200 import binding as B
from paper_2201_05587_b200 import workloads as W
import util

pytestmark = pytest.mark.gpu

INVARIANCE_TOL = 1e-5   # between two valid records on the same precision path


def tc(**kw):
    return B.make_record(B.TT_FAMILY_GEMM_TC, **kw)


GUARD_FLOATS = 16384          # 64 KB of a fixed pattern on either side of every output tensor
GUARD_VALUE = -7.5e37
ELEM_TF32 = 1e-4              # max |y - truncation-mode oracle| / max |oracle|: fp32 accumulation of up to 4608 exact products
ELEM_FP32 = 1e-5              # the same for the fp32 SIMT families against the exact oracle


def guarded_output(spec, device="cuda"):
    """An output tensor that sits between two guard bands: returns (y view, whole buffer)."""
    import torch
    shape = W.tensor_shapes(spec)[4]
    n = int(np.prod(shape))
    buf = torch.full((n + 2 * GUARD_FLOATS,), GUARD_VALUE, dtype=torch.float32, device=device)
    y = buf[GUARD_FLOATS:GUARD_FLOATS + n].view(shape)
    y.fill_(float("nan"))
    return y, buf


def guards_intact(buf):
    return bool((buf[:GUARD_FLOATS] == GUARD_VALUE).all()) and bool((buf[-GUARD_FLOATS:] == GUARD_VALUE).all())


def run_spec(spec, rec, arrays, ref=None, tol=None, mode=B.TT_MODE_LEGALISE, ref_elem=None):
    """Run `spec` under `rec` through the C ABI.  ref: exact oracle (whole-tensor rel-L2, the pass/fail of record).
    ref_elem: the oracle every single output is bounded against -- the truncation-mode oracle for the TF32 families
    (the tensor core reads its operands truncated to TF32), the exact oracle for the fp32 SIMT families -- so that
    one wrong output in a large tensor cannot hide inside the L2 norm.  The output sits between guard bands."""
    wl = spec.workload()
    info = wl.apply(rec, mode=mode)
    if info.legal.precision == 1 and ref is not None:
        ref_elem = ref if ref_elem is not None else None      # compensated products: bounded against the exact oracle
    t, _ = W.device_tensors(spec, arrays)
    t["y"], buf = guarded_output(spec)
    tt = B.tensors(t["x"], t["w"], t["bias"], t["residual"], t["y"])
    wl.run(tt)
    assert wl.status() == B.TT_OK
    y = t["y"].cpu().numpy()
    wl.close()
    assert guards_intact(buf), f"{spec.name} {rec.short()} wrote outside its output tensor"
    assert not np.isnan(y).any(), "kernel left outputs unwritten"
    if ref is not None:
        err = util.rel_l2(y, ref)
        assert err <= (tol or util.tolerance(spec.op)), f"{spec.name} {rec.short()} rel-L2 {err:.3e}"
    if ref_elem is not None:
        bound = (ELEM_FP32 if spec.op in (B.TT_OP_DWCONV2D, B.TT_OP_SOFTMAX) else ELEM_TF32) * max(float(np.abs(ref_elem).max()), 1e-30)
        worst = float(np.abs(y.astype(np.float64) - ref_elem.astype(np.float64)).max())
        assert worst <= bound, f"{spec.name} {rec.short()} max element error {worst:.3e} > {bound:.3e}"
    return y


def elem_ref(spec, arrays, ref):
    """The oracle against which single outputs are bounded (see run_spec)."""
    if spec.op in (B.TT_OP_DWCONV2D, B.TT_OP_SOFTMAX):
        return ref
    return util.oracle_ref(spec, arrays, mode=orc.MODE_TF32_TRUNC)


GEMM_RECORDS = [
    tc(tile_n=128, tile_k=32, stages=4, mma_m_axis=1),
    tc(tile_n=64, tile_k=16, stages=3, mma_m_axis=1),
    tc(tile_n=16, tile_k=8, stages=2, mma_m_axis=1),
    tc(tile_n=256, tile_k=64, stages=2, mma_m_axis=1),
    tc(tile_n=48, tile_k=32, stages=1, raster=1, mma_m_axis=1),
    tc(tile_n=96, tile_k=32, stages=6, split_k=3, mma_m_axis=1),
    tc(tile_n=128, tile_k=64, stages=3, split_k=2, mma_m_axis=2),
    tc(tile_n=32, tile_k=128, stages=2, split_k=1, raster=1, mma_m_axis=2),
    tc(tile_n=192, tile_k=16, stages=4, split_k=5, mma_m_axis=2),
    # convolutions: the input rows are staged for 1, 2 or 3 reduction tiles at a time (double-buffered chunks)
    tc(tile_n=64, tile_k=16, stages=3, slab_tiles=1, mma_m_axis=1),
    tc(tile_n=128, tile_k=32, stages=2, slab_tiles=2, mma_m_axis=2),
    tc(tile_n=32, tile_k=8, stages=4, split_k=2, slab_tiles=3, mma_m_axis=1),
    # more than 8 splits: partial tiles through the global workspace (2..8 splits reduce inside a thread-block cluster)
    tc(tile_n=64, tile_k=16, stages=2, split_k=12, mma_m_axis=1),
    # tap-major reduction order (stride-1 convolutions with 16-byte image rows; elsewhere legalised to the stored order)
    tc(tile_n=128, tile_k=32, stages=3, k_order=1, mma_m_axis=1),
    tc(tile_n=256, tile_k=64, stages=2, k_order=1, split_k=2, mma_m_axis=2),
    tc(tile_n=48, tile_k=32, stages=1, k_order=1, raster=1, mma_m_axis=1),
    tc(tile_n=64, tile_k=96, stages=2, k_order=1, mma_m_axis=1),            # three taps per pipeline stage where 3 divides r*s
    # several accumulators in tensor memory, reduction steps dealt round-robin, summed on read-out
    tc(tile_n=32, tile_k=32, stages=4, acc_split=4, mma_m_axis=1),
    tc(tile_n=48, tile_k=16, stages=3, acc_split=8, split_k=2, mma_m_axis=2),
    tc(tile_n=256, tile_k=64, stages=2, acc_split=2, mma_m_axis=1),
    # the persistent form (tile loop, two alternating accumulators; operands by TMA, row-contiguous ones transposed in
    # shared memory), alone and as CTA pairs; the register-capped two-CTAs-per-SM build of the one-tile form.  Kernels
    # that have no such form legalise these records back
    tc(tile_n=64, tile_k=32, stages=4, persistent=1, mma_m_axis=1),
    tc(tile_n=16, tile_k=16, stages=3, persistent=1, raster=1, mma_m_axis=2),
    tc(tile_n=128, tile_k=64, stages=2, persistent=1, mma_m_axis=2),
    tc(tile_n=96, tile_k=8, stages=8, persistent=1, mma_m_axis=0),
    tc(tile_n=64, tile_k=32, stages=3, persistent=1, cta_group=2, mma_m_axis=1),
    tc(tile_n=256, tile_k=32, stages=2, persistent=1, cta_group=2, mma_m_axis=2),
    tc(tile_n=32, tile_k=128, stages=2, persistent=1, cta_group=2, raster=1, mma_m_axis=1),
    tc(tile_n=128, tile_k=32, stages=3, k_order=1, persistent=1, mma_m_axis=1),          # tap-major in the persistent form
    tc(tile_n=64, tile_k=96, stages=2, k_order=1, persistent=1, raster=1, mma_m_axis=1),
    tc(tile_n=64, tile_k=32, stages=2, ctas_per_sm=2, mma_m_axis=1),
    tc(tile_n=128, tile_k=16, stages=3, ctas_per_sm=1, split_k=2, mma_m_axis=2),
    # error-compensated products (dense, batch_matmul NT; legalised away elsewhere)
    tc(tile_n=64, tile_k=32, stages=2, precision=1, mma_m_axis=1),
    tc(tile_n=128, tile_k=64, stages=3, precision=1, split_k=3, mma_m_axis=2),
]


def check_all_records(spec, seed, records=GEMM_RECORDS):
    a = W.make_inputs(spec, seed)
    ref = util.oracle_ref(spec, a)
    # a record whose tiles (for a convolution: plus the staged input rows) exceed shared memory on this shape is an
    # invalid pair, as in the evaluator; everything that applies must be right, and most records must apply
    probe = spec.workload()
    valid = [r for r in records if probe.check(r)[0] == B.TT_OK]
    assert all(probe.check(r)[0] in (B.TT_OK, B.TT_ERR_RESOURCE) for r in records)
    assert probe.check(probe.default_schedule())[0] == B.TT_OK
    compensated = [probe.check(r)[1].legal.precision == 1 for r in valid]      # (kept only where the kernel has that form)
    probe.close()
    assert len(valid) >= len(records) - 6
    re = elem_ref(spec, a, ref)
    outs = [run_spec(spec, r, a, ref, ref_elem=re) for r in valid]
    # a schedule changes speed, never semantics: every valid record gives the same output up to the order of the
    # fp32 additions (tile_k and split_k regroup them): sqrt(K) * 2^-24 is about 4e-6 at the largest K here.  Records
    # with error-compensated products are another precision path: compared among themselves
    for group in (False, True):
        ys = [y for y, c in zip(outs, compensated) if c == group]
        for y in ys[1:]:
            assert util.rel_l2(y, ys[0]) <= INVARIANCE_TOL
    return outs


@pytest.mark.parametrize("spec", [
    W._dense(128, 768, 768, name="bert_dense"),
    W._dense(200, 300, 100, act=B.TT_ACT_RELU, name="ragged_dense"),        # ragged M, N, K tails; K % 8 != 0
    W._dense(129, 147, 257, act=B.TT_ACT_GELU_ERF, name="odd_dense_gatherK"),   # K % 4 != 0: gathered operands
    W._dense(1, 512, 1000, name="head_m1"),
    W._dense(1, 1, 1, name="one_by_one"),
    W._dense(3, 5, 7, name="tiny"),
], ids=lambda s: s.name)
def test_dense_parity_all_records(spec):
    check_all_records(spec, seed=31)


@pytest.mark.parametrize("spec", [
    W.single_conv()[0],
    W._conv(3, 32, 64, 7, 2, 3, name="stem_like_7x7s2"),                    # reduction 147: gathered filters
    W._conv(24, 15, 40, 3, 2, 1, name="conv3x3s2_odd"),
    W._conv(32, 14, 64, 1, 1, 0, act=B.TT_ACT_RELU6, name="conv1x1_relu6"),
    W._conv(64, 14, 128, 1, 2, 0, act=B.TT_ACT_NONE, name="downsample_1x1s2"),
    W._conv(20, 7, 24, 3, 1, 1, name="conv3x3_7x7"),
    W.Spec(B.TT_OP_CONV2D, B.conv2d_shapes(2, 8, 9, 11, 12, 3, 3, 1, 1, True, B.TT_ACT_RELU, True), 1, "batch2_residual", "uniform"),
    W.Spec(B.TT_OP_CONV2D, B.make_shapes(n=1, c=6, h=10, w=12, k=9, r=3, s=2, stride_h=2, stride_w=1, pad_h=0, pad_w=1,
                                         has_bias=0, act=B.TT_ACT_NONE), 1, "asym_nobias", "uniform"),
    W._conv(20, 12, 40, 3, 1, 1, name="conv3x3_12x12_tap"),                 # rows of 48 bytes: the tap-major path applies
    W._conv(72, 16, 136, 3, 1, 1, act=B.TT_ACT_NONE, name="conv3x3_72ch_tap"),   # 3 channel blocks (the last one partial), 2 filter tiles
    W.Spec(B.TT_OP_CONV2D, B.conv2d_shapes(2, 33, 8, 20, 10, 5, 3, 1, 2, True, B.TT_ACT_RELU6), 1, "conv5x3_batch2_tap", "uniform"),
    W._conv(20, 10, 40, 1, 1, 0, name="conv1x1_100px_20ch"),
    W._conv(136, 12, 200, 1, 1, 0, act=B.TT_ACT_NONE, name="conv1x1_136ch"),
    # pointwise layers whose pixels are re-viewed as rows that tile the CTA exactly: 400 = 16 x 25, 784 = 16 x 49,
    # 3136 = 64 x 49 (batch 3, a partial last tile, a residual), and one whose pixel count has no such divisor
    W.Spec(B.TT_OP_CONV2D, B.conv2d_shapes(3, 40, 20, 20, 24, 1, 1, 1, 0, True, B.TT_ACT_RELU, True), 1, "conv1x1_400px_batch3_residual", "uniform"),
    W._conv(64, 28, 80, 1, 1, 0, act=B.TT_ACT_RELU6, name="conv1x1_784px"),
    W.Spec(B.TT_OP_CONV2D, B.conv2d_shapes(2, 24, 56, 56, 40, 1, 1, 1, 0, True, B.TT_ACT_NONE), 1, "conv1x1_3136px_batch2", "uniform"),
    W._conv(48, 18, 32, 1, 1, 0, name="conv1x1_324px_no_row_view"),
    W._conv(96, 9, 48, 3, 1, 1, name="conv3x3_96ch_chunks"),                # 864 reduction indices: many slab chunks
    W._conv(40, 12, 24, 5, 1, 2, act=B.TT_ACT_RELU6, name="conv5x5_pad2"),
    W._conv(32, 17, 16, 1, 3, 0, name="conv1x1s3"),                         # stride beyond the filter: rows are skipped
    W.Spec(B.TT_OP_CONV2D, B.make_shapes(n=2, c=5, h=9, w=13, k=7, r=2, s=4, stride_h=3, stride_w=2, pad_h=1, pad_w=3,
                                         has_bias=1, act=B.TT_ACT_RELU), 1, "asym_2x4_s3x2_p1x3", "uniform"),
], ids=lambda s: s.name)
def test_conv_parity_all_records(spec):
    check_all_records(spec, seed=32)


@pytest.mark.parametrize("spec", [
    W.Spec(B.TT_OP_BATCH_MATMUL, B.bmm_shapes(12, 128, 128, 64, True), 1, "qk_nt", "bert"),
    W.Spec(B.TT_OP_BATCH_MATMUL, B.bmm_shapes(12, 128, 64, 128, False), 1, "pv_nn", "bert"),
    W.Spec(B.TT_OP_BATCH_MATMUL, B.bmm_shapes(3, 50, 70, 36, False), 1, "ragged_nn", "bert"),
    W.Spec(B.TT_OP_BATCH_MATMUL, B.bmm_shapes(2, 45, 76, 52, False), 1, "ragged_nn_76", "bert"),
    W.Spec(B.TT_OP_BATCH_MATMUL, B.bmm_shapes(2, 33, 17, 10, True), 1, "ragged_nt_k10", "bert"),
], ids=lambda s: s.name)
def test_batch_matmul_parity_all_records(spec):
    check_all_records(spec, seed=33)


def test_config1_every_pool_record_and_selection():
    spec = W.single_conv()[0]
    a = W.make_inputs(spec, 1)
    ref = util.oracle_ref(spec, a)
    pool = W.single_conv_pool()
    outs = [run_spec(spec, r, a, ref) for r in pool]
    for y in outs[1:]:
        assert util.rel_l2(y, outs[0]) <= INVARIANCE_TOL
    wl = spec.workload()
    t, tt = W.device_tensors(spec, a)
    res = B.transfer_tune([wl], [tt], pool)
    assert res["pairs_timed"] == 5 and res["pairs_invalid"] == 0
    times = res["times_us"][0]
    assert all(v > 0 for v in times)
    # selection is the oracle's argmin on the measured table
    assert res["chosen"] == orc.select(times, 1, 5) == B.select(times, 1, 5)
    assert res["best_us"][0] == pytest.approx(min(times))
    # the chosen record is left applied: running now reproduces the oracle
    t["y"].zero_()
    wl.run(tt)
    assert wl.status() == B.TT_OK
    assert util.rel_l2(t["y"].cpu().numpy(), ref) <= util.TOL_TF32


def test_evaluator_records_invalid_pairs_and_falls_back_to_default():
    conv = W._conv(16, 12, 24, 3, 1, 1)
    dw = W._dw(16, 12, 1)
    a1, a2 = W.make_inputs(conv, 7), W.make_inputs(dw, 7, 1)
    w1, w2 = conv.workload(), dw.workload()
    t1, tt1 = W.device_tensors(conv, a1)
    t2, tt2 = W.device_tensors(dw, a2)
    fat = tc(tile_n=256, tile_k=128, stages=8, mma_m_axis=1)           # legal fields, too much shared memory... on big shapes
    nonsense = tc(tile_n=64, tile_k=32, stages=0)
    pool = [tc(tile_n=32, tile_k=16, stages=2), nonsense, B.make_record(B.TT_FAMILY_ROW_SIMT)]
    res = B.transfer_tune([w1, w2], [tt1, tt2], pool)
    st = res["status"]
    assert st[0][0] == B.TT_OK and st[0][1] == B.TT_OK
    assert st[0][2] == B.TT_ERR_INVALID_SCHEDULE and st[0][3] == B.TT_ERR_CLASS_MISMATCH
    assert res["times_us"][0][2] == -1.0 and res["times_us"][0][3] == -1.0
    # the depthwise kernel has no compatible record in this pool: it keeps its default schedule
    assert st[1][1] == st[1][2] == st[1][3] == B.TT_ERR_CLASS_MISMATCH
    assert res["chosen"][1] == 0 and res["best_us"][1] > 0
    assert res["pairs_invalid"] == 5 and res["pairs_timed"] == 3
    w2.run(tt2)
    assert util.rel_l2(t2["y"].cpu().numpy(), util.oracle_ref(dw, a2)) <= util.TOL_FP32
    del fat


@pytest.mark.parametrize("spec", [s for s in W.mobilenet_v2() if s.op == B.TT_OP_DWCONV2D][::3] + [
    W._dw(5, 9, 2), W._dw(40, 28, 1, r=5), W._dw(1, 1, 1),
    W.Spec(B.TT_OP_DWCONV2D, B.make_shapes(n=3, c=7, h=13, w=10, r=3, s=3, stride_h=1, stride_w=2, pad_h=1, pad_w=0,
                                           has_bias=0, act=B.TT_ACT_RELU), 1, "dw_batch3_asym", "uniform"),
], ids=lambda s: s.name)
def test_depthwise_parity_records(spec):
    a = W.make_inputs(spec, 34)
    ref = util.oracle_ref(spec, a)
    recs = [spec.workload().default_schedule()]
    # unroll 0: shared-memory staged kernel; 1, 2, 4: register-window kernel with that many output rows per thread
    # (3x3 / 5x5 "same" filters; other filters fall back to the staged kernel)
    for tcn, by, bx, it, vw, th, un in ((4, 8, 32, 4, 4, 256, 0), (16, 4, 16, 2, 2, 128, 0), (1, 16, 64, 8, 4, 64, 0),
                                        (32, 7, 7, 1, 1, 512, 0), (3, 5, 24, 8, 1, 96, 0),
                                        (4, 8, 32, 4, 4, 256, 1), (1, 16, 64, 8, 4, 64, 2), (2, 7, 12, 4, 4, 512, 4),
                                        (8, 5, 8, 1, 1, 32, 4), (3, 6, 112, 4, 2, 96, 2), (2, 3, 16, 8, 4, 128, 1), (5, 9, 24, 8, 1, 64, 4)):
        recs.append(B.make_record(B.TT_FAMILY_DW_SIMT, tile_m=tcn, block_y=by, block_x=bx, items_per_thread=it,
                                  vec_width=vw, threads=th, unroll=un))
    # raster = 1: input boxes staged by TMA, persistent CTAs (image rows of 16-byte multiples; elsewhere legalised away)
    for tcn, by, bx, it, vw, th, un, st in ((4, 8, 32, 4, 4, 128, 2, 3), (1, 7, 16, 4, 4, 64, 4, 2), (16, 4, 8, 4, 2, 256, 1, 4),
                                            (3, 5, 28, 4, 4, 96, 2, 2), (8, 6, 56, 8, 4, 256, 2, 2), (5, 3, 16, 8, 4, 32, 1, 3),
                                            (32, 56, 56, 4, 4, 256, 1, 2)):
        recs.append(B.make_record(B.TT_FAMILY_DW_SIMT, tile_m=tcn, block_y=by, block_x=bx, items_per_thread=it, vec_width=vw,
                                  threads=th, unroll=un, raster=1, stages=st))
    outs = [run_spec(spec, r, a, ref, ref_elem=ref) for r in recs]
    for y in outs[1:]:
        np.testing.assert_array_equal(y, outs[0])       # same fp32 operations in the same order: bit-identical


@pytest.mark.parametrize("shape", [(12, 128, 128), (1, 1, 1), (3, 5, 37), (2, 9, 1000), (1, 300, 6)])
def test_softmax_parity_records(shape):
    spec = W.Spec(B.TT_OP_SOFTMAX, B.softmax_shapes(*shape, scale=0.125), 1, "softmax", "bert")
    a = W.make_inputs(spec, 35)
    a["x"] = a["x"] * 6.0
    ref = util.oracle_ref(spec, a)
    for bx, by, vw in ((32, 4, 1), (8, 16, 4), (1, 32, 1), (16, 3, 2), (4, 64, 4)):
        run_spec(spec, B.make_record(B.TT_FAMILY_ROW_SIMT, block_x=bx, block_y=by, vec_width=vw), a, ref, ref_elem=ref)


def test_split_k_is_bit_reproducible():
    spec = W._dense(128, 3072, 768)
    a = W.make_inputs(spec, 36)
    for sk in (8, 16):        # cluster reduction through distributed shared memory; workspace + last-arriving split
        r = tc(tile_n=128, tile_k=32, stages=4, split_k=sk, mma_m_axis=1)
        y1 = run_spec(spec, r, a)
        y2 = run_spec(spec, r, a)
        np.testing.assert_array_equal(y1, y2)


def test_run_requires_apply_and_pointers():
    spec = W._dense(8, 16, 8)
    wl = spec.workload()
    a = W.make_inputs(spec, 37)
    t, tt = W.device_tensors(spec, a)
    assert B.lib().tt_run(wl.handle, ctypes.byref(tt), None) == B.TT_ERR_NOT_APPLIED
    wl.apply(wl.default_schedule())
    bad = B.tensors(t["x"], t["w"], None, None, t["y"])
    assert B.lib().tt_run(wl.handle, ctypes.byref(bad), None) == B.TT_ERR_INVALID_ARG
    # an invalid record leaves the applied one in force
    st, _ = wl.try_apply(tc(stages=0))
    assert st == B.TT_ERR_INVALID_SCHEDULE
    wl.run(tt)
    assert util.rel_l2(t["y"].cpu().numpy(), util.oracle_ref(spec, a)) <= util.TOL_TF32


def test_run_host_matches_oracle():
    import torch
    spec = W._conv(16, 14, 32, 3, 1, 1)
    a = W.make_inputs(spec, 38)
    wl = spec.workload()
    wl.apply(tc(tile_n=64, tile_k=32, stages=3))
    host = {k: (None if v is None else torch.from_numpy(v).pin_memory()) for k, v in a.items()}
    y = torch.empty(W.tensor_shapes(spec)[4], dtype=torch.float32).pin_memory()
    up, down = wl.run_host(B.tensors(host["x"], host["w"], host["bias"], None, y))
    assert up == 4 * (a["x"].size + a["w"].size + a["bias"].size) and down == 4 * y.numel()
    assert util.rel_l2(y.numpy(), util.oracle_ref(spec, a)) <= util.TOL_TF32


def test_run_host_async_on_several_streams_matches_oracle():
    """tt_run_host_async: several workloads enqueued on different streams (each workload always on its own), twice
    each, nothing synchronised in between; after tt_workload_status every output equals the oracle's."""
    import torch
    specs = [W._conv(16, 14, 32, 3, 1, 1), W._dw(24, 28, 1), W._dense(8, 96, 40), W._conv(32, 14, 64, 1, 1, 0)]
    streams = [torch.cuda.Stream() for _ in range(3)]
    jobs = []
    for i, spec in enumerate(specs):
        a = W.make_inputs(spec, 60 + i)
        wl = spec.workload()
        wl.apply(wl.default_schedule())
        host = {k: (None if v is None else torch.from_numpy(v).pin_memory()) for k, v in a.items()}
        y = torch.full(W.tensor_shapes(spec)[4], float("nan"), dtype=torch.float32).pin_memory()
        jobs.append((spec, a, wl, host, y, streams[i % len(streams)]))
    torch.cuda.synchronize()
    for _ in range(2):
        for spec, a, wl, host, y, st in jobs:
            up, down = wl.run_host_async(B.tensors(host["x"], host["w"], host["bias"], None, y), st)
            assert down == 4 * y.numel() and up > 0
    for spec, a, wl, host, y, st in jobs:
        assert wl.status(st) == B.TT_OK                  # synchronises that workload's stream
        assert util.rel_l2(y.numpy(), util.oracle_ref(spec, a)) <= util.tolerance(spec.op), spec.name
        wl.close()


def test_timing_and_grid_tuner_smoke():
    spec = W._conv(32, 14, 64, 3, 1, 1)
    a = W.make_inputs(spec, 39)
    wl = spec.workload()
    t, tt = W.device_tensors(spec, a)
    wl.apply(wl.default_schedule())
    o = B.tt_timing_opts()
    o.batches, o.warmup_batches, o.min_batch_us = 4, 1, 50
    tm = wl.time(tt, o)
    assert 0 < tm.min_us <= tm.median_us <= tm.max_us and tm.batches == 4
    o.use_graph = 1
    tg = wl.time([tt, tt], o)
    assert tg.median_us > 0
    best, tried = wl.grid_tune(tt, o, level=0, top_k=3)
    assert tried > 10 and 1 <= len(best) <= 3
    assert best[0][1] <= best[-1][1]
    assert best[0][0].origin_op == B.TT_OP_CONV2D and best[0][0].origin.c == 32
    wl.run(tt)                                     # the best record is left applied
    assert util.rel_l2(t["y"].cpu().numpy(), util.oracle_ref(spec, a)) <= util.TOL_TF32


@pytest.mark.parametrize("spec,start", [
    (W._conv(128, 28, 128, 3, 1, 1), tc(tile_n=32, tile_k=16, stages=2, split_k=1, mma_m_axis=2)),
    (W._dw(96, 56, 1), B.make_record(B.TT_FAMILY_DW_SIMT, tile_m=1, block_y=2, block_x=8, items_per_thread=1, vec_width=1,
                                     threads=32, unroll=0)),
], ids=lambda v: getattr(v, "name", None) or "start")
def test_refining_a_transferred_record_never_loses_time_and_stays_correct(spec, start):
    """tt_refine: greedy one-field-at-a-time descent from a (deliberately poor) transferred record.  The result is at
    least as fast as the start by the search's own timings, is left applied, and computes what the oracle does."""
    a = W.make_inputs(spec, 41)
    wl = spec.workload()
    t, tt = W.device_tensors(spec, a)
    o = B.tt_timing_opts()
    o.batches, o.warmup_batches, o.min_batch_us, o.use_graph = 5, 1, 100, 1
    best, best_us, start_us, timed = wl.refine(tt, start, o, max_rounds=3, min_gain=0.02)
    assert 0 < best_us <= start_us and timed >= 2
    assert wl.check(best)[0] == B.TT_OK
    if best_us < start_us:                          # a move was made: the record differs from the (legalised) start
        assert best.as_dict() != wl.check(start)[1].legal.as_dict()
    t["y"].fill_(float("nan"))
    wl.run(tt)                                      # the best record is left applied
    assert wl.status() == B.TT_OK
    assert util.rel_l2(t["y"].cpu().numpy(), util.oracle_ref(spec, a)) <= util.tolerance(spec.op)
    wl.close()


def _model_parity(model, seed, recs):
    specs = W.MODELS[model]()
    for i, spec in enumerate(specs):
        a = W.make_inputs(spec, seed, i)
        ref = util.oracle_ref(spec, a)
        re = elem_ref(spec, a, ref)
        rr = [spec.workload().default_schedule()] + (recs if spec.op in (B.TT_OP_CONV2D, B.TT_OP_DENSE, B.TT_OP_BATCH_MATMUL) else [])
        for r in rr:
            run_spec(spec, r, a, ref, ref_elem=re)


def test_resnet18_full_size_every_kernel():
    _model_parity("resnet18", 2, [tc(tile_n=64, tile_k=64, stages=3, split_k=4, mma_m_axis=2),
                                  tc(tile_n=256, tile_k=32, stages=3, split_k=1, raster=1, mma_m_axis=1)])


def test_mobilenet_v2_full_size_every_kernel():
    _model_parity("mobilenet_v2", 4, [tc(tile_n=32, tile_k=16, stages=4, split_k=2, mma_m_axis=2)])


def test_bert_base_full_size_every_kernel():
    _model_parity("bert_base", 5, [tc(tile_n=64, tile_k=32, stages=4, split_k=3, mma_m_axis=1)])


def test_resnet50_full_size_sampled_filters():
    """Full-size kernels under three records, outputs sampled by filter: a convolution restricted to some filters is
    exactly those output channels, so the oracle computes only them (exact mode for the rel-L2 of record, truncation
    mode for the bound on every single sampled output)."""
    specs = W.resnet50()
    recs = [tc(tile_n=128, tile_k=32, stages=4, split_k=2, mma_m_axis=1),
            tc(tile_n=64, tile_k=64, stages=3, split_k=1, raster=1, mma_m_axis=2, slab_tiles=2),
            tc(tile_n=256, tile_k=32, stages=2, split_k=1, mma_m_axis=1, k_order=1)]
    for i, spec in enumerate(specs):
        a = W.make_inputs(spec, 3, i)
        ys = [run_spec(spec, rec, a) for rec in recs if spec.workload().check(rec)[0] == B.TT_OK]
        assert len(ys) >= 2, spec.name
        if spec.op == B.TT_OP_CONV2D:
            ks = sorted({0, spec.shapes.k // 3, spec.shapes.k - 1})
            geo = ((spec.shapes.stride_h,) * 2, (spec.shapes.pad_h,) * 2, spec.shapes.act)
            res = None if a["residual"] is None else np.ascontiguousarray(a["residual"][:, ks])
            sub = orc.conv2d(a["x"], a["w"][ks], a["bias"][ks], *geo, residual=res)
            sub_t = orc.conv2d(a["x"], a["w"][ks], a["bias"][ks], *geo, residual=res, mode=orc.MODE_TF32_TRUNC)
            for y in ys:
                assert util.rel_l2(y[:, ks], sub) <= util.TOL_TF32, spec.name
                assert np.abs(y[:, ks].astype(np.float64) - sub_t).max() <= ELEM_TF32 * np.abs(sub_t).max(), spec.name
        else:
            for y in ys:
                assert util.rel_l2(y, util.oracle_ref(spec, a)) <= util.TOL_TF32
        for y in ys[1:]:
            assert util.rel_l2(y, ys[0]) <= INVARIANCE_TOL, spec.name


def test_largest_dense_sampled_outputs():
    """The largest kernel of the pool sources (25088 -> 4096, 411 MB of weights), checked on sampled out-features."""
    spec = W._dense(1, 25088, 4096, B.TT_ACT_RELU)
    a = W.make_inputs(spec, 40)
    y = run_spec(spec, tc(tile_n=16, tile_k=64, stages=4, split_k=16), a)
    rows = [0, 1, 127, 128, 2047, 4000, 4095]
    sub = orc.dense(a["x"], a["w"][rows], a["bias"][rows], B.TT_ACT_RELU)
    assert util.rel_l2(y[:, rows], sub) <= util.TOL_TF32


def test_chained_kernels_on_one_stream_see_each_others_results():
    """Kernels are launched so that a kernel's set-up may overlap the tail of the one before it in the stream; every
    global access still comes after the previous kernel has finished.  A chain in which each layer reads the output of
    the layer before it (conv3x3 -> conv1x1/2 cluster split-K -> depthwise -> conv3x3 workspace split-K), launched back
    to back without any synchronisation, several times over, must equal the same chain on the oracle."""
    import torch
    layers = [
        (W._conv(16, 20, 32, 3, 1, 1), tc(tile_n=64, tile_k=32, stages=3, mma_m_axis=1)),
        (W._conv(32, 20, 48, 1, 2, 0, act=B.TT_ACT_NONE), tc(tile_n=32, tile_k=8, stages=2, split_k=4, mma_m_axis=2)),
        (W._dw(48, 10, 1), B.make_record(B.TT_FAMILY_DW_SIMT, tile_m=4, block_y=4, block_x=8, items_per_thread=4, vec_width=2,
                                          threads=64, unroll=2)),
        (W._conv(48, 10, 24, 3, 1, 1, act=B.TT_ACT_RELU6), tc(tile_n=48, tile_k=16, stages=2, split_k=12, mma_m_axis=1)),
    ]
    arrays = [W.make_inputs(sp, 61, i) for i, (sp, _) in enumerate(layers)]
    # oracle chain
    x = arrays[0]["x"]
    for (sp, _), a in zip(layers, arrays):
        a = dict(a)
        a["x"] = x
        x = util.oracle_ref(sp, a)
    ref = x
    # device chain: layer i writes the buffer layer i + 1 reads
    wls, tts, keep = [], [], []
    first = cur = torch.from_numpy(arrays[0]["x"]).cuda()      # `first` keeps the chain's input alive
    for (sp, rec), a in zip(layers, arrays):
        wl = sp.workload()
        wl.apply(rec)
        t, _ = W.device_tensors(sp, a)
        assert tuple(cur.shape) == tuple(t["x"].shape)
        tts.append(B.tensors(cur, t["w"], t["bias"], None, t["y"]))
        keep.append(t)
        wls.append(wl)
        cur = t["y"]
    for _ in range(5):
        for t in keep:
            t["y"].fill_(float("nan"))
        for wl, tt in zip(wls, tts):
            wl.run(tt)
        torch.cuda.synchronize()
        y = cur.cpu().numpy()
        assert not np.isnan(y).any()
        assert util.rel_l2(y, ref) <= 3 * util.TOL_TF32      # three TF32 layers in a row
    for wl in wls:
        assert wl.status() == B.TT_OK
        wl.close()
    del first


def _sampled_filters_ok(spec, rec, seed):
    a = W.make_inputs(spec, seed)
    y = run_spec(spec, rec, a)
    ks = sorted({0, spec.shapes.k // 2 + 1, spec.shapes.k - 1})
    sub = orc.conv2d(a["x"], a["w"][ks], a["bias"][ks], (spec.shapes.stride_h,) * 2, (spec.shapes.pad_h,) * 2, spec.shapes.act)
    assert util.rel_l2(y[:, ks], sub) <= util.TOL_TF32, (spec.name, rec.short())


def test_vgg_shaped_pool_source_convs_sampled_filters():
    """The widest images of the pool sources (224 x 224: the slab rows are 228 floats, chunks of a few channels) and a
    512-channel layer whose reduction needs many slab chunks, checked on sampled filters."""
    recs = [tc(tile_n=128, tile_k=32, stages=3, mma_m_axis=1),
            tc(tile_n=256, tile_k=64, stages=2, slab_tiles=2, mma_m_axis=1),
            tc(tile_n=64, tile_k=32, stages=2, split_k=3, mma_m_axis=2)]
    for i, spec in enumerate([W._conv(3, 224, 64, 3, 1, 1), W._conv(64, 224, 64, 3, 1, 1), W._conv(512, 28, 512, 3, 1, 1)]):
        for rec in recs:
            _sampled_filters_ok(spec, rec, 70 + i)


def test_batched_kernels_of_the_saturating_size_points():
    """The batched shapes that bench.py times at saturating size, at a smaller batch, under the records it uses:
    sampled filters for the convolutions, every output for depthwise and softmax."""
    conv = W.Spec(B.TT_OP_CONV2D, B.conv2d_shapes(6, 128, 28, 28, 128, 3, 3, 1, 1, True, B.TT_ACT_RELU), 1, "conv3x3_n6_128x28")
    _sampled_filters_ok(conv, tc(tile_n=256, tile_k=32, stages=2, mma_m_axis=1), 80)
    _sampled_filters_ok(conv, tc(tile_n=128, tile_k=64, stages=2, mma_m_axis=2), 80)
    pw = W.Spec(B.TT_OP_CONV2D, B.conv2d_shapes(5, 256, 56, 56, 64, 1, 1, 1, 0, True, B.TT_ACT_RELU), 1, "conv1x1_n5_256x56")
    _sampled_filters_ok(pw, tc(tile_n=256, tile_k=32, stages=2, mma_m_axis=1), 81)
    dw = W.Spec(B.TT_OP_DWCONV2D, B.make_shapes(n=3, c=144, h=56, w=56, k=144, r=3, s=3, stride_h=1, stride_w=1, pad_h=1,
                                                  pad_w=1, has_bias=1, act=B.TT_ACT_RELU6), 1, "dw_n3_144x56")
    a = W.make_inputs(dw, 82)
    ref = util.oracle_ref(dw, a)
    for rec in (B.make_record(B.TT_FAMILY_DW_SIMT, tile_m=8, block_y=56, block_x=56, items_per_thread=8, vec_width=4,
                              threads=128, unroll=2),
                B.make_record(B.TT_FAMILY_DW_SIMT, tile_m=4, block_y=16, block_x=56, items_per_thread=4, vec_width=4,
                              threads=128, unroll=4)):
        run_spec(dw, rec, a, ref)
    sm = W.Spec(B.TT_OP_SOFTMAX, B.softmax_shapes(12 * 8, 128, 128, 0.125), 1, "softmax_96x128x128", "bert")
    a = W.make_inputs(sm, 83)
    run_spec(sm, B.make_record(B.TT_FAMILY_ROW_SIMT, block_x=16, block_y=4, vec_width=4), a, util.oracle_ref(sm, a))


def _random_records(family, n, seed):
    """Seeded draws from the record space the tuner walks (and a little beyond it): any legal record, however ill
    suited to the shape, must still compute the same kernel."""
    import random
    rng = random.Random(seed)
    recs = []
    for _ in range(n):
        if family == B.TT_FAMILY_GEMM_TC:
            recs.append(tc(tile_n=rng.choice([16, 32, 48, 64, 96, 128, 160, 192, 256]), tile_k=rng.choice([8, 16, 32, 64, 96, 128]),
                           stages=rng.choice([1, 2, 3, 4, 6, 8]), split_k=rng.choice([1, 1, 2, 3, 4, 5, 8, 9, 16]),
                           raster=rng.choice([0, 1]), mma_m_axis=rng.choice([0, 1, 2]), slab_tiles=rng.choice([0, 0, 1, 2, 5]),
                           acc_split=rng.choice([1, 1, 2, 4, 8]), k_order=rng.choice([0, 0, 1]),
                           persistent=rng.choice([0, 0, 1]), cta_group=rng.choice([1, 1, 2]), ctas_per_sm=rng.choice([0, 1, 2]),
                           precision=rng.choice([0, 0, 0, 1])))
        else:
            recs.append(B.make_record(B.TT_FAMILY_DW_SIMT, tile_m=rng.choice([1, 2, 4, 8, 16, 32]), block_y=rng.choice([1, 2, 4, 7, 8, 14, 28]),
                                      block_x=rng.choice([4, 8, 16, 28, 32, 56]), items_per_thread=rng.choice([1, 2, 4, 8]),
                                      vec_width=rng.choice([1, 2, 4]), threads=rng.choice([32, 64, 128, 256, 512]),
                                      unroll=rng.choice([0, 1, 2, 4]), raster=rng.choice([0, 1]), stages=rng.choice([1, 2, 3, 4, 6])))
    return recs


@pytest.mark.parametrize("spec,n", [
    (W._conv(48, 20, 80, 3, 1, 1, name="rand_conv3x3"), 40),
    (W._conv(40, 14, 72, 3, 2, 1, act=B.TT_ACT_RELU6, name="rand_conv3x3s2"), 25),
    (W._dense(70, 300, 200, act=B.TT_ACT_GELU_ERF, name="rand_dense"), 25),
    (W.Spec(B.TT_OP_BATCH_MATMUL, B.bmm_shapes(3, 40, 56, 48, False), 1, "rand_bmm_nn", "bert"), 15),
    (W._dw(24, 28, 1), 25),
], ids=lambda v: getattr(v, "name", str(v)))
def test_a_schedule_changes_speed_never_semantics_random_records(spec, n):
    a = W.make_inputs(spec, 90)
    ref = util.oracle_ref(spec, a)
    fam = B.TT_FAMILY_DW_SIMT if spec.op == B.TT_OP_DWCONV2D else B.TT_FAMILY_GEMM_TC
    re = elem_ref(spec, a, ref)
    probe = spec.workload()
    ran = 0
    for rec in _random_records(fam, n, seed=sum(map(ord, spec.name))):
        st, _ = probe.check(rec)
        assert st in (B.TT_OK, B.TT_ERR_RESOURCE), (rec.short(), st)
        if st == B.TT_OK:
            run_spec(spec, rec, a, ref, ref_elem=re)
            ran += 1
    probe.close()
    assert ran >= n * 2 // 3


def test_sequence_length_transfer_256_tokens_under_records_tuned_on_128():
    """Section 5.4: schedules tuned for one input size of a model reused on another.  The kernels of the 256-token
    encoder run under records natively tuned on the 128-token encoder's kernels (and the reverse for one layer): every
    output within tolerance, element-wise bound included, and the evaluator's selection reproduces the oracle's argmin."""
    o = B.tt_timing_opts()
    o.batches, o.warmup_batches, o.min_batch_us, o.use_graph = 3, 1, 50, 1
    pool = []
    for j, sp in enumerate(W.bert_base()):
        a = W.make_inputs(sp, 105, j)
        wl = sp.workload()
        _, tt = W.device_tensors(sp, a)
        best, _ = wl.grid_tune(tt, o, level=0, top_k=2)
        pool += [r for r, _ in best]
        wl.close()
    assert all(r.origin.m == 128 for r in pool)
    for i, sp in enumerate(W.bert_base_256()):
        a = W.make_inputs(sp, 5, i)
        ref = util.oracle_ref(sp, a)
        re = elem_ref(sp, a, ref)
        probe = sp.workload()
        fam = probe.family()
        ran = 0
        for rec in pool:
            if rec.family != fam or probe.check(rec)[0] != B.TT_OK:
                continue
            run_spec(sp, rec, a, ref, ref_elem=re)
            ran += 1
        probe.close()
        assert ran >= 2, sp.name
    # the evaluator on the 256-token kernels with the 128-token pool: a complete, valid table
    specs = W.bert_base_256()
    arrays = [W.make_inputs(sp, 5, i) for i, sp in enumerate(specs)]
    wls = [sp.workload() for sp in specs]
    keep, tts = zip(*[W.device_tensors(sp, a) for sp, a in zip(specs, arrays)])
    opts = B.tt_tune_opts()
    opts.include_default = 1
    opts.timing = o
    res = B.transfer_tune(list(wls), list(tts), pool, opts)
    n_cols = len(pool) + 1
    flat = [v for row in res["times_us"] for v in row]
    assert res["chosen"] == orc.select(flat, len(wls), n_cols)
    assert all(c >= 0 for c in res["chosen"]) and res["pairs_timed"] >= len(wls) * 3
    for w in wls:
        w.close()


def test_bounded_wait_expires_reports_timeout_and_the_workload_recovers():
    """A wait inside the kernel that can never be satisfied (the first stage's barrier is told to expect more bytes
    than its copies deliver: every copy lands, the barrier never completes) runs into the wait limit: tt_run returns,
    the status word says TT_ERR_TIMEOUT, nothing traps, and the same workload then runs normally.  An invalid pair is
    a result of the search, which goes on (Section 4.3)."""
    import torch
    # (a) one CTA, no split; (b) twelve splits through the workspace, of which only split 0 stalls: the other eleven
    # arrive at the tile counters, which the status path has to clear again or the next run finishes tiles early;
    # (c) three splits as a thread-block cluster: split 0 gives up and sends nothing, its peers send it their bands, then
    # give up waiting for its band, and all three leave together
    for spec, rec in ((W._dense(8, 16, 8, name="stall_one_cta"), tc(tile_n=16, tile_k=16, stages=2, mma_m_axis=1)),
                      (W._dense(96, 1536, 200, name="stall_split12"), tc(tile_n=64, tile_k=32, stages=3, split_k=12, mma_m_axis=1)),
                      (W._dense(96, 768, 200, name="stall_cluster3"), tc(tile_n=64, tile_k=32, stages=3, split_k=3, mma_m_axis=2))):
        a = W.make_inputs(spec, 77)
        ref = util.oracle_ref(spec, a)
        wl = spec.workload()
        info = wl.apply(rec)
        assert info.legal.split_k == rec.split_k
        t, tt = W.device_tensors(spec, a)
        wl.set_wait_limit(2_000_000)                    # 2 ms
        wl.test_stall(64)
        t["y"].fill_(float("nan"))
        wl.run(tt)
        assert wl.status() == B.TT_ERR_TIMEOUT
        assert wl.status() == B.TT_OK                   # reading the status cleared it
        torch.cuda.synchronize()                        # the context is alive
        wl.test_stall(0)
        for _ in range(2):
            t["y"].fill_(float("nan"))
            wl.run(tt)
            assert wl.status() == B.TT_OK
            y = t["y"].cpu().numpy()
            assert not np.isnan(y).any()
            assert util.rel_l2(y, ref) <= util.TOL_TF32, spec.name
        # and after a fresh apply with the default limit
        wl.set_wait_limit(1_000_000_000)
        wl.apply(rec)
        wl.run(tt)
        assert wl.status() == B.TT_OK
        assert util.rel_l2(t["y"].cpu().numpy(), ref) <= util.TOL_TF32
        wl.close()


def _tf32_depth(steps):
    """Per node: the number of TF32 layers on the longest path that leads to it (each may add the TF32 tolerance)."""
    depth = []
    for st in steps:
        if st.spec is None:
            depth.append(0)
            continue
        d = max([depth[i] for i in (st.x, st.res, st.w_from) if i is not None])
        depth.append(d + (1 if st.spec.op in (B.TT_OP_CONV2D, B.TT_OP_DENSE, B.TT_OP_BATCH_MATMUL) else 0))
    return depth


@pytest.mark.parametrize("model,make,seed", [
    ("resnet18", W.resnet18_net, 2),
    ("mobilenet_v2", W.mobilenet_v2_net, 4),
    ("resnet50", W.resnet50_net, 3),
    ("bert_base_2_layers", lambda: W.bert_base_net(layers=2), 5),
], ids=lambda v: v if isinstance(v, str) else "")
def test_data_chained_model_pass_matches_the_oracle_chain(model, make, seed):
    """The whole model as a chain: every layer reads the buffer its producer wrote (and the skip tensor of its block),
    all launched back to back on one stream without synchronisation, three passes.  Every layer's output is compared
    with the same chain on the oracle; a layer k TF32 layers deep may be off by k times the TF32 tolerance.  Run once
    under the default records and once under a record that uses cluster split-K and the other accumulator axis."""
    import torch
    specs, steps = make()
    arrays = W.make_chain_inputs(steps, seed, init="bert" if model.startswith("bert") else "he")
    refs = util.oracle_chain(steps, arrays)
    depth = _tf32_depth(steps)
    alt = tc(tile_n=64, tile_k=32, stages=3, split_k=2, mma_m_axis=2)
    for use_alt in (False, True):
        wls = [sp.workload() for sp in specs]
        for wl in wls:
            rec = alt if use_alt and wl.family() == B.TT_FAMILY_GEMM_TC else wl.default_schedule()
            wl.apply(rec)
            wl.set_constant_weights(use_alt)              # the second pass also fetches the weights early
        bufs, tts = W.chain_device_tensors(steps, arrays)
        for _ in range(3):
            for st, b in zip(steps, bufs):
                if st.spec is not None:
                    b["y"].fill_(float("nan"))
            for st, tt in zip(steps, tts):
                if st.spec is not None:
                    wls[st.kernel].run(tt)
            torch.cuda.synchronize()
        for wl in wls:
            assert wl.status() == B.TT_OK
        for i, (st, b, ref, d) in enumerate(zip(steps, bufs, refs, depth)):
            if st.spec is None:
                continue
            y = b["y"].cpu().numpy()
            assert not np.isnan(y).any(), (model, i, st.spec.name)
            tol = max(d, 1) * util.TOL_TF32 if d else util.TOL_FP32
            assert util.rel_l2(y, ref) <= tol, (model, i, st.spec.name, d, util.rel_l2(y, ref))
        for wl in wls:
            wl.close()


@pytest.mark.parametrize("spec", [
    W._dense(700, 520, 900, act=B.TT_ACT_GELU_ERF, name="ps_dense_many_tiles"),
    W._dense(300, 64, 5000, act=B.TT_ACT_RELU, name="ps_dense_short_k"),
    W.Spec(B.TT_OP_BATCH_MATMUL, B.bmm_shapes(200, 128, 128, 64, True), 1, "ps_bmm_nt_200", "bert"),
    W.Spec(B.TT_OP_BATCH_MATMUL, B.bmm_shapes(200, 128, 64, 128, False), 1, "ps_bmm_nn_200", "bert"),
    W.Spec(B.TT_OP_BATCH_MATMUL, B.bmm_shapes(7, 150, 76, 52, False), 1, "ps_bmm_nn_ragged", "bert"),
    W.Spec(B.TT_OP_CONV2D, B.conv2d_shapes(5, 96, 28, 28, 200, 1, 1, 1, 0, True, B.TT_ACT_RELU6), 1, "ps_conv1x1_n5", "uniform"),
    W.Spec(B.TT_OP_CONV2D, B.conv2d_shapes(3, 40, 14, 14, 24, 1, 1, 1, 0, True, B.TT_ACT_NONE, True), 1, "ps_conv1x1_res", "uniform"),
], ids=lambda s: s.name)
def test_persistent_form_walks_many_tiles(spec):
    """More tiles than SMs (or many batch entries), so that every CTA of the persistent form walks several tiles, both
    accumulators are used over and over and the operand pipeline wraps across tile boundaries; ragged tails in every
    dimension.  The one-tile form under the same tile sizes gives the same values up to the fp32 summation order."""
    a = W.make_inputs(spec, 91)
    ref = util.oracle_ref(spec, a)
    re = elem_ref(spec, a, ref)
    outs = []
    probe = spec.workload()
    for rec in (tc(tile_n=16, tile_k=32, stages=4, mma_m_axis=1),
                tc(tile_n=16, tile_k=32, stages=4, persistent=1, mma_m_axis=1),
                tc(tile_n=32, tile_k=16, stages=7, persistent=1, mma_m_axis=2),
                tc(tile_n=48, tile_k=64, stages=2, persistent=1, raster=1, mma_m_axis=1),
                tc(tile_n=32, tile_k=32, stages=3, persistent=1, cta_group=2, mma_m_axis=1),
                tc(tile_n=64, tile_k=32, stages=5, persistent=1, cta_group=2, raster=1, mma_m_axis=2)):
        st, info = probe.check(rec)
        assert st == B.TT_OK
        if rec.persistent:
            assert info.legal.persistent == 1, "this kernel has the persistent form"
            assert info.grid_y == 1 and info.grid_z == 1
        outs.append(run_spec(spec, rec, a, ref, ref_elem=re))
    probe.close()
    for y in outs[1:]:
        assert util.rel_l2(y, outs[0]) <= INVARIANCE_TOL


def test_constant_weights_are_fetched_early_and_results_do_not_change():
    """With the caller's promise that the weights are constants, a dense or conv2d kernel requests their first tiles
    before it waits for the kernel in front of it.  Layers launched back to back -- each reading its predecessor's
    output, with that promise and without it -- give bit-identical results, equal to the oracle chain."""
    import torch
    layers = [(W._dense(128, 768, 768, name="cw_a"), tc(tile_n=64, tile_k=32, stages=3, split_k=8, mma_m_axis=2)),
              (W._dense(128, 768, 3072, act=B.TT_ACT_GELU_ERF, name="cw_b"), tc(tile_n=32, tile_k=128, stages=2, mma_m_axis=1)),
              (W._dense(128, 3072, 768, name="cw_c"), tc(tile_n=64, tile_k=64, stages=3, split_k=6, mma_m_axis=2)),
              (W._dense(128, 768, 768, name="cw_d"), tc(tile_n=64, tile_k=32, stages=4, persistent=1, mma_m_axis=1))]
    arrays = [W.make_inputs(sp, 95, i) for i, (sp, _) in enumerate(layers)]
    x = arrays[0]["x"]
    for (sp, _), a in zip(layers, arrays):
        a = dict(a)
        a["x"] = x
        x = util.oracle_ref(sp, a)
    ref = x
    results = []
    for promise in (False, True):
        wls, tts, keep = [], [], []
        first = cur = torch.from_numpy(arrays[0]["x"]).cuda()
        for (sp, rec), a in zip(layers, arrays):
            wl = sp.workload()
            wl.apply(rec)
            wl.set_constant_weights(promise)
            t, _ = W.device_tensors(sp, a)
            tts.append(B.tensors(cur, t["w"], t["bias"], None, t["y"]))
            keep.append(t)
            wls.append(wl)
            cur = t["y"]
        for _ in range(4):
            for t in keep:
                t["y"].fill_(float("nan"))
            for wl, tt in zip(wls, tts):
                wl.run(tt)
            torch.cuda.synchronize()
        for wl in wls:
            assert wl.status() == B.TT_OK
            wl.close()
        y = cur.cpu().numpy()
        assert util.rel_l2(y, ref) <= 4 * util.TOL_TF32
        results.append(y)
        del first
    np.testing.assert_array_equal(results[0], results[1])


@pytest.mark.parametrize("spec", [
    W.Spec(B.TT_OP_CONV2D, B.conv2d_shapes(20, 40, 20, 20, 72, 3, 3, 1, 1, True, B.TT_ACT_RELU), 1, "ps_tap_conv3x3_n20", "uniform"),
    W.Spec(B.TT_OP_CONV2D, B.conv2d_shapes(9, 33, 12, 16, 136, 5, 3, 1, 2, True, B.TT_ACT_RELU6), 1, "ps_tap_conv5x3_n9", "uniform"),
    W.Spec(B.TT_OP_CONV2D, B.conv2d_shapes(30, 8, 8, 8, 16, 3, 3, 1, 1, False, B.TT_ACT_NONE), 1, "ps_tap_small_n30", "uniform"),
], ids=lambda s: s.name)
def test_persistent_tap_major_convolution_walks_many_tiles(spec):
    """The tap-major reduction order in the persistent form: filter stages, the staging ring and the two pixel-major
    slab buffers all run on across tile boundaries (several tiles per CTA, one or several 32-channel blocks per tile,
    a partial last block, two filter tiles).  Same values as the one-tile form and as the stored reduction order."""
    a = W.make_inputs(spec, 92)
    ref = util.oracle_ref(spec, a)
    re = elem_ref(spec, a, ref)
    outs = []
    probe = spec.workload()
    for rec in (tc(tile_n=32, tile_k=32, stages=3, mma_m_axis=1),
                tc(tile_n=48, tile_k=32, stages=3, k_order=1, mma_m_axis=1),
                tc(tile_n=48, tile_k=32, stages=3, k_order=1, persistent=1, mma_m_axis=1),
                tc(tile_n=16, tile_k=96, stages=2, k_order=1, persistent=1, raster=1, mma_m_axis=1),
                tc(tile_n=96, tile_k=32, stages=6, k_order=1, persistent=1, mma_m_axis=1),
                tc(tile_n=256, tile_k=64, stages=2, k_order=1, persistent=1, mma_m_axis=1)):
        st, info = probe.check(rec)
        assert st == B.TT_OK
        if rec.persistent:
            assert info.legal.persistent == 1 and info.legal.k_order == 1
        outs.append(run_spec(spec, rec, a, ref, ref_elem=re))
    probe.close()
    for y in outs[1:]:
        assert util.rel_l2(y, outs[0]) <= INVARIANCE_TOL


def test_subsampled_evaluator_skips_what_the_rule_says_and_keeps_a_valid_choice():
    """Pool sub-sampling: the seeded subset is evaluated first; with a bar nothing can clear (100 % gain) every record is
    still evaluated, with a bar everything clears (a negative gain) only the subset is, the rest is marked TT_SKIPPED,
    and the chosen record is the argmin over what was evaluated."""
    spec = W._conv(32, 14, 64, 3, 1, 1)
    a = W.make_inputs(spec, 44)
    wl = spec.workload()
    t, tt = W.device_tensors(spec, a)
    pool = [tc(tile_n=tn, tile_k=tk, stages=st) for tn in (32, 64, 128) for tk in (16, 32) for st in (2, 3)]   # 12 records
    o = B.tt_tune_opts()
    o.include_default = 1
    o.timing.warmup_batches, o.timing.batches, o.timing.min_batch_us, o.timing.use_graph = 1, 3, 50, 1
    o.subsample_percent, o.subsample_seed = 25, 11
    first = B.pool_subsample(len(pool), 3, 11)
    assert first == orc.pool_subsample(len(pool), 3, 11)
    o.subsample_gain_percent = 100                       # unreachable: the whole pool gets evaluated
    res = B.transfer_tune([wl], [tt], pool, o)
    assert res["pairs_skipped"] == 0 and res["pairs_timed"] == 13
    o.subsample_gain_percent = -1000                     # any valid subset record ends the search
    res = B.transfer_tune([wl], [tt], pool, o)
    st = res["status"][0]
    evaluated = {0} | {f + 1 for f in first}
    assert {j for j, s in enumerate(st) if s == B.TT_OK} == evaluated
    assert all(st[j] == B.TT_SKIPPED and res["times_us"][0][j] == -1.0 for j in range(13) if j not in evaluated)
    assert res["pairs_skipped"] == 9 and res["pairs_timed"] == 4
    assert res["chosen"] == orc.select(res["times_us"][0], 1, 13) and res["chosen"][0] in evaluated
    wl.run(tt)                                           # the chosen record is left applied
    assert util.rel_l2(t["y"].cpu().numpy(), util.oracle_ref(spec, a)) <= util.TOL_TF32
    wl.close()


@pytest.mark.parametrize("model,make,seed", [("resnet18", W.resnet18_net, 2), ("bert_base", lambda: W.bert_base_net(layers=2), 5)])
def test_chain_on_several_streams_matches_the_oracle_chain(model, make, seed):
    """The same chain with layers that do not depend on one another on side streams (the attention projections, a
    block's downsample beside its first convolution), enqueued directly and replayed as one captured graph: every
    layer's output against the oracle chain.  The projections share one workload object and run beside one another."""
    import torch
    specs, steps = make()
    arrays = W.make_chain_inputs(steps, seed, init="bert" if model.startswith("bert") else "he")
    refs = util.oracle_chain(steps, arrays)
    depth = _tf32_depth(steps)
    wls = [sp.workload() for sp in specs]
    rec = tc(tile_n=64, tile_k=64, stages=2, split_k=4, mma_m_axis=2)
    for wl in wls:
        wl.apply(rec if wl.family() == B.TT_FAMILY_GEMM_TC else wl.default_schedule())
        wl.set_constant_weights(True)
    bufs, tts = W.chain_device_tensors(steps, arrays)
    plan = W.chain_lanes(steps, max_lanes=4)
    assert len({pl[0] for pl in plan if pl}) == 4
    side = [torch.cuda.Stream() for _ in range(3)]

    def clear():
        for st, b in zip(steps, bufs):
            if st.spec is not None:
                b["y"].fill_(float("nan"))

    def check(what):
        for wl in wls:
            assert wl.status() == B.TT_OK
        for i, (st, b, ref, d) in enumerate(zip(steps, bufs, refs, depth)):
            if st.spec is None:
                continue
            y = b["y"].cpu().numpy()
            assert not np.isnan(y).any(), (what, model, i, st.spec.name)
            tol = max(d, 1) * util.TOL_TF32 if d else util.TOL_FP32
            assert util.rel_l2(y, ref) <= tol, (what, model, i, st.spec.name, d, util.rel_l2(y, ref))

    main = torch.cuda.Stream()
    with torch.cuda.stream(main):
        for _ in range(2):
            clear()
            W.run_chain(wls, steps, tts, plan, [main] + side)
        main.synchronize()
    torch.cuda.synchronize()
    check("direct")
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=main):
        W.run_chain(wls, steps, tts, plan, [torch.cuda.current_stream()] + side)
    for _ in range(3):
        clear()
        torch.cuda.synchronize()
        graph.replay()
        torch.cuda.synchronize()
    check("graph")
    for wl in wls:
        wl.close()


@pytest.mark.parametrize("spec", [
    W._dense(300, 1024, 520, act=B.TT_ACT_GELU_ERF, name="x3_dense"),
    W.Spec(B.TT_OP_BATCH_MATMUL, B.bmm_shapes(6, 200, 136, 256, True), 1, "x3_bmm_nt", "bert"),
])
def test_compensated_products_come_within_fp32_accumulation_of_the_exact_result(spec):
    """precision = 1: what the tensor core drops of each operand (everything below TF32's ten mantissa bits) is fed
    back through two more products per step, so the result must sit far inside the TF32 tolerance: at least twenty
    times closer to the exact oracle than the same record with plain TF32 products, and within 2e-5 in rel-L2 (fp32
    accumulation of up to 1024 terms plus the dropped second-order term); under a split-K cluster too."""
    a = W.make_inputs(spec, 91)
    ref = util.oracle_ref(spec, a)
    for kw in (dict(tile_n=64, tile_k=32, stages=3, mma_m_axis=1), dict(tile_n=128, tile_k=64, stages=2, split_k=2, mma_m_axis=2)):
        y0 = run_spec(spec, tc(**kw), a, ref)
        y3 = run_spec(spec, tc(precision=1, **kw), a, ref)
        e0, e3 = util.rel_l2(y0, ref), util.rel_l2(y3, ref)
        assert e3 <= 2e-5 and e3 * 20 <= e0, (spec.name, kw, e0, e3)
