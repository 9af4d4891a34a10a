"""Host logic of the library (no GPU): ABI exports, workloads, classes, legaliser/validator, selector."""
import ctypes
import os
import re

import numpy as np
import pytest

from oracle import oracle as orc
from paper_2201_05587_b200 import binding as B
from paper_2201_05587_b200 import workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
GOLDEN = os.path.join(ROOT, "tests", "golden")


def test_library_exports_every_declared_symbol():
    text = open(os.path.join(ROOT, "include", "tt.h")).read()
    declared = set(re.findall(r"\b(tt_[a-z_]+)\s*\(", text))
    declared -= {"tt_op", "tt_act"}
    assert declared, "no declarations found"
    lib = B.lib()
    for name in sorted(declared):
        assert hasattr(lib, name), f"{name} declared in tt.h but not exported"
        assert name in B.EXPORTS, f"{name} has no binding"
    assert set(B.EXPORTS) <= declared


def test_struct_sizes_match_header_layout():
    assert ctypes.sizeof(B.tt_shapes) == 20 * 4
    assert ctypes.sizeof(B.tt_schedule_record) == 3 * 4 + 80 + 21 * 4
    assert B.status_string(B.TT_ERR_INVALID_SCHEDULE) != B.status_string(B.TT_OK)


def test_split_check_matches_paper_examples_and_oracle():
    with open(os.path.join(GOLDEN, "split_validity.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            extent, form, factors, valid = line.split()
            extent, valid = int(extent), bool(int(valid))
            fs = [int(v) for v in factors.split(",")]
            if form == "fixed":
                assert B.split_check(extent, fs) == valid == orc.split_covers(extent, fs), line
            elif form == "reform":
                assert B.split_check(extent, fs, reformulate=True) == valid, line
    for n in (1, 7, 8, 24, 49, 196, 1000, 4096):
        for f in (1, 2, 3, 8, 16):
            assert B.split_check(n, [f], True) == orc.split_reformulated_valid(n, f)
            assert B.split_check(n, [n // f if n % f == 0 else 1, f]) == orc.split_covers(n, [n // f if n % f == 0 else 1, f])


def test_select_matches_oracle_on_hand_tables():
    t = [5.0, 3.0, -1.0, 3.0, -1.0, -1.0, -1.0, -1.0, 2.0, -1.0, 1.5, 9.0, float("nan"), 4.0, 4.0, -1.0]
    assert B.select(t, 4, 4) == orc.select(t, 4, 4) == [1, -1, 2, 1]
    lat = B.model_latency(t, 4, 4, [1, -1, 2, 1], [2, 5, 3, 1])
    assert lat == pytest.approx(orc.model_latency([2, 5, 3, 1], [0 if v != v else v for v in t], [1, -1, 2, 1], 4))
    # deterministic: same table, same answer
    assert all(B.select(t, 4, 4) == [1, -1, 2, 1] for _ in range(5))


def test_resnet18_inventory_matches_table1():
    rows = []
    with open(os.path.join(GOLDEN, "resnet18_table1.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                i, cls, ic, ihw, oc, ohw, use = line.split()
                rows.append((cls, int(ic), int(ihw), int(oc), int(ohw), int(use)))
    specs = W.resnet18()
    assert len(specs) == 16                               # A 3, E 8, F 4, D 1
    want = {(cls, ic, ihw, oc, ohw): use for cls, ic, ihw, oc, ohw, use in rows}
    got = {}
    for sp in specs:
        s = sp.shapes
        if sp.op == B.TT_OP_DENSE:
            got[("D", s.kk, 1, s.nn, 1)] = sp.use_count
        else:
            p = (s.h + 2 * s.pad_h - s.r) // s.stride_h + 1
            kind = "A" if (s.r == 1 and s.act == B.TT_ACT_NONE) else ("F" if s.has_residual else "E")
            got[(kind, s.c, s.h, s.k, p)] = sp.use_count
    assert got == want
    assert sum(sp.use_count for sp in specs) == 21          # 20 convolutions + 1 dense
    # the residual variants are kernels of their own class and workload ID, although they share their sibling's sizes
    e = [sp for sp in specs if sp.shapes.c == 64 and sp.shapes.k == 64 and sp.shapes.r == 3]
    assert len(e) == 2 and e[0].workload().kernel_class() != e[1].workload().kernel_class()
    assert e[0].workload().key() != e[1].workload().key()


def test_chains_are_consistent_with_their_inventories():
    """A model is written once as wired layers; the inventory is derived from it.  Every wire connects buffers of the
    same element count, every skip tensor has the consumer's output shape, and the use counts are the layer counts."""
    for name, make in W.CHAINS.items():
        specs, steps = make()
        assert [sp.use_count for sp in specs] == [sum(1 for st in steps if st.kernel == i) for i in range(len(specs))], name
        for i, st in enumerate(steps):
            if st.spec is None:
                assert st.shape and st.note, (name, i)
                continue
            xs, ws, bs, rs, ys = W.tensor_shapes(st.spec)
            assert bytes(specs[st.kernel].shapes) == bytes(st.spec.shapes)
            assert 0 <= st.x < i and np.prod(steps[st.x].out_shape()) == np.prod(xs), (name, i)
            if st.w_from is not None:
                assert 0 <= st.w_from < i and np.prod(steps[st.w_from].out_shape()) == np.prod(ws), (name, i)
            assert (st.res is not None) == bool(st.spec.shapes.has_residual), (name, i)
            if st.res is not None:
                assert 0 <= st.res < i and steps[st.res].out_shape() == tuple(ys), (name, i)
    # the ResNet-18-shaped chain: a block's second convolution adds the block's input, or its 1x1 downsample
    specs, steps = W.resnet18_net()
    f = [st for st in steps if st.spec is not None and st.spec.shapes.has_residual]
    assert len(f) == 8 and sum(1 for st in f if steps[st.res].spec is not None and steps[st.res].spec.shapes.r == 1) == 3


def test_unique_kernel_counts_of_table2():
    """Table 2: ResNet50 A4 E16 G4 D1; VGG-16 E9 (+ 3 dense shapes); MobileNetV2 A7+K5 J8 L10 D1; BERT Q3 R2."""
    r50 = W.resnet50()
    convs = [s for s in r50 if s.op == B.TT_OP_CONV2D]
    down = [s for s in convs if s.shapes.act == B.TT_ACT_NONE]
    g = [s for s in convs if s.shapes.has_residual]
    assert len(down) == 4 and len(g) == 4 and len(convs) - len(down) - len(g) == 16 and len(r50) == 25    # A, G, E
    vgg = W.vgg16()
    assert len([s for s in vgg if s.op == B.TT_OP_CONV2D]) == 9 and len(vgg) == 12
    mb = W.mobilenet_v2()
    dw = [s for s in mb if s.op == B.TT_OP_DWCONV2D]
    proj = [s for s in mb if s.op == B.TT_OP_CONV2D and s.shapes.act == B.TT_ACT_NONE]
    relu6 = [s for s in mb if s.op == B.TT_OP_CONV2D and s.shapes.act == B.TT_ACT_RELU6]
    assert (len(dw), len(proj), len(relu6)) == (10, 12, 8)
    assert len([s for s in proj if s.shapes.has_residual]) == 5                 # class K; the other 7 are class A
    bert = W.bert_base()
    assert len([s for s in bert if s.op == B.TT_OP_DENSE]) == 3
    assert len([s for s in bert if s.op == B.TT_OP_BATCH_MATMUL]) == 2


def test_workload_key_and_class():
    a = W._conv(64, 56, 64, 3, 1, 1).workload()
    b = W._conv(64, 56, 64, 3, 1, 1).workload()
    c = W._conv(128, 28, 128, 3, 1, 1).workload()
    d = W._conv(64, 56, 128, 1, 2, 0, act=B.TT_ACT_NONE).workload()
    e = W._dense(1, 512, 1000).workload()
    assert a.key() == b.key() != c.key()
    assert a.kernel_class() == c.kernel_class()          # same operators, other sizes: same class
    assert a.kernel_class() != d.kernel_class()          # conv2d_add is another class than conv2d_bias_relu
    assert a.kernel_class() != e.kernel_class()
    assert a.family() == e.family() == B.TT_FAMILY_GEMM_TC
    v = a.gemm_view()
    assert (v.batch, v.gm, v.gn, v.gk) == (1, 64, 3136, 576)
    assert v.flops == pytest.approx(2 * 64 * 3136 * 576)


def test_workload_create_rejects_bad_shapes():
    for bad in (B.conv2d_shapes(1, 0, 8, 8, 4, 3, 3), B.conv2d_shapes(1, 4, 2, 2, 4, 5, 5), B.conv2d_shapes(1, 4, 8, 8, 4, 3, 3, 0)):
        h = ctypes.c_void_p()
        assert B.lib().tt_workload_create(B.TT_OP_CONV2D, ctypes.byref(bad), ctypes.byref(h)) == B.TT_ERR_INVALID_ARG
    h = ctypes.c_void_p()
    assert B.lib().tt_workload_create(99, ctypes.byref(B.dense_shapes(1, 2, 3)), ctypes.byref(h)) == B.TT_ERR_INVALID_ARG


def test_cross_family_and_cross_class_records_are_invalid():
    conv = W._conv(64, 56, 64, 3, 1, 1).workload()
    dw = W._dw(32, 112, 1).workload()
    dense = W._dense(1, 512, 1000).workload()
    st, _ = dw.check(conv.default_schedule())
    assert st == B.TT_ERR_CLASS_MISMATCH
    st, _ = conv.check(dw.default_schedule())
    assert st == B.TT_ERR_CLASS_MISMATCH
    # the paper's rule: a conv schedule on a dense kernel is always invalid
    rec = conv.default_schedule()
    st, _ = dense.check(rec, strict_class=True)
    assert st == B.TT_ERR_CLASS_MISMATCH
    # with family matching (the stated extension) the same record applies
    st, _ = dense.check(rec, strict_class=False)
    assert st == B.TT_OK
    # same class, other sizes: valid in both
    other = W._conv(256, 14, 256, 3, 1, 1).workload()
    assert other.check(rec, strict_class=True)[0] == B.TT_OK


def test_legaliser_clamps_and_strict_mode_rejects():
    wl = W.single_conv()[0].workload()         # GEMM view 32 x 196 x 144
    for rec in W.single_conv_pool():
        st, info = wl.check(rec)
        assert st == B.TT_OK
        L = info.legal
        assert L.tile_m == 128 and L.tile_n % 16 == 0 and L.tile_k in (8, 16)
        assert info.changed & B.TT_CHG_TILE_M
    big = B.make_record(B.TT_FAMILY_GEMM_TC, tile_n=256, tile_k=64, stages=2, split_k=64, mma_m_axis=1)
    st, info = wl.check(big)
    assert st == B.TT_OK
    assert info.legal.tile_n == 208 and info.legal.split_k == 3 and info.changed & B.TT_CHG_SPLIT_K
    # strict: a factor larger than the loop, or more splits than reduction tiles, is invalid code
    assert wl.check(big, mode=B.TT_MODE_STRICT)[0] == B.TT_ERR_INVALID_SCHEDULE
    ok = B.make_record(B.TT_FAMILY_GEMM_TC, tile_m=32, tile_n=64, tile_k=16, stages=2, split_k=3, mma_m_axis=1)
    assert wl.check(ok, mode=B.TT_MODE_STRICT)[0] == B.TT_OK
    # resources: 8 stages of 128x256x128 do not fit shared memory
    fat = B.make_record(B.TT_FAMILY_GEMM_TC, tile_n=256, tile_k=128, stages=8, mma_m_axis=1)
    huge = W._dense(512, 4096, 4096).workload()
    # reformulated: the pipeline is made shallower until it fits (one 192 KB stage); kept as written it is invalid
    st, info = huge.check(fat)
    assert st == B.TT_OK and info.legal.stages == 1 and info.changed & B.TT_CHG_STAGES
    st, info = huge.check(fat, mode=B.TT_MODE_STRICT)
    assert st == B.TT_ERR_RESOURCE and info.smem_bytes > 227 * 1024
    # a 128-pixel x 128-channel tile of a strided 1x1 convolution: its input slab alone exceeds shared memory at any depth
    wide = W._conv(256, 56, 512, 1, 2, 0).workload()
    st, info = wide.check(B.make_record(B.TT_FAMILY_GEMM_TC, tile_n=32, tile_k=128, stages=2, mma_m_axis=2))
    assert st == B.TT_ERR_RESOURCE and info.smem_bytes > 227 * 1024
    # the slab is part of the record: a request for more reduction tiles per staging than fit is lowered
    conv = W._conv(512, 28, 512, 3, 1, 1).workload()
    st, info = conv.check(B.make_record(B.TT_FAMILY_GEMM_TC, tile_n=128, tile_k=32, stages=3, slab_tiles=64, mma_m_axis=1))
    assert st == B.TT_OK and 1 <= info.legal.slab_tiles < 64 and info.changed & B.TT_CHG_SLAB
    # nonsense fields
    for kw in (dict(tile_n=0), dict(stages=0), dict(split_k=-1), dict(raster=5), dict(mma_m_axis=7)):
        assert wl.check(B.make_record(B.TT_FAMILY_GEMM_TC, **kw))[0] == B.TT_ERR_INVALID_SCHEDULE
    bad = B.make_record(B.TT_FAMILY_GEMM_TC)
    bad.version = 77
    assert wl.check(bad)[0] == B.TT_ERR_INVALID_SCHEDULE


def test_gemm_records_transfer_between_512_and_1024():
    """The GEMM example of Section 4.1: records of the 512^3 and 1024^3 kernels apply to each other unchanged."""
    a, b = W._dense(512, 512, 512).workload(), W._dense(1024, 1024, 1024).workload()
    ra = B.make_record(B.TT_FAMILY_GEMM_TC, tile_n=128, tile_k=32, stages=4, split_k=2, mma_m_axis=1)
    rb = B.make_record(B.TT_FAMILY_GEMM_TC, tile_n=256, tile_k=64, stages=2, split_k=1, raster=1, mma_m_axis=1)
    for wl in (a, b):
        for r in (ra, rb):
            st, info = wl.check(r, mode=B.TT_MODE_STRICT)
            assert st == B.TT_OK and info.changed == 0


def test_simt_legalisers():
    dw = W._dw(96, 7, 1).workload()
    r = B.make_record(B.TT_FAMILY_DW_SIMT, tile_m=2048, block_y=16, block_x=64, items_per_thread=4, vec_width=4, threads=256)
    st, info = dw.check(r)
    assert st == B.TT_OK
    L = info.legal
    assert L.tile_m == 96 and L.block_y == 7 and L.vec_width == 1 and L.block_x % L.items_per_thread == 0
    assert dw.check(r, mode=B.TT_MODE_STRICT)[0] == B.TT_ERR_INVALID_SCHEDULE
    sm = [s for s in W.bert_base() if s.op == B.TT_OP_SOFTMAX][0].workload()
    st, info = sm.check(B.make_record(B.TT_FAMILY_ROW_SIMT, block_x=24, block_y=3, vec_width=4))
    assert st == B.TT_OK and info.legal.block_x == 16 and info.threads % 32 == 0 and info.legal.vec_width == 4


def test_device_calls_fail_loudly_without_gpu():
    import torch
    if torch.cuda.is_available():
        pytest.skip("GPU present")
    wl = W._dense(8, 16, 8).workload()
    st, _ = wl.try_apply(wl.default_schedule())
    assert st == B.TT_ERR_CUDA                      # no CPU fallback
    t = B.tt_tensors()
    assert B.lib().tt_run(wl.handle, ctypes.byref(t), None) == B.TT_ERR_NOT_APPLIED


def test_rank_pools_matches_the_oracle_on_the_papers_tables():
    """tt_rank_pools (Equation 1) against the oracle on Table 2, target by target, and its argument checks."""
    import test_oracle_pins as pins
    feats, choices = pins._load_tables()
    classes = sorted({c for f in feats.values() for c in f})
    for target in feats:
        cands = [m for m in feats if m != target]
        share_d = {c: pct / 100.0 for c, (_, pct) in feats[target].items()}
        counts_d = [{c: n for c, (n, _) in feats[m].items()} for m in cands]
        want_scores, want_order = orc.rank_pools(share_d, counts_d)
        share = [share_d.get(c, 0.0) for c in classes]
        counts = [[cd.get(c, 0) for c in classes] for cd in counts_d]
        scores, order = B.rank_pools(share, counts)
        assert order == want_order
        assert scores == pytest.approx(want_scores, rel=1e-12, abs=1e-15)
        assert [cands[i] for i in order[:len(choices[target])]] == choices[target]
    with pytest.raises(B.TTError):
        B.rank_pools([0.5], [[-1]])


def test_tap_major_reduction_order_is_legalised_per_kernel():
    """k_order = 1 exists for stride-1 convolutions whose image rows are 16-byte multiples; elsewhere the record is
    reformulated to the stored order (legalise) or invalid (strict)."""
    rec = B.make_record(B.TT_FAMILY_GEMM_TC, tile_n=128, tile_k=32, stages=3, k_order=1, mma_m_axis=1)
    st, info = W._conv(64, 28, 64, 3, 1, 1).workload().check(rec)
    assert st == B.TT_OK and info.legal.k_order == 1 and info.launches == 2
    assert info.workspace_bytes == 64 * 2 * 9 * 32 * 4        # re-packed filters: 2 blocks of 32 channels x 9 taps
    assert info.grid_x == (28 * 32 + 127) // 128              # padded-linear pixels: 28 rows of 28 + 4
    for sp in (W._conv(64, 56, 128, 3, 2, 1), W._conv(64, 14, 64, 3, 1, 1), W._dense(128, 768, 768)):
        wl = sp.workload()
        st, info = wl.check(rec)
        assert st == B.TT_OK and info.legal.k_order == 0 and info.changed & B.TT_CHG_KORDER and info.launches == 1
        assert wl.check(rec, mode=B.TT_MODE_STRICT)[0] == B.TT_ERR_INVALID_SCHEDULE
    # the mode fixes tile_k, split_k and the row axis; other values are reformulated
    odd = B.make_record(B.TT_FAMILY_GEMM_TC, tile_n=100, tile_k=64, stages=9, split_k=4, k_order=1, mma_m_axis=2)
    st, info = W._conv(64, 28, 64, 3, 1, 1).workload().check(odd)
    L = info.legal
    assert st == B.TT_OK and (L.tile_n, L.tile_k, L.split_k, L.mma_m_axis, L.k_order) == (112, 32, 1, 1, 1) and L.stages <= 8


# ---- refinement of a transferred record: neighbourhood and greedy descent against the oracle's definitions ----
_FAMILY_NAME = {B.TT_FAMILY_GEMM_TC: "gemm_tc", B.TT_FAMILY_DW_SIMT: "dw_simt", B.TT_FAMILY_ROW_SIMT: "row_simt"}


def _rec_key(r):
    return tuple(int(getattr(r, f)) for f in B.tt_schedule_record.FIELDS)


def _legal_neighbours_by_definition(wl, rec):
    """The oracle's raw one-step variations, mapped onto this workload by the validity layer (tt_schedule_check):
    invalid ones, ones that coincide with the legalised start and repeats are dropped, order kept."""
    st, info = wl.check(rec)
    assert st == B.TT_OK
    start = info.legal
    fam = _FAMILY_NAME[int(start.family)]
    out, seen = [], {_rec_key(start)}
    for d in orc.raw_neighbours({f: int(getattr(start, f)) for f in B.tt_schedule_record.FIELDS}, fam):
        r = B.make_record(int(start.family), **d)
        st, info = wl.check(r)
        if st != B.TT_OK or _rec_key(info.legal) in seen:
            continue
        seen.add(_rec_key(info.legal))
        out.append(info.legal)
    return out


def _refine_cases():
    r18 = W.resnet18()
    mb = [s for s in W.mobilenet_v2() if s.op == B.TT_OP_DWCONV2D]
    bert = W.bert_base()
    cases = [(r18[1], B.make_record(B.TT_FAMILY_GEMM_TC, tile_n=64, tile_k=32, stages=3, mma_m_axis=1)),
             (r18[1], B.make_record(B.TT_FAMILY_GEMM_TC, tile_n=256, tile_k=64, stages=4, split_k=8, mma_m_axis=2, k_order=1)),
             (r18[-1], B.make_record(B.TT_FAMILY_GEMM_TC, tile_n=16, tile_k=8, stages=1, split_k=3, mma_m_axis=1)),
             (mb[0], B.make_record(B.TT_FAMILY_DW_SIMT, tile_m=4, block_y=8, block_x=32, items_per_thread=4, vec_width=4, threads=128, unroll=2)),
             (mb[-1], B.make_record(B.TT_FAMILY_DW_SIMT, tile_m=32, block_y=56, block_x=112, items_per_thread=8, vec_width=4, threads=512, unroll=4,
                                    raster=1, stages=4)),
             ([s for s in bert if s.op == B.TT_OP_SOFTMAX][0], B.make_record(B.TT_FAMILY_ROW_SIMT, block_x=8, block_y=4, vec_width=2))]
    return cases


def test_record_neighbours_are_the_legalised_one_step_variations():
    for spec, rec in _refine_cases():
        wl = spec.workload()
        got = wl.neighbours(rec)
        want = _legal_neighbours_by_definition(wl, rec)
        assert [_rec_key(r) for r in got] == [_rec_key(r) for r in want], spec.name
        assert 0 < len(got) <= 18
        _, info = wl.check(rec)
        for r in got:                                    # each differs from the start, and is legal as written
            assert _rec_key(r) != _rec_key(info.legal)
            st, i2 = wl.check(r)
            assert st == B.TT_OK and _rec_key(i2.legal) == _rec_key(r)
        wl.close()


def test_refine_with_follows_the_oracles_descent_on_synthetic_times():
    import math
    for spec, rec in _refine_cases():
        wl = spec.workload()
        # a deterministic, bumpy "time" per record: separable bowls plus a hash term, some records unable to run
        def cost(key):
            h = (hash(key) % 1000) / 1000.0
            if int(h * 1000) % 7 == 0:
                return -1.0
            return float(np.float32(50.0 + sum(abs(math.log2(v + 1) - 3.0) * (i % 3 + 1) for i, v in enumerate(key)) + 3.0 * h))
        _, info = wl.check(rec)
        start_key = _rec_key(info.legal)
        if cost(start_key) < 0:
            wl.close()
            continue
        by_key = {}
        def nb(key):
            r = by_key.get(key) or info.legal
            out = _legal_neighbours_by_definition(wl, r)
            for x in out:
                by_key[_rec_key(x)] = x
            return [_rec_key(x) for x in out]
        by_key[start_key] = info.legal
        for rounds, gain in ((0, 0.0), (1, 0.0), (6, 0.0), (6, 0.03)):
            want = orc.refine(start_key, nb, cost, rounds, gain)
            best, best_us, start_us, timed = wl.refine_with(rec, lambda r: cost(_rec_key(r)), rounds, gain)
            assert _rec_key(best) == want[0], (spec.name, rounds, gain)
            assert best_us == pytest.approx(want[1]) and start_us == pytest.approx(want[2]) and timed == want[3]
        wl.close()


def test_refine_rejects_bad_arguments_and_needs_a_device_for_device_times():
    spec, rec = _refine_cases()[0]
    wl = spec.workload()
    other = B.make_record(B.TT_FAMILY_ROW_SIMT, block_x=8, block_y=4, vec_width=2)
    with pytest.raises(B.TTError):
        wl.neighbours(other)                             # a record of another family
    with pytest.raises(B.TTError):
        wl.refine_with(rec, lambda r: -1.0, 3, 0.0)      # the start itself cannot run
    with pytest.raises(B.TTError):
        wl.refine_with(rec, lambda r: 1.0, -1, 0.0)
    import torch
    if not torch.cuda.is_available():
        t, best, us = B.tt_tensors(), B.tt_schedule_record(), ctypes.c_float()
        assert B.lib().tt_refine(wl.handle, ctypes.byref(t), None, None, ctypes.byref(rec), 2, 0.0, ctypes.byref(best),
                                 ctypes.byref(us), None, None) == B.TT_ERR_CUDA      # no CPU fallback
    wl.close()


def test_depthwise_tma_records_are_legalised_by_shape():
    """raster = 1 names the TMA-staged persistent depthwise kernel: kept where image rows are 16-byte multiples and the
    filter is one the window kernels cover, with 2..4 staging buffers that fit shared memory; legalised away elsewhere
    (strict mode: invalid)."""
    rec = B.make_record(B.TT_FAMILY_DW_SIMT, tile_m=8, block_y=14, block_x=56, items_per_thread=4, vec_width=4, threads=256,
                        unroll=2, raster=1, stages=3)
    ok = W._dw(144, 56, 1).workload()                     # 56-pixel rows: 224 bytes
    st, info = ok.check(rec)
    assert st == B.TT_OK and info.legal.raster == 1 and info.legal.stages == 3 and info.grid_y == 1
    assert 0 < info.smem_bytes <= 227 * 1024 and info.grid_x <= 148 * 8
    assert ok.check(rec, mode=B.TT_MODE_STRICT)[0] == B.TT_OK
    deep = B.make_record(B.TT_FAMILY_DW_SIMT, tile_m=8, block_y=14, block_x=56, items_per_thread=4, vec_width=4, threads=256,
                         unroll=2, raster=1, stages=9)
    st, info = ok.check(deep)
    assert st == B.TT_OK and info.legal.raster == 1 and info.legal.stages == 4 and info.changed & B.TT_CHG_STAGES
    assert ok.check(deep, mode=B.TT_MODE_STRICT)[0] == B.TT_ERR_INVALID_SCHEDULE
    odd = W._dw(96, 14, 1).workload()                     # 14-pixel rows: 56 bytes, no aligned TMA rows
    st, info = odd.check(rec)
    assert st == B.TT_OK and info.legal.raster == 0 and info.changed & B.TT_CHG_BLOCK
    assert odd.check(rec, mode=B.TT_MODE_STRICT)[0] == B.TT_ERR_INVALID_SCHEDULE
    staged = B.make_record(B.TT_FAMILY_DW_SIMT, tile_m=8, block_y=8, block_x=32, items_per_thread=4, vec_width=4, threads=256,
                           unroll=0, raster=1, stages=2)  # unroll 0 asks for the staged kernel: no TMA form of it
    st, info = ok.check(staged)
    assert st == B.TT_OK and info.legal.raster == 0
    bad = B.make_record(B.TT_FAMILY_DW_SIMT, tile_m=8, block_y=8, block_x=32, items_per_thread=4, vec_width=4, threads=256,
                        unroll=2, raster=2, stages=2)
    assert ok.check(bad)[0] == B.TT_ERR_INVALID_SCHEDULE
    for w in (ok, odd):
        w.close()


def test_pointwise_convolutions_take_the_whole_row_view():
    """A 1x1, stride-1, unpadded convolution is legalised on rows that tile the CTA's pixels exactly: less shared
    memory than the same record needs on a 3x3 layer's slab geometry would suggest, and never more than the image-row
    view of a layer whose pixel count has no suitable divisor."""
    rec = B.make_record(B.TT_FAMILY_GEMM_TC, tile_n=64, tile_k=32, stages=2, mma_m_axis=2, slab_tiles=1)
    pw = W._conv(256, 56, 64, 1, 1, 0).workload()         # 3136 pixels = 49 rows of 64
    st, info = pw.check(rec)
    assert st == B.TT_OK and info.smem_bytes <= 90 * 1024
    strided = W._conv(256, 56, 64, 1, 2, 0).workload()    # stride 2: the image's own rows
    st2, info2 = strided.check(rec)
    assert st2 == B.TT_OK
    v = pw.gemm_view()
    assert (v.gm, v.gn, v.gk) == (64, 3136, 256)          # the view changes nothing the caller sees
    for w in (pw, strided):
        w.close()


def test_depthwise_record_naming_a_kernel_form_the_shape_lacks_is_a_reformulation():
    """A register-window (unroll >= 1) or TMA-staged (raster = 1) depthwise record on a filter that has no such kernel
    runs the staged kernel instead: legalise mode says so in `changed`, strict mode rejects the record (a primitive
    that does not fit the loop nest is invalid code, Sections 4.1 and 4.2)."""
    dw7 = B.Workload(B.TT_OP_DWCONV2D, B.make_shapes(n=1, c=8, h=20, w=20, k=8, r=7, s=7, stride_h=1, stride_w=1, pad_h=3,
                                                     pad_w=3, has_bias=1, act=B.TT_ACT_RELU), "dw7x7")
    dw3s3 = B.Workload(B.TT_OP_DWCONV2D, B.make_shapes(n=1, c=8, h=20, w=20, k=8, r=3, s=3, stride_h=3, stride_w=3, pad_h=1,
                                                       pad_w=1, has_bias=1, act=B.TT_ACT_RELU), "dw3x3s3")
    dw3 = B.Workload(B.TT_OP_DWCONV2D, B.make_shapes(n=1, c=8, h=20, w=20, k=8, r=3, s=3, stride_h=1, stride_w=1, pad_h=1,
                                                     pad_w=1, has_bias=1, act=B.TT_ACT_RELU), "dw3x3")
    win = B.make_record(B.TT_FAMILY_DW_SIMT, tile_m=4, block_y=4, block_x=20, items_per_thread=4, vec_width=4, threads=128, unroll=2)
    for wl in (dw7, dw3s3):
        st, info = wl.check(win)
        assert st == B.TT_OK and info.legal.unroll == 0 and info.changed & B.TT_CHG_FORM
        assert wl.check(win, mode=B.TT_MODE_STRICT)[0] == B.TT_ERR_INVALID_SCHEDULE
    st, info = dw3.check(win)
    assert st == B.TT_OK and info.legal.unroll == 2 and not info.changed & B.TT_CHG_FORM
    assert dw3.check(win, mode=B.TT_MODE_STRICT)[0] == B.TT_OK
    three = B.make_record(B.TT_FAMILY_DW_SIMT, tile_m=4, block_y=4, block_x=20, items_per_thread=4, vec_width=4, threads=128, unroll=3)
    st, info = dw3.check(three)
    assert st == B.TT_OK and info.legal.unroll == 2 and info.changed & B.TT_CHG_FORM
    assert dw3.check(three, mode=B.TT_MODE_STRICT)[0] == B.TT_ERR_INVALID_SCHEDULE
    tma = B.make_record(B.TT_FAMILY_DW_SIMT, tile_m=4, block_y=4, block_x=20, items_per_thread=4, vec_width=4, threads=256,
                        unroll=2, raster=1, stages=2)
    st, info = dw7.check(tma)
    assert st == B.TT_OK and info.legal.raster == 0 and info.changed & B.TT_CHG_FORM
    assert dw3.check(tma)[1].legal.raster == 1


def test_pool_file_round_trip_and_rejections(tmp_path):
    """Schedules persist as records keyed by the kernel they were tuned on (Section 2): a pool written as text reads
    back bit for bit; a damaged line, an unknown field or another record version is refused, not guessed at."""
    recs = W.single_conv_pool()
    recs[2].origin.scale = 0.125
    recs.append(B.make_record(B.TT_FAMILY_DW_SIMT, tile_m=8, block_y=14, block_x=28, items_per_thread=4, vec_width=4, threads=256,
                              unroll=2, raster=1, stages=2))
    path = str(tmp_path / "pool.txt")
    B.pool_save(path, recs, [1.5, 2.25, -1.0, 7.0, 40.5])
    back, us = B.pool_load(path)
    assert us == [1.5, 2.25, -1.0, 7.0, 40.5]
    assert [bytes(r) for r in back] == [bytes(r) for r in recs]
    B.pool_save(path, [], None)
    assert B.pool_load(path) == ([], [])
    good = open(str(tmp_path / "pool.txt")).read()
    B.pool_save(path, recs[:1], None)
    line = [l for l in open(path).read().splitlines() if not l.startswith("#")][0]
    assert "us=-1" in line
    for bad in (line.replace("tile_n=", "tile_q="), line.replace("version=3", "version=99"), line.replace("stages=2", "stages=two"),
                line.replace("origin=1,", "origin=1;")):
        with open(path, "w") as f:
            f.write(bad + "\n")
        n = ctypes.c_size_t()
        assert B.lib().tt_pool_load(path.encode(), None, None, 0, ctypes.byref(n)) == B.TT_ERR_INVALID_ARG, bad
    n = ctypes.c_size_t()
    assert B.lib().tt_pool_load(str(tmp_path / "missing.txt").encode(), None, None, 0, ctypes.byref(n)) == B.TT_ERR_INVALID_ARG
    del good


def test_bench_counts_algorithmic_work_like_the_library():
    """bench.py's reference arm counts flops and bytes from the shapes alone; they are the library's gemm view."""
    import bench
    for model in ("resnet18", "mobilenet_v2", "bert_base"):
        for sp in W.MODELS[model]():
            v = sp.workload().gemm_view()
            f, b = bench.algorithmic_work(sp)
            assert f == pytest.approx(v.flops) and b == pytest.approx(v.bytes), sp.name


def test_pool_subsample_matches_the_oracle():
    for n, c, seed in ((1, 1, 0), (10, 4, 7), (56, 14, 2024), (111, 111, 5), (50, 0, 9)):
        assert B.pool_subsample(n, c, seed) == orc.pool_subsample(n, c, seed)
    out = (ctypes.c_int32 * 4)()
    assert B.lib().tt_pool_subsample(3, 4, 0, out) == B.TT_ERR_INVALID_ARG


@pytest.mark.parametrize("model", ["resnet18", "resnet50", "mobilenet_v2", "bert_base"])
def test_chain_lanes_order_every_dependency(model):
    """The side-by-side plan of a chain: every producer of a layer (input, skip tensor, second operand, and the layer a
    stand-in tensor replaces) either ran earlier on the layer's own lane or is waited for; kernels declared serial
    never overlap with themselves; the attention projections and the downsample convolutions do leave lane 0."""
    specs, steps = W.CHAINS[model]()
    serial = {0}
    plan = W.chain_lanes(steps, max_lanes=4, serial_kernels=serial)
    assert len(plan) == len(steps)
    seen_on_lane = {}
    last_serial = {}
    for i, (st, pl) in enumerate(zip(steps, plan)):
        assert (pl is None) == (st.spec is None)
        if pl is None:
            continue
        lane, waits = pl
        assert 0 <= lane < 4 and all(w < i and plan[w] is not None for w in waits)
        need = [p for p in (st.x, st.w_from, st.res) if p is not None and steps[p].spec is not None]
        for p in (st.x, st.w_from, st.res):
            if p is not None and p > 0 and steps[p].spec is None:
                need += [q for q in range(p - 1, -1, -1) if steps[q].spec is not None][:1]
        if st.kernel in serial and st.kernel in last_serial:
            need.append(last_serial[st.kernel])
        for p in need:
            assert plan[p][0] == lane or p in waits, (model, i, p)
        seen_on_lane.setdefault(lane, []).append(i)
        last_serial[st.kernel] = i
    lanes_used = len(seen_on_lane)
    assert lanes_used == (1 if model == "mobilenet_v2" else 4)


def test_compensated_precision_is_kept_where_it_exists_and_reported_elsewhere():
    """Record field `precision` = 1 (three TF32 products per step): dense and batch_matmul NT in the one-tile form keep
    it, with twice the shared memory per stage and one accumulator; convolutions, NN products and the persistent form
    legalise it away as a change of form (strict mode: invalid)."""
    rec = B.make_record(B.TT_FAMILY_GEMM_TC, tile_n=64, tile_k=32, stages=2, mma_m_axis=1, precision=1, acc_split=4)
    plain = B.make_record(B.TT_FAMILY_GEMM_TC, tile_n=64, tile_k=32, stages=2, mma_m_axis=1)
    dense = W._dense(256, 512, 384).workload()
    st, info = dense.check(rec)
    st0, info0 = dense.check(plain)
    assert st == B.TT_OK and st0 == B.TT_OK and info.legal.precision == 1 and info.legal.acc_split == 1
    assert info.smem_bytes - 1024 == 2 * (info0.smem_bytes - 1024)
    assert dense.check(rec, mode=B.TT_MODE_STRICT)[0] == B.TT_ERR_INVALID_SCHEDULE       # (acc_split was changed)
    rec.acc_split = 1
    assert dense.check(rec, mode=B.TT_MODE_STRICT)[0] == B.TT_OK
    nt = W.Spec(B.TT_OP_BATCH_MATMUL, B.bmm_shapes(4, 128, 128, 64, True), 1, "nt").workload()
    assert nt.check(rec)[1].legal.precision == 1
    for other in (W._conv(32, 14, 64, 3, 1, 1).workload(), W._conv(64, 28, 64, 1, 1, 0).workload(),
                  W.Spec(B.TT_OP_BATCH_MATMUL, B.bmm_shapes(4, 128, 64, 128, False), 1, "nn").workload()):
        st, info = other.check(rec)
        assert st == B.TT_OK and info.legal.precision == 0 and info.changed & B.TT_CHG_FORM
        assert other.check(rec, mode=B.TT_MODE_STRICT)[0] == B.TT_ERR_INVALID_SCHEDULE
    rec.persistent = 1
    st, info = dense.check(rec)
    assert st == B.TT_OK and info.legal.precision == 1 and info.legal.persistent == 0 and info.changed & B.TT_CHG_FORM
    bad = B.make_record(B.TT_FAMILY_GEMM_TC, precision=2)
    assert dense.check(bad)[0] == B.TT_ERR_INVALID_SCHEDULE
