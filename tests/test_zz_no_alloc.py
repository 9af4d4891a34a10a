"""The dense layer for callers that cannot allocate device memory (tt_dense_static_scratch).

Such callers -- a host whose memory pool already owns the whole device, a loop that may not take the allocator's
lock -- get the split-K scratch from a fixed array inside the library instead of a cudaMalloc'd workspace.  The
result must be the one the allocating path (tt_schedule_apply + tt_run) gives for the same record, and a second
call, which finds the first call's partial sums and counters still in the array, must be just as right.

Collected last on purpose: a failure here cannot hide the other tests' results in a run that stops at the first
failure.
"""
import numpy as np
import pytest

from paper_2201_05587_b200 import binding as B
from paper_2201_05587_b200 import workloads as W
import util

pytestmark = pytest.mark.gpu


def _both_paths(spec, rec, seed):
    import torch
    a = W.make_inputs(spec, seed)
    # existing entry points: the workspace is allocated by tt_schedule_apply
    wl = spec.workload()
    wl.apply(rec)
    t, tt = W.device_tensors(spec, a)
    t["y"].fill_(float("nan"))
    wl.run(tt)
    assert wl.status() == B.TT_OK
    y_alloc = t["y"].cpu().numpy()
    wl.close()
    # the entry point that allocates nothing
    y2 = torch.full_like(t["y"], float("nan"))
    st, used = B.dense_static_scratch(t["x"], t["w"], t["bias"], y2, spec.shapes.act, rec)
    assert st == B.TT_OK, B.status_string(st)
    assert 0 < used <= B.TT_STATIC_SCRATCH_BYTES
    y_static = y2.cpu().numpy()
    assert not np.isnan(y_static).any()
    # same kernel, same fixed reduction order: the two paths agree far inside the TF32 tolerance
    assert util.rel_l2(y_static, y_alloc) <= 1e-6
    assert util.rel_l2(y_static, util.oracle_ref(spec, a)) <= util.TOL_TF32


def test_static_scratch_matches_allocating_path_twice_in_a_row():
    # more than 8 splits, so that the partial sums go through scratch memory (fewer reduce inside a cluster)
    rec = B.make_record(B.TT_FAMILY_GEMM_TC, tile_n=64, tile_k=32, stages=3, split_k=12, mma_m_axis=1)
    _both_paths(W._dense(96, 1500, 200, act=B.TT_ACT_RELU, name="static_a"), rec, seed=41)
    # second call: other sizes and split count, the array still holds the first call's partial sums
    rec2 = B.make_record(B.TT_FAMILY_GEMM_TC, tile_n=128, tile_k=16, stages=2, split_k=11, mma_m_axis=2)
    _both_paths(W._dense(40, 704, 333, act=B.TT_ACT_NONE, name="static_b"), rec2, seed=42)
    # and the first case again, after a differently shaped one
    _both_paths(W._dense(96, 1500, 200, act=B.TT_ACT_RELU, name="static_a"), rec, seed=43)


def test_static_scratch_cluster_split_and_no_allocation_between_calls():
    """Two to eight splits reduce inside a thread-block cluster: the fixed array then only holds the status word and
    the counters.  And the point of the entry point: the device's free memory is the same before and after calls
    (the first call on a device may load the library's image; the later ones must not change anything)."""
    import torch
    rec4 = B.make_record(B.TT_FAMILY_GEMM_TC, tile_n=64, tile_k=32, stages=3, split_k=4, mma_m_axis=1)
    _both_paths(W._dense(96, 1500, 200, act=B.TT_ACT_RELU, name="static_cluster4"), rec4, seed=44)
    spec = W._dense(64, 1024, 256, act=B.TT_ACT_NONE, name="static_free_mem")
    a = W.make_inputs(spec, 45)
    t, _ = W.device_tensors(spec, a)
    y = torch.empty_like(t["y"])
    rec12 = B.make_record(B.TT_FAMILY_GEMM_TC, tile_n=64, tile_k=32, stages=3, split_k=12, mma_m_axis=1)
    assert B.dense_static_scratch(t["x"], t["w"], t["bias"], y, spec.shapes.act, rec12)[0] == B.TT_OK
    torch.cuda.synchronize()
    free0 = torch.cuda.mem_get_info()[0]
    for rec in (rec12, rec4, rec12):
        assert B.dense_static_scratch(t["x"], t["w"], t["bias"], y, spec.shapes.act, rec)[0] == B.TT_OK
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free0
    assert util.rel_l2(y.cpu().numpy(), util.oracle_ref(spec, a)) <= util.TOL_TF32


def test_static_scratch_rejects_what_does_not_fit():
    import torch
    # 2048 x 2048 outputs x 16 splits x 4 bytes = 256 MB of partial sums: far beyond the fixed array
    m = nn = 2048
    kk = 512
    x = torch.zeros(m, kk, device="cuda")
    w = torch.zeros(nn, kk, device="cuda")
    y = torch.zeros(m, nn, device="cuda")
    rec = B.make_record(B.TT_FAMILY_GEMM_TC, tile_n=128, tile_k=32, stages=2, split_k=16, mma_m_axis=1)
    st, used = B.dense_static_scratch(x, w, None, y, B.TT_ACT_NONE, rec)
    assert st == B.TT_ERR_RESOURCE
    assert used > B.TT_STATIC_SCRATCH_BYTES
