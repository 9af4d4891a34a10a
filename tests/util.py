"""Shared test helpers: oracle reference for a workload spec, tolerances."""
import numpy as np

from oracle import oracle as orc
from paper_2201_05587_b200 import binding as B

TOL_TF32 = 2e-3     # tensor-core TF32 paths (conv2d, dense, batch_matmul)
TOL_FP32 = 1e-5     # SIMT fp32 paths (depthwise, softmax)


def tolerance(op):
    return TOL_FP32 if op in (B.TT_OP_DWCONV2D, B.TT_OP_SOFTMAX) else TOL_TF32


def oracle_ref(spec, a, mode=orc.MODE_EXACT, threads=0):
    s = spec.shapes
    if spec.op == B.TT_OP_CONV2D:
        return orc.conv2d(a["x"], a["w"], a["bias"], (s.stride_h, s.stride_w), (s.pad_h, s.pad_w), s.act,
                          a.get("residual"), mode=mode, threads=threads)
    if spec.op == B.TT_OP_DWCONV2D:
        return orc.dwconv2d(a["x"], a["w"], a["bias"], (s.stride_h, s.stride_w), (s.pad_h, s.pad_w), s.act,
                            threads=threads)
    if spec.op == B.TT_OP_DENSE:
        return orc.dense(a["x"], a["w"], a["bias"], s.act, mode=mode, threads=threads)
    if spec.op == B.TT_OP_BATCH_MATMUL:
        return orc.batch_matmul(a["x"], a["w"], None, bool(s.trans_b), s.act, mode=mode, threads=threads)
    return orc.softmax(a["x"], s.scale, threads=threads)


def rel_l2(y, ref):
    return orc.rel_l2(y, ref)
