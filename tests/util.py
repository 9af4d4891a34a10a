"""Shared test helpers: oracle reference for a workload spec, tolerances."""
import numpy as np

from oracle import oracle as orc
from paper_2201_05587_b200 import binding as B

TOL_TF32 = 2e-3     # tensor-core TF32 paths (conv2d, dense, batch_matmul)
TOL_FP32 = 1e-5     # SIMT fp32 paths (depthwise, softmax)


def tolerance(op):
    return TOL_FP32 if op in (B.TT_OP_DWCONV2D, B.TT_OP_SOFTMAX) else TOL_TF32


def oracle_ref(spec, a, mode=orc.MODE_EXACT, threads=0):
    return orc.reference(spec.op, spec.shapes, a, mode=mode, threads=threads)


def rel_l2(y, ref):
    return orc.rel_l2(y, ref)
