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


def oracle_chain(steps, arrays, mode=orc.MODE_EXACT):
    """The chain on the oracle: every layer computed by the plain definition from the outputs of the nodes it is wired
    to (reshaped where the consumer's shape differs from the producer's).  Returns every node's output."""
    from paper_2201_05587_b200 import workloads as W
    outs = []
    for st, a in zip(steps, arrays):
        if st.spec is None:
            outs.append(a["x"])
            continue
        xs, ws, bs, rs, ys = W.tensor_shapes(st.spec)
        a = dict(a)
        a["x"] = outs[st.x].reshape(xs)
        if st.w_from is not None:
            a["w"] = outs[st.w_from].reshape(ws)
        if st.res is not None:
            a["residual"] = outs[st.res].reshape(rs)
        outs.append(orc.reference(st.spec.op, st.spec.shapes, a, mode=mode))
    return outs
