"""Run one kernel under one schedule record a few times and print its device time.

A small command-line front end for looking at a single (kernel, record) pair, e.g. under a profiler:

    python -m paper_2201_05587_b200.run_case dense --m 4096 --kk 4096 --nn 4096 --tile-n 256 --tile-k 32 --stages 4
    python -m paper_2201_05587_b200.run_case conv --n 32 --c 64 --hw 56 --k 64 --r 3 --pad 1 --tile-n 64
    python -m paper_2201_05587_b200.run_case dw --n 64 --c 144 --hw 56
    python -m paper_2201_05587_b200.run_case softmax --batch 768 --m 128 --nn 128

Record fields that are not given keep the family's default record.  `--tune LEVEL` replaces the record by the best
one of the native grid tuner first.
"""
from __future__ import annotations

import argparse
import sys

from . import binding as B
from . import workloads as W

ACTS = {"none": B.TT_ACT_NONE, "relu": B.TT_ACT_RELU, "relu6": B.TT_ACT_RELU6, "gelu": B.TT_ACT_GELU_ERF}
RECORD_FIELDS = ("tile_m", "tile_n", "tile_k", "stages", "split_k", "raster", "block_x", "block_y",
                 "items_per_thread", "vec_width", "threads", "unroll", "mma_m_axis", "slab_tiles", "acc_split", "k_order",
                 "persistent", "cta_group", "ctas_per_sm", "precision")


def build_spec(a) -> W.Spec:
    act = ACTS[a.act]
    if a.op == "conv":
        return W.Spec(B.TT_OP_CONV2D, B.conv2d_shapes(a.n, a.c, a.hw, a.hw, a.k, a.r, a.r, a.stride, a.pad, True, act), 1,
                      f"conv{a.r}x{a.r}s{a.stride}_n{a.n}_{a.c}x{a.hw}->{a.k}")
    if a.op == "dw":
        s = B.make_shapes(n=a.n, c=a.c, h=a.hw, w=a.hw, k=a.c, r=a.r, s=a.r, stride_h=a.stride, stride_w=a.stride,
                          pad_h=a.r // 2, pad_w=a.r // 2, has_bias=1, act=act)
        return W.Spec(B.TT_OP_DWCONV2D, s, 1, f"dw{a.r}x{a.r}s{a.stride}_n{a.n}_{a.c}x{a.hw}")
    if a.op == "dense":
        return W.Spec(B.TT_OP_DENSE, B.dense_shapes(a.m, a.nn, a.kk, True, act), 1, f"dense_{a.m}x{a.kk}->{a.nn}")
    if a.op == "bmm":
        return W.Spec(B.TT_OP_BATCH_MATMUL, B.bmm_shapes(a.batch, a.m, a.nn, a.kk, bool(a.trans_b)), 1, "bmm", "bert")
    return W.Spec(B.TT_OP_SOFTMAX, B.softmax_shapes(a.batch, a.m, a.nn, a.scale), 1, "softmax", "bert")


def main(argv=None) -> int:
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("op", choices=["conv", "dw", "dense", "bmm", "softmax"])
    for name, default in (("n", 1), ("c", 64), ("hw", 56), ("k", 64), ("r", 3), ("stride", 1), ("pad", 1),
                          ("batch", 12), ("m", 128), ("nn", 128), ("kk", 64), ("trans_b", 1)):
        ap.add_argument(f"--{name.replace('_', '-')}", type=int, default=default)
    ap.add_argument("--scale", type=float, default=0.125)
    ap.add_argument("--act", choices=sorted(ACTS), default="none")
    for f in RECORD_FIELDS:
        ap.add_argument(f"--{f.replace('_', '-')}", type=int, default=None)
    ap.add_argument("--tune", type=int, default=-1, help="grid-tune at this level first and use the best record")
    ap.add_argument("--iters", type=int, default=3, help="plain launches after the timed batches")
    ap.add_argument("--seed", type=int, default=7)
    ap.add_argument("--no-graph", action="store_true", help="time plain stream launches instead of graph replays")
    ap.add_argument("--constant-weights", action="store_true", help="promise that w and bias are constants (fetched early)")
    a = ap.parse_args(argv)

    import torch
    if not torch.cuda.is_available():
        raise SystemExit("run_case needs a CUDA device: there is no CPU fallback")
    spec = build_spec(a)
    wl = spec.workload()
    arrays = W.make_inputs(spec, a.seed)
    t, tt = W.device_tensors(spec, arrays)
    rec = wl.default_schedule()
    for f in RECORD_FIELDS:
        v = getattr(a, f)
        if v is not None:
            setattr(rec, f, v)
    if a.tune >= 0:
        best, tried = wl.grid_tune(tt, None, level=a.tune, top_k=1)
        rec = best[0][0]
        print(f"grid tuner tried {tried} records")
    info = wl.apply(rec)
    wl.set_constant_weights(a.constant_weights)
    topts = B.tt_timing_opts()
    topts.use_graph = 0 if a.no_graph else 1            # batches replayed as CUDA graphs: no CPU launch gaps
    tm = wl.time(tt, topts)
    v = wl.gemm_view()
    print(f"{spec.name} {info.legal.short()} grid ({info.grid_x},{info.grid_y},{info.grid_z}) x {info.threads} threads, "
          f"smem {info.smem_bytes} B: median {tm.median_us:.2f} us, {v.flops / tm.median_us / 1e6:.1f} TFLOP/s, "
          f"{v.bytes / tm.median_us / 1e3:.1f} GB/s (algorithmic: {v.flops / 1e9:.3f} GFLOP, {v.bytes / 1e6:.2f} MB)")
    for _ in range(a.iters):
        wl.run(tt)
    torch.cuda.synchronize()
    st = wl.status()
    wl.close()
    if st != B.TT_OK:
        print(f"device status: {B.status_string(st)}")
        return 1
    return 0


if __name__ == "__main__":
    sys.exit(main())
