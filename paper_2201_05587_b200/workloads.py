"""Workload inventories shaped like the paper's models, their data-flow chains, and seeded inputs for them.

The paper evaluates ImageNet CNNs and BERT (Section 5.1); a schedule depends only on
the operator and the data sizes of a kernel (Section 2), never on weight values, so
each model is represented by the list of its unique kernels (operator, sizes, use
count) with synthetic tensors.  No dataset item or trained weight is involved.

Kernel classes follow Tables 1 and 2: conv2d_add (class A: 1x1 downsample or projection,
no activation), conv2d_bias_relu (class E), conv2d_bias_add_relu (classes F and G: the
last convolution of a residual block, skip tensor added before the ReLU),
conv2d_bias_add (class K: MobileNetV2 projection with a skip), depthwise (class L),
dense_add (class D).  A model is written down once, as the ordered list of its layers
with their wiring (which layer's output each layer reads, which one it adds as a
skip); the unique-kernel inventory and its use counts are derived from that list, so
the two always agree.  Pooling, layer normalisation and the reshapes between
attention heads are outside the hot path (about 0 % of inference time, Table 2): where one
would sit the chain reads a seeded tensor of the right shape (pools) or reinterprets
the producer's buffer (head reshapes), and says so in the step.
"""
from __future__ import annotations

import math
from collections import OrderedDict

import numpy as np

from . import binding as B
from . import inputs


class Spec:
    """One unique kernel of a model: operator, sizes, how often the model uses it, and a label."""

    def __init__(self, op, shapes, use_count=1, name="", init="he"):
        self.op, self.shapes, self.use_count, self.name, self.init = op, shapes, use_count, name, init

    def workload(self) -> "B.Workload":
        return B.Workload(self.op, self.shapes, self.name, self.use_count)


def _conv(c, hw, k, r, stride, pad, act=B.TT_ACT_RELU, use=1, name=None, bias=True, residual=False):
    nm = name or f"conv{r}x{r}s{stride}_{c}x{hw}->{k}" + ("+res" if residual else "")
    return Spec(B.TT_OP_CONV2D, B.conv2d_shapes(1, c, hw, hw, k, r, r, stride, pad, bias, act, residual), use, nm)


def _dw(c, hw, stride, r=3, act=B.TT_ACT_RELU6, use=1):
    s = B.make_shapes(n=1, c=c, h=hw, w=hw, k=c, r=r, s=r, stride_h=stride, stride_w=stride, pad_h=r // 2, pad_w=r // 2,
                      has_bias=1, act=act)
    return Spec(B.TT_OP_DWCONV2D, s, use, f"dw{r}x{r}s{stride}_{c}x{hw}")


def _dense(m, kk, nn, act=B.TT_ACT_NONE, use=1, init="he", name=None):
    return Spec(B.TT_OP_DENSE, B.dense_shapes(m, nn, kk, True, act), use, name or f"dense_{m}x{kk}->{nn}", init)


def _dedup(specs):
    """Identical kernels (same workload ID: operator + sizes) are one kernel with a summed use count."""
    seen = OrderedDict()
    for sp in specs:
        key = (sp.op, bytes(sp.shapes))
        if key in seen:
            seen[key].use_count += sp.use_count
        else:
            seen[key] = Spec(sp.op, sp.shapes, sp.use_count, sp.name, sp.init)
    return list(seen.values())


class Step:
    """One node of a model in execution order: a layer (spec is its kernel), or, with spec None, a seeded tensor of
    `shape` that enters the chain from outside the hot path (the model's input, or the stand-in for the output of an
    operator that is not part of it, named in `note`).  x / res / w_from: index of the node whose buffer this layer
    reads as its input / adds as its skip tensor / (batch_matmul) takes as second operand.  A producer's buffer is
    read with the consumer's shape (same number of elements): that is how the head reshapes of the attention block
    are represented."""

    def __init__(self, spec, x=None, res=None, note="", shape=None):
        self.spec, self.x, self.res, self.note, self.shape = spec, x, res, note, shape
        self.w_from = None        # batch_matmul only; None = the layer's own seeded second operand
        self.kernel = -1          # index into the unique-kernel inventory, filled by Net.finish

    def out_shape(self):
        return tuple(self.shape) if self.spec is None else tuple(tensor_shapes(self.spec)[4])


class Net:
    """A model as an ordered list of wired nodes; the inventory of unique kernels is derived from it."""

    def __init__(self):
        self.steps = []

    def external(self, shape, note):
        self.steps.append(Step(None, shape=tuple(shape), note=note))
        return len(self.steps) - 1

    def add(self, spec, x, res=None, note=""):
        self.steps.append(Step(spec, x, res, note))
        return len(self.steps) - 1

    def finish(self):
        specs = _dedup([st.spec for st in self.steps if st.spec is not None])
        index = {(sp.op, bytes(sp.shapes)): i for i, sp in enumerate(specs)}
        for st in self.steps:
            if st.spec is not None:
                st.kernel = index[(st.spec.op, bytes(st.spec.shapes))]
        return specs, self.steps


def single_conv():
    """One conv2d+bias+ReLU: C=16, 14x14, 32 filters 3x3, stride 1, pad 1."""
    return [Spec(B.TT_OP_CONV2D, B.conv2d_shapes(1, 16, 14, 14, 32, 3, 3, 1, 1, True, B.TT_ACT_RELU), 1,
                 "conv3x3s1_16x14->32", init="uniform")]


def single_conv_pool():
    """Four records sized for a C=32, 28x28, K=64 conv: tile M/N/K in {32,64}x{32,64}x{8,16}, 2-3 stages."""
    origin = B.conv2d_shapes(1, 32, 28, 28, 64, 3, 3, 1, 1, True, B.TT_ACT_RELU)
    recs = []
    for tm, tn, tk, st in ((32, 32, 8, 2), (64, 32, 16, 2), (32, 64, 8, 3), (64, 64, 16, 3)):
        r = B.make_record(B.TT_FAMILY_GEMM_TC, tile_m=tm, tile_n=tn, tile_k=tk, stages=st)
        r.origin_op = B.TT_OP_CONV2D
        r.origin = origin
        recs.append(r)
    return recs


def resnet18_net():
    """Table 1: classes A (3 kernels), E (8), F (4), D (1) = 16 unique kernels, 21 uses."""
    net = Net()
    net.add(_conv(3, 224, 64, 7, 2, 3, name="stem7x7s2_3x224->64"), x=net.external((1, 3, 224, 224), "the image"))
    cur = net.external((1, 64, 56, 56), "stands in for the max-pool's output")
    ch, hw = 64, 56
    for stage, k in enumerate((64, 128, 256, 512)):
        for block in range(2):
            if stage > 0 and block == 0:
                c1 = net.add(_conv(ch, hw, k, 3, 2, 1), x=cur)                                   # first 3x3, strided
                skip = net.add(_conv(ch, hw, k, 1, 2, 0, act=B.TT_ACT_NONE), x=cur)               # downsample (class A)
                hw //= 2
            else:
                c1 = net.add(_conv(k, hw, k, 3, 1, 1), x=cur)
                skip = cur
            cur = net.add(_conv(k, hw, k, 3, 1, 1, residual=True), x=c1, res=skip)               # class F
            ch = k
    net.add(_dense(1, 512, 1000), x=net.external((1, 512), "stands in for the global average pool's output"))
    return net.finish()


def resnet50_net():
    """Bottleneck 1x1 / 3x3 / 1x1 kernels (stride on the 3x3; the expanding 1x1 adds the skip: class G), 1x1
    downsamples (class A), the 2048->1000 dense layer.  Table 2: E 16, G 4, A 4, D 1."""
    net = Net()
    net.add(_conv(3, 224, 64, 7, 2, 3, name="stem7x7s2_3x224->64"), x=net.external((1, 3, 224, 224), "the image"))
    cur = net.external((1, 64, 56, 56), "stands in for the max-pool's output")
    in_ch, hw = 64, 56
    for stage, (mid, blocks) in enumerate(((64, 3), (128, 4), (256, 6), (512, 3))):
        out_ch = mid * 4
        stride = 1 if stage == 0 else 2
        for b in range(blocks):
            s = stride if b == 0 else 1
            r1 = net.add(_conv(in_ch, hw, mid, 1, 1, 0), x=cur)                                  # reduce
            m3 = net.add(_conv(mid, hw, mid, 3, s, 1), x=r1)                                     # 3x3
            skip = cur
            if b == 0:
                skip = net.add(_conv(in_ch, hw, out_ch, 1, s, 0, act=B.TT_ACT_NONE), x=cur)      # downsample
            hw2 = hw // s
            cur = net.add(_conv(mid, hw2, out_ch, 1, 1, 0, residual=True), x=m3, res=skip)       # expand + skip
            in_ch, hw = out_ch, hw2
    net.add(_dense(1, 2048, 1000), x=net.external((1, 2048), "stands in for the global average pool's output"))
    return net.finish()


def resnet18():
    return resnet18_net()[0]


def resnet50():
    return resnet50_net()[0]


def vgg16():
    specs = []
    ch, hw = 3, 224
    for k, n in ((64, 2), (128, 2), (256, 3), (512, 3), (512, 3)):
        for _ in range(n):
            specs.append(_conv(ch, hw, k, 3, 1, 1))
            ch = k
        hw //= 2
    specs += [_dense(1, 25088, 4096, B.TT_ACT_RELU), _dense(1, 4096, 4096, B.TT_ACT_RELU), _dense(1, 4096, 1000)]
    return _dedup(specs)


_MBV2 = ((1, 16, 1, 1), (6, 24, 2, 2), (6, 32, 3, 2), (6, 64, 4, 2), (6, 96, 3, 1), (6, 160, 3, 2), (6, 320, 1, 1))


def mobilenet_v2_net():
    """Table 2: J 8 (stem, six expansions, last 1x1: +ReLU6), L 10 (depthwise), A 7 (projection), K 5 (projection that
    adds the block's input), D 1."""
    net = Net()
    cur = net.add(_conv(3, 224, 32, 3, 2, 1, act=B.TT_ACT_RELU6, name="stem3x3s2_3x224->32"),
                  x=net.external((1, 3, 224, 224), "the image"))
    ch, hw = 32, 112
    for t, c, n, s in _MBV2:
        for i in range(n):
            stride = s if i == 0 else 1
            hid = ch * t
            h = cur
            if t != 1:
                h = net.add(_conv(ch, hw, hid, 1, 1, 0, act=B.TT_ACT_RELU6), x=cur)              # expand
            d = net.add(_dw(hid, hw, stride), x=h)
            hw //= stride
            skip = stride == 1 and ch == c
            cur = net.add(_conv(hid, hw, c, 1, 1, 0, act=B.TT_ACT_NONE, residual=skip), x=d, res=cur if skip else None)
            ch = c
    net.add(_conv(320, 7, 1280, 1, 1, 0, act=B.TT_ACT_RELU6), x=cur)
    net.add(_dense(1, 1280, 1000), x=net.external((1, 1280), "stands in for the global average pool's output"))
    return net.finish()


def mobilenet_v2():
    return mobilenet_v2_net()[0]


def efficientnet_b0_like():
    """1x1 expand/project, depthwise 3x3/5x5 and dense shapes of an EfficientNet-B0-shaped network (pool source)."""
    cfg = ((1, 16, 1, 1, 3), (6, 24, 2, 2, 3), (6, 40, 2, 2, 5), (6, 80, 3, 2, 3), (6, 112, 3, 1, 5), (6, 192, 4, 2, 5),
           (6, 320, 1, 1, 3))
    specs = []
    ch, hw = 32, 112
    for t, c, n, s, r in cfg:
        for i in range(n):
            stride = s if i == 0 else 1
            hid = ch * t
            if t != 1:
                specs.append(_conv(ch, hw, hid, 1, 1, 0, act=B.TT_ACT_RELU6))
            specs.append(_dw(hid, hw, stride, r=r))
            hw //= stride
            specs.append(_conv(hid, hw, c, 1, 1, 0, act=B.TT_ACT_NONE))
            ch = c
    specs.append(_conv(320, 7, 1280, 1, 1, 0, act=B.TT_ACT_RELU6))
    specs.append(_dense(1, 1280, 1000))
    return _dedup(specs)


def bert_base_net(seq=128, hidden=768, heads=12, ffn=3072, layers=12):
    """Encoder layers as the hot path sees them: three projections of the layer input, scores, softmax, context,
    output projection, the two feed-forward layers.  The reshapes between [seq, hidden] and [heads, seq, hidden/heads]
    are layout shuffles outside the hot path: a consumer reads the producer's buffer with its own shape.  Layer
    normalisation and the skip additions around it are separate, negligible kernel classes (Table 2: 0 %)."""
    d = hidden // heads
    proj = lambda: _dense(seq, hidden, hidden, init="bert", name=f"dense_{seq}x{hidden}->{hidden}")
    net = Net()
    cur = net.external((seq, hidden), "the embedded tokens")
    for _ in range(layers):
        q = net.add(proj(), x=cur)
        k = net.add(proj(), x=cur)
        v = net.add(proj(), x=cur)
        sc = net.add(Spec(B.TT_OP_BATCH_MATMUL, B.bmm_shapes(heads, seq, seq, d, True), 1, "bmm_qk_nt", "bert"), x=q, res=None,
                     note="w = the key projection's buffer")
        net.steps[sc].w_from = k
        pr = net.add(Spec(B.TT_OP_SOFTMAX, B.softmax_shapes(heads, seq, seq, 1.0 / math.sqrt(d)), 1, "softmax", "bert"), x=sc)
        cx = net.add(Spec(B.TT_OP_BATCH_MATMUL, B.bmm_shapes(heads, seq, d, seq, False), 1, "bmm_pv_nn", "bert"), x=pr,
                     note="w = the value projection's buffer")
        net.steps[cx].w_from = v
        o = net.add(proj(), x=cx)
        f1 = net.add(_dense(seq, hidden, ffn, act=B.TT_ACT_GELU_ERF, init="bert", name=f"dense_gelu_{seq}x{hidden}->{ffn}"), x=o)
        cur = net.add(_dense(seq, ffn, hidden, init="bert", name=f"dense_{seq}x{ffn}->{hidden}"), x=f1)
    return net.finish()


def bert_base(seq=128):
    return bert_base_net(seq=seq)[0]


def bert_base_256():
    """The same encoder on 256 tokens: source or target of the sequence-length transfer of Section 5.4."""
    return bert_base(seq=256)


MODELS = {
    "single_conv": single_conv, "resnet18": resnet18, "resnet50": resnet50, "vgg16": vgg16,
    "mobilenet_v2": mobilenet_v2, "efficientnet_b0_like": efficientnet_b0_like, "bert_base": bert_base,
    "bert_base_256": bert_base_256,
}

# model -> (unique kernels, wired layers in execution order)
CHAINS = {
    "resnet18": resnet18_net, "resnet50": resnet50_net, "mobilenet_v2": mobilenet_v2_net, "bert_base": bert_base_net,
    "bert_base_256": lambda: bert_base_net(seq=256),
}

# target model -> models whose natively tuned records form its schedule pool
POOL_SOURCES = {
    "resnet18": ("resnet50",),
    "resnet50": ("resnet18", "vgg16"),
    "mobilenet_v2": ("resnet50", "efficientnet_b0_like"),
    "bert_base": ("resnet50", "mobilenet_v2"),
    "bert_base_256": ("bert_base",),          # same model, other input size (Section 5.4)
}


def tensor_shapes(spec: Spec):
    """Shapes of (x, w, bias, residual, y) for a spec; None where the tensor does not exist."""
    s = spec.shapes
    if spec.op in (B.TT_OP_CONV2D, B.TT_OP_DWCONV2D):
        p = (s.h + 2 * s.pad_h - s.r) // s.stride_h + 1
        q = (s.w + 2 * s.pad_w - s.s) // s.stride_w + 1
        if spec.op == B.TT_OP_CONV2D:
            wshape, k = (s.k, s.c, s.r, s.s), s.k
        else:
            wshape, k = (s.c, 1, s.r, s.s), s.c
        y = (s.n, k, p, q)
        return (s.n, s.c, s.h, s.w), wshape, (k,) if s.has_bias else None, y if s.has_residual else None, y
    if spec.op == B.TT_OP_DENSE:
        return (s.m, s.kk), (s.nn, s.kk), (s.nn,) if s.has_bias else None, None, (s.m, s.nn)
    if spec.op == B.TT_OP_BATCH_MATMUL:
        wshape = (s.batch, s.nn, s.kk) if s.trans_b else (s.batch, s.kk, s.nn)
        return (s.batch, s.m, s.kk), wshape, None, None, (s.batch, s.m, s.nn)
    return (s.batch, s.m, s.nn), None, None, None, (s.batch, s.m, s.nn)


def make_inputs(spec: Spec, seed: int, index: int = 0):
    """Seeded numpy tensors {x, w, bias, residual} for a spec.

    init "uniform": everything U[-1,1].  "he": activations U[-1,1], weights N(0, 2/fan_in), bias U[-0.1,0.1].
    "bert": activations N(0,1), weights N(0,0.02), bias U[-0.1,0.1]; the batch_matmul operands are N(0,1).
    """
    xs, ws, bs, rs, _ = tensor_shapes(spec)
    tid = index * 8
    out = {"x": None, "w": None, "bias": None, "residual": None}
    if spec.init == "uniform":
        out["x"] = inputs.uniform(xs, seed, tid)
        if ws:
            out["w"] = inputs.uniform(ws, seed, tid + 1)
        if bs:
            out["bias"] = inputs.uniform(bs, seed, tid + 2)
    elif spec.init == "bert":
        out["x"] = inputs.normal(xs, seed, tid)
        if ws:
            std = 1.0 if spec.op == B.TT_OP_BATCH_MATMUL else 0.02
            out["w"] = inputs.normal(ws, seed, tid + 1, std=std)
        if bs:
            out["bias"] = inputs.uniform(bs, seed, tid + 2, -0.1, 0.1)
    else:
        out["x"] = inputs.uniform(xs, seed, tid)
        if ws:
            fan_in = int(np.prod(ws[1:]))
            out["w"] = inputs.normal(ws, seed, tid + 1, std=math.sqrt(2.0 / fan_in))
        if bs:
            out["bias"] = inputs.uniform(bs, seed, tid + 2, -0.1, 0.1)
    if rs:
        out["residual"] = inputs.uniform(rs, seed, tid + 3)
    return out


def device_tensors(spec: Spec, arrays, device="cuda"):
    """Copy the numpy inputs to torch tensors on `device`, allocate y; returns (dict of tensors, tt_tensors)."""
    import torch
    t = {k: (None if v is None else torch.from_numpy(v).to(device)) for k, v in arrays.items()}
    t["y"] = torch.empty(tensor_shapes(spec)[4], dtype=torch.float32, device=device)
    return t, B.tensors(t["x"], t["w"], t["bias"], t["residual"], t["y"])


def make_chain_inputs(steps, seed: int, init="he"):
    """Seeded numpy tensors for every node of a chain: a layer's own weights and bias (and second batch_matmul
    operand where that is not wired), an external node's tensor ("x": U[-1,1], or N(0,1) for init "bert")."""
    out = []
    for i, st in enumerate(steps):
        if st.spec is None:
            x = inputs.normal(st.shape, seed, 8 * (1000 + i)) if init == "bert" else inputs.uniform(st.shape, seed, 8 * (1000 + i))
            out.append({"x": x, "w": None, "bias": None, "residual": None})
            continue
        a = make_inputs(st.spec, seed, 1000 + i)
        a["x"] = None
        if st.w_from is not None:
            a["w"] = None
        a["residual"] = None
        out.append(a)
    return out


def chain_device_tensors(steps, arrays, device="cuda"):
    """Wire a chain on the device: every layer writes its own output buffer, and reads its input, skip tensor and
    (batch_matmul) second operand from the buffers of the nodes that produce them, viewed with its own shapes.
    Returns (per-node dicts of torch tensors, with the node's buffer under "y"; per-node tt_tensors, None for
    external nodes)."""
    import torch
    bufs, tts = [], []
    for st, a in zip(steps, arrays):
        if st.spec is None:
            bufs.append({"y": torch.from_numpy(a["x"]).to(device)})
            tts.append(None)
            continue
        xs, ws, bs, rs, ys = tensor_shapes(st.spec)
        t = {k: (None if v is None else torch.from_numpy(v).to(device)) for k, v in a.items()}
        t["x"] = bufs[st.x]["y"].view(xs)
        if st.w_from is not None:
            t["w"] = bufs[st.w_from]["y"].view(ws)
        if st.res is not None:
            t["residual"] = bufs[st.res]["y"].view(rs)
        t["y"] = torch.empty(ys, dtype=torch.float32, device=device)
        bufs.append(t)
        tts.append(B.tensors(t["x"], t["w"], t["bias"], t["residual"], t["y"]))
    return bufs, tts


def chain_lanes(steps, max_lanes=4, serial_kernels=()):
    """Which layers of a chain may run side by side.  A layer depends only on the nodes it is wired to (x, res, w_from):
    the three projections of an attention block read the same input, a residual block's 1x1 downsample and its first
    3x3 convolution read the same block input.  Returns, per node, None (an external tensor) or (lane, waits): the
    layer is enqueued on stream `lane`, after waiting for the events of the layers in `waits` (its producers on other
    lanes).  A layer follows its input's producer on that producer's lane when it is the first to do so, otherwise it
    takes the lane that has been idle longest.  Kernels in `serial_kernels` (their applied record keeps per-workload
    scratch: a split-K workspace, re-packed filters) never overlap with themselves: each of their layers also waits
    for the previous one.  Every lane's work is ordered, so any assignment is correct; the choice only decides how
    much runs concurrently."""
    lane_of, tail, last_used, plan = {}, [], [], []
    last_of_kernel = {}
    for i, st in enumerate(steps):
        if st.spec is None:
            plan.append(None)
            continue
        prods = [p for p in (st.x, st.w_from, st.res) if p is not None and steps[p].spec is not None]
        for p in (st.x, st.w_from, st.res):
            # a stand-in tensor replaces an operator outside the hot path that the model feeds from the layer in front
            # of it: the dependency stays (the model's own input, node 0, has none)
            if p is not None and p > 0 and steps[p].spec is None:
                prods += [q for q in range(p - 1, -1, -1) if steps[q].spec is not None][:1]
        if st.kernel in serial_kernels and st.kernel in last_of_kernel:
            prods.append(last_of_kernel[st.kernel])
        lane = None
        for p in prods:                                   # continue a producer's lane if nobody has yet
            if tail[lane_of[p]] == p:
                lane = lane_of[p]
                break
        if lane is None:
            lane = len(tail) if len(tail) < max_lanes else min(range(len(tail)), key=lambda l: last_used[l])
        if lane == len(tail):
            tail.append(None)
            last_used.append(-1)
        waits = sorted({p for p in prods if lane_of[p] != lane})
        # work that ran earlier on this lane is ordered before this layer by the stream itself
        lane_of[i], tail[lane], last_used[lane] = lane, i, i
        last_of_kernel[st.kernel] = i
        plan.append((lane, waits))
    return plan


def run_chain(wls, steps, tts, plan, streams):
    """Enqueue one pass of a chain: streams[0] is the caller's current stream (under stream capture: the capturing one),
    the others are side streams that fork from it and join it again at the end."""
    import torch
    events, used = {}, set()
    needed = {p for pl in plan if pl is not None for p in pl[1]}
    start = torch.cuda.Event()
    start.record(streams[0])
    for i, (st, tt, pl) in enumerate(zip(steps, tts, plan)):
        if pl is None:
            continue
        lane, waits = pl
        s = streams[lane]
        if lane != 0 and lane not in used:
            s.wait_event(start)                           # the side stream joins (a capture, or the caller's ordering)
        used.add(lane)
        for p in waits:
            s.wait_event(events[p])
        with torch.cuda.stream(s):
            wls[st.kernel].run(tt)
        if i in needed:
            events[i] = torch.cuda.Event()
            events[i].record(s)
    for lane in sorted(used - {0}):
        e = torch.cuda.Event()
        e.record(streams[lane])
        streams[0].wait_event(e)
