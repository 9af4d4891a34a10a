"""CPU oracle for the hot path of transfer-tuning.  TEST INFRASTRUCTURE ONLY.

Nothing in the product path imports this module.  It wraps the plain C loops of
``tt_oracle.c`` (fp64 accumulation) with numpy in/out and adds, in plain Python,
the host-side definitions the paper fixes:

* ``split_covers`` / ``split_reformulated_valid`` / ``factor_fits`` — the validity
  examples of Section 4.1 (a split must traverse the whole loop; the reformulated
  split is valid when the inner factor divides the extent) and Section 4.2 (a
  split factor larger than the loop is invalid; a schedule of another kernel class
  is always invalid).
* ``select`` — keep, per kernel, the fastest schedule that produced valid code
  (Section 4.3); invalid pairs carry a negative time as in Figure 4.
* ``model_latency`` — sum of use count x chosen standalone time.
* ``rank_pools`` — the model-selection heuristic, Equation 1 (Section 4.4).
* ``ladder_steps`` / ``raw_neighbours`` / ``refine`` — varying the parameters of a
  transferred schedule (Section 7, future work) as a greedy one-field-at-a-time descent.

Parity pinning status: conv2d, dwconv2d, dense/batch_matmul, softmax, the
activations, the split rules and ``select`` are pinned by closed forms, brute
force and the paper's worked examples in ``tests/test_oracle_pins.py``;
``rank_pools`` by Tables 2 and 3 of the paper (all ten top-3 rankings).
``refine`` is pinned by exhaustive search on small separable cost tables (on a
separable convex cost a one-field descent must reach the global minimum).
The absolute kernel times and which schedule wins on a given kernel are
"parity unpinned": the paper's per-kernel times exist only in a figure.
"""
from __future__ import annotations

import ctypes
import math
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "tt_oracle.c")
_LIB = os.path.join(_HERE, "libtt_oracle.so")

ACT_NONE, ACT_RELU, ACT_RELU6, ACT_GELU_ERF = 0, 1, 2, 3
MODE_EXACT, MODE_TF32_TRUNC, MODE_TF32_ROUND = 0, 1, 2

_lib = None


def build(force: bool = False) -> str:
    """Compile tt_oracle.c with gcc into libtt_oracle.so next to it."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["gcc", "-O3", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-o", _LIB, _SRC, "-lm"]
        )
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        fp = ctypes.POINTER(ctypes.c_float)
        i = ctypes.c_int
        lib.orc_max_threads.restype = i
        lib.orc_conv2d.restype = i
        lib.orc_conv2d.argtypes = [fp, fp, fp, fp, fp] + [i] * 14
        lib.orc_dwconv2d.restype = i
        lib.orc_dwconv2d.argtypes = [fp, fp, fp, fp] + [i] * 12
        lib.orc_batch_matmul.restype = i
        lib.orc_batch_matmul.argtypes = [fp, fp, fp, fp] + [i] * 8
        lib.orc_softmax.restype = i
        lib.orc_softmax.argtypes = [fp, fp, ctypes.c_long, i, ctypes.c_float, i]
        _lib = lib
    return _lib


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def _p(a):
    if a is None:
        return None
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_float))


def max_threads() -> int:
    return int(_load().orc_max_threads())


def conv2d(x, w, bias=None, stride=(1, 1), pad=(0, 0), act=ACT_NONE, residual=None,
           mode=MODE_EXACT, threads=0, return_threads=False):
    """Algorithm 2: act(conv2d(pad(x), w) + bias [+ residual]); x NCHW, w KCRS."""
    x, w = _f32(x), _f32(w)
    n, c, h, wd = x.shape
    k, c2, r, s = w.shape
    assert c2 == c
    bias = None if bias is None else _f32(bias)
    residual = None if residual is None else _f32(residual)
    p = (h + 2 * pad[0] - r) // stride[0] + 1
    q = (wd + 2 * pad[1] - s) // stride[1] + 1
    y = np.empty((n, k, p, q), dtype=np.float32)
    used = _load().orc_conv2d(_p(x), _p(w), _p(bias), _p(residual), _p(y), n, c, h, wd, k, r, s,
                              stride[0], stride[1], pad[0], pad[1], act, mode, threads)
    return (y, used) if return_threads else y


def dwconv2d(x, w, bias=None, stride=(1, 1), pad=(0, 0), act=ACT_NONE, threads=0,
             return_threads=False):
    """Depthwise Algorithm 2: x NCHW, w [C,1,R,S]."""
    x, w = _f32(x), _f32(w)
    n, c, h, wd = x.shape
    assert w.shape[0] == c and w.shape[1] == 1
    r, s = w.shape[2], w.shape[3]
    bias = None if bias is None else _f32(bias)
    p = (h + 2 * pad[0] - r) // stride[0] + 1
    q = (wd + 2 * pad[1] - s) // stride[1] + 1
    y = np.empty((n, c, p, q), dtype=np.float32)
    used = _load().orc_dwconv2d(_p(x), _p(w), _p(bias), _p(y), n, c, h, wd, r, s,
                                stride[0], stride[1], pad[0], pad[1], act, threads)
    return (y, used) if return_threads else y


def batch_matmul(a, b, bias=None, trans_b=False, act=ACT_NONE, mode=MODE_EXACT, threads=0,
                 return_threads=False):
    """Algorithm 1 per batch entry: a [B,N,K]; b [B,K,M] or, with trans_b, [B,M,K]."""
    a, b = _f32(a), _f32(b)
    bt, n, k = a.shape
    if trans_b:
        assert b.shape[0] == bt and b.shape[2] == k
        m = b.shape[1]
    else:
        assert b.shape[0] == bt and b.shape[1] == k
        m = b.shape[2]
    bias = None if bias is None else _f32(bias)
    c = np.empty((bt, n, m), dtype=np.float32)
    used = _load().orc_batch_matmul(_p(a), _p(b), _p(bias), _p(c), bt, n, m, k, int(trans_b), act,
                                    mode, threads)
    return (c, used) if return_threads else c


def dense(x, w, bias=None, act=ACT_NONE, mode=MODE_EXACT, threads=0, return_threads=False):
    """dense+bias: y[m,n] = act(bias[n] + sum_k x[m,k] w[n,k]); weight stored [out, in]."""
    x, w = _f32(x), _f32(w)
    out = batch_matmul(x[None], w[None], bias, trans_b=True, act=act, mode=mode, threads=threads,
                       return_threads=return_threads)
    if return_threads:
        return out[0][0], out[1]
    return out[0]


def softmax(s, scale=1.0, threads=0):
    """Row softmax of scale*s over the last axis."""
    s = _f32(s)
    cols = s.shape[-1]
    rows = s.size // cols
    p = np.empty_like(s)
    _load().orc_softmax(_p(s), _p(p), rows, cols, float(scale), threads)
    return p


# operator numbering of the C ABI under test (tt_op in include/tt.h), restated here: the oracle imports nothing
OP_CONV2D, OP_DWCONV2D, OP_DENSE, OP_BATCH_MATMUL, OP_SOFTMAX = range(5)


def reference(op: int, s, a, mode=MODE_EXACT, threads=0):
    """Reference output of one kernel: `s` carries the size fields of the ABI's shape struct (any object with
    those attributes), `a` maps 'x', 'w', 'bias', 'residual' to numpy arrays or None."""
    if op == OP_CONV2D:
        return conv2d(a["x"], a["w"], a.get("bias"), (s.stride_h, s.stride_w), (s.pad_h, s.pad_w), s.act,
                      a.get("residual"), mode=mode, threads=threads)
    if op == OP_DWCONV2D:
        return dwconv2d(a["x"], a["w"], a.get("bias"), (s.stride_h, s.stride_w), (s.pad_h, s.pad_w), s.act,
                        threads=threads)
    if op == OP_DENSE:
        return dense(a["x"], a["w"], a.get("bias"), s.act, mode=mode, threads=threads)
    if op == OP_BATCH_MATMUL:
        return batch_matmul(a["x"], a["w"], None, bool(s.trans_b), s.act, mode=mode, threads=threads)
    if op == OP_SOFTMAX:
        return softmax(a["x"], s.scale, threads=threads)
    raise ValueError(f"unknown operator {op}")


def rel_l2(y, ref) -> float:
    """||y - ref||_2 / ||ref||_2 in double; absolute norm of y when ref is all zero."""
    y = np.asarray(y, dtype=np.float64).ravel()
    ref = np.asarray(ref, dtype=np.float64).ravel()
    den = np.linalg.norm(ref)
    if den == 0.0:
        return float(np.linalg.norm(y))
    return float(np.linalg.norm(y - ref) / den)


# ---- host-side definitions (Sections 4.1 - 4.3) --------------------------------

def split_covers(extent: int, factors) -> bool:
    """Split(N, f0, f1, ...) replaces the loop over (0, N) by nested loops over
    (0, f0), (0, f1), ...; it is valid only when those traverse exactly N elements."""
    prod = 1
    for f in factors:
        if f <= 0:
            return False
        prod *= int(f)
    return prod == int(extent)


def split_reformulated_valid(extent: int, inner: int) -> bool:
    """Split(N, N/inner, inner) is valid exactly when inner divides N."""
    return inner > 0 and extent > 0 and extent % inner == 0


def factor_fits(extent: int, factor: int) -> bool:
    """A split factor larger than the loop itself produces invalid code."""
    return 0 < factor <= extent


def same_class(ops_a, ops_b) -> bool:
    """Schedules transfer only between kernels with the same sequence of operations."""
    return tuple(ops_a) == tuple(ops_b)


def select(times, n_wl: int, n_sched: int):
    """Per kernel, the index of the smallest non-negative time; ties keep the lowest
    index; a row with no valid entry gives -1."""
    t = np.asarray(times, dtype=np.float64).reshape(n_wl, n_sched)
    chosen = []
    for row in t:
        best, best_t = -1, None
        for j, v in enumerate(row):
            if v < 0 or not np.isfinite(v):
                continue
            if best_t is None or v < best_t:
                best, best_t = j, v
        chosen.append(best)
    return chosen


def model_latency(use_counts, times, chosen, n_sched: int) -> float:
    """Sum over kernels of use count x time of the chosen schedule."""
    t = np.asarray(times, dtype=np.float64).reshape(len(use_counts), n_sched)
    return float(sum(u * t[i, c] for i, (u, c) in enumerate(zip(use_counts, chosen)) if c >= 0))


def rank_pools(target_share, candidate_counts):
    """Equation 1 (model-selection heuristic): score of candidate model T for a target model with class shares P_c is
    sum over the target's classes c of P_c^2 * sqrt(|W_Tc|), |W_Tc| = number of kernels of class c in T.

    target_share: {class: share of untuned inference time, as a fraction};
    candidate_counts: list of {class: number of kernels}, one per candidate.
    Returns (scores, order): order lists candidate indices by decreasing score, ties keeping the lower index first."""
    scores = []
    for counts in candidate_counts:
        s = 0.0
        for cls, p in target_share.items():
            n = counts.get(cls, 0)
            s += (p * p) * math.sqrt(n)
        scores.append(s)
    order = sorted(range(len(scores)), key=lambda i: (-scores[i], i))
    return scores, order


# ---- refining a transferred schedule (named as future work in Section 7): local search over a record's fields ----
# The paper names the idea only; the reading taken here: each parameter has an ordered ladder of values, a step moves
# one parameter to the next lower or next higher rung, and the search is a greedy descent over those steps.
LADDERS = {
    "gemm_tc": [("tile_n", [16, 32, 48, 64, 96, 128, 160, 192, 224, 256]), ("tile_k", [8, 16, 32, 64, 96, 128]),
                ("stages", [1, 2, 3, 4, 5, 6, 7, 8]), ("split_k", [1, 2, 3, 4, 5, 6, 7, 8, 12, 16, 24, 32]),
                ("raster", [0, 1]), ("mma_m_axis", [1, 2]), ("slab_tiles", [0, 1, 2, 4, 8]), ("acc_split", [1, 2, 4, 8]),
                ("k_order", [0, 1]), ("persistent", [0, 1]), ("cta_group", [1, 2]), ("ctas_per_sm", [1, 2])],
    "dw_simt": [("tile_m", [1, 2, 4, 8, 16, 32]), ("block_y", [1, 2, 4, 7, 8, 14, 16, 28, 56]),
                ("block_x", [8, 16, 28, 32, 56, 64, 112]), ("items_per_thread", [1, 2, 4, 8]), ("vec_width", [1, 2, 4]),
                ("threads", [32, 64, 128, 256, 512]), ("unroll", [0, 1, 2, 4]), ("raster", [0, 1]), ("stages", [2, 3, 4])],
    "row_simt": [("block_x", [1, 2, 4, 8, 16, 32]), ("block_y", [1, 2, 4, 8, 16]), ("vec_width", [1, 2, 4])],
}


def ladder_steps(value: int, ladder):
    """The rungs next to `value`: the largest rung below it and the smallest above it (either may be missing;
    `value` itself need not be a rung)."""
    below = [r for r in ladder if r < value]
    above = [r for r in ladder if r > value]
    out = []
    if below:
        out.append(max(below))
    if above:
        out.append(min(above))
    return out


def raw_neighbours(record: dict, family: str):
    """One-step variations of a schedule given as {parameter: value}: per parameter of the family, in ladder order,
    the lower step then the upper step, everything else unchanged.  (Mapping a variation onto a kernel's legal
    schedules, and dropping those that coincide, is the validity layer's job, not part of this definition.)"""
    out = []
    for name, ladder in LADDERS[family]:
        for v in ladder_steps(record[name], ladder):
            r = dict(record)
            r[name] = v
            out.append(r)
    return out


def refine(start, neighbours, time_us, max_rounds: int, min_gain: float = 0.0):
    """Greedy descent: time the start; then, up to max_rounds times, time every neighbour of the current schedule
    that was not timed before and move to the fastest one if it is faster than the current one by more than the
    fraction min_gain (ties keep the earlier neighbour); stop otherwise.  `neighbours(s)` lists hashable schedules,
    `time_us(s)` is negative for a schedule that cannot run.  Returns (best, best_us, start_us, number of timings)."""
    cur, cur_us = start, time_us(start)
    timed = 1
    start_us = cur_us
    if not cur_us >= 0:
        raise ValueError("the start schedule cannot run")
    seen = {start}
    for _ in range(max_rounds):
        pick, pick_us = None, cur_us
        for nb in neighbours(cur):
            if nb in seen:
                continue
            seen.add(nb)
            us = time_us(nb)
            timed += 1
            if us >= 0 and us < pick_us:
                pick, pick_us = nb, us
        if pick is None or not pick_us < cur_us * (1.0 - min_gain):
            break
        cur, cur_us = pick, pick_us
    return cur, cur_us, start_us, timed


# ---- pool sub-sampling (the paper notes that a larger pool lengthens the search, Section 5.5) ----
_M64 = (1 << 64) - 1


def splitmix64(state: int):
    """One step of the splitmix64 generator (Steele, Lea, Flood 2014; Vigna's public-domain reference): the state
    advances by the golden-ratio increment, the output is the state after two xor-shift-multiply rounds and a final
    xor-shift.  Returns (new state, output)."""
    state = (state + 0x9E3779B97F4A7C15) & _M64
    z = state
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _M64
    return state, z ^ (z >> 31)


def pool_subsample(n_pool: int, count: int, seed: int):
    """The first `count` entries of a Fisher-Yates shuffle of range(n_pool) taken from the front: position i is swapped
    with position i + r mod (n_pool - i), r the next splitmix64 output of the generator started at `seed`."""
    if count > n_pool:
        raise ValueError("more records asked for than the pool holds")
    perm = list(range(n_pool))
    state = seed & _M64
    for i in range(count):
        state, r = splitmix64(state)
        j = i + r % (n_pool - i)
        perm[i], perm[j] = perm[j], perm[i]
    return perm[:count]


def evaluate_subsampled(times_row, first, gain_percent: float):
    """Which columns of one kernel's row get evaluated under sub-sampling, given what every column WOULD measure:
    column 0 (the default record) and the subset `first` (pool indices) always; the rest only if the subset's best
    valid time is not below the default's by more than gain_percent.  Returns the set of evaluated columns."""
    cols = {0} | {f + 1 for f in first}
    valid = [times_row[f + 1] for f in first if times_row[f + 1] >= 0]
    default = times_row[0]
    if valid and default >= 0 and min(valid) <= default * (1.0 - gain_percent / 100.0):
        return cols
    return set(range(len(times_row)))
