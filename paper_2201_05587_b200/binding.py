"""ctypes binding of libtt.so: argument marshalling only.

Names mirror ``include/tt.h``.  Torch tensors supply device memory and the current
stream; every step of the hot path runs inside the library's CUDA kernels.  There
is no fallback: if the library is missing or no GPU is present the calls raise.
"""
from __future__ import annotations

import ctypes as C
import os

from . import build as _build

HERE = os.path.dirname(os.path.abspath(__file__))

# enums
TT_OK, TT_ERR_INVALID_ARG, TT_ERR_INVALID_SCHEDULE, TT_ERR_CLASS_MISMATCH, TT_ERR_RESOURCE, \
    TT_ERR_NOT_APPLIED, TT_ERR_CUDA, TT_ERR_TIMEOUT, TT_ERR_OOM, TT_ERR_NOT_IMPLEMENTED, TT_SKIPPED = range(11)
TT_OP_CONV2D, TT_OP_DWCONV2D, TT_OP_DENSE, TT_OP_BATCH_MATMUL, TT_OP_SOFTMAX = range(5)
TT_ACT_NONE, TT_ACT_RELU, TT_ACT_RELU6, TT_ACT_GELU_ERF = range(4)
TT_FAMILY_GEMM_TC, TT_FAMILY_DW_SIMT, TT_FAMILY_ROW_SIMT = range(3)
TT_MODE_LEGALISE, TT_MODE_STRICT = 0, 1
TT_RECORD_VERSION = 3
TT_CHG_TILE_M, TT_CHG_TILE_N, TT_CHG_TILE_K, TT_CHG_STAGES, TT_CHG_SPLIT_K, TT_CHG_VEC, TT_CHG_BLOCK, TT_CHG_ITEMS, TT_CHG_SLAB, TT_CHG_ACC, TT_CHG_KORDER, TT_CHG_FORM = \
    1, 2, 4, 8, 16, 32, 64, 128, 256, 512, 1024, 2048

i32, u32, f32 = C.c_int32, C.c_uint32, C.c_float


class tt_shapes(C.Structure):
    _fields_ = [(n, i32) for n in ("n", "c", "h", "w", "k", "r", "s", "stride_h", "stride_w", "pad_h", "pad_w",
                                   "batch", "m", "nn", "kk", "trans_b", "has_bias", "has_residual", "act")] + \
               [("scale", f32)]


class tt_schedule_record(C.Structure):
    _fields_ = [("version", u32), ("family", u32), ("origin_op", i32), ("origin", tt_shapes)] + \
               [(n, i32) for n in ("tile_m", "tile_n", "tile_k", "stages", "split_k", "raster", "block_x", "block_y",
                                   "items_per_thread", "vec_width", "unroll", "threads", "mma_m_axis", "slab_tiles", "acc_split", "k_order",
                                   "persistent", "cta_group", "ctas_per_sm", "warp_layout", "precision")]

    FIELDS = ("tile_m", "tile_n", "tile_k", "stages", "split_k", "raster", "block_x", "block_y",
              "items_per_thread", "vec_width", "unroll", "threads", "mma_m_axis", "slab_tiles", "acc_split", "k_order",
              "persistent", "cta_group", "ctas_per_sm", "warp_layout", "precision")

    def as_dict(self):
        d = {"family": int(self.family), "origin_op": int(self.origin_op)}
        d.update({k: int(getattr(self, k)) for k in self.FIELDS})
        return d

    def short(self):
        if self.family == TT_FAMILY_GEMM_TC:
            return (f"tc[{self.tile_m}x{self.tile_n}x{self.tile_k} st{self.stages} sk{self.split_k} "
                    f"r{self.raster} ax{self.mma_m_axis}" + (f" sl{self.slab_tiles}" if self.slab_tiles else "") +
                    (f" acc{self.acc_split}" if self.acc_split > 1 else "") + (" tap" if self.k_order else "") +
                    (" ps" if self.persistent else "") + (" cg2" if self.cta_group == 2 else "") +
                    (" 2/sm" if self.ctas_per_sm == 2 else "") + (" x3" if self.precision else "") + "]")
        if self.family == TT_FAMILY_DW_SIMT:
            return (f"dw[c{self.tile_m} {self.block_y}x{self.block_x} it{self.items_per_thread} "
                    f"v{self.vec_width} t{self.threads} u{self.unroll}" + (f" tma st{self.stages}" if self.raster else "") + "]")
        return f"row[{self.block_x}x{self.block_y} v{self.vec_width}]"


class tt_tensors(C.Structure):
    _fields_ = [("x", C.c_void_p), ("w", C.c_void_p), ("bias", C.c_void_p), ("residual", C.c_void_p), ("y", C.c_void_p)]


class tt_gemm_view(C.Structure):
    _fields_ = [("batch", i32), ("gm", i32), ("gn", i32), ("gk", i32), ("flops", C.c_double), ("bytes", C.c_double)]


class tt_apply_info(C.Structure):
    _fields_ = [("legal", tt_schedule_record), ("changed", i32), ("grid_x", i32), ("grid_y", i32), ("grid_z", i32),
                ("threads", i32), ("smem_bytes", i32), ("tmem_cols", i32), ("workspace_bytes", C.c_int64),
                ("launches", i32)]


class tt_timing_opts(C.Structure):
    _fields_ = [("warmup_batches", i32), ("batches", i32), ("min_batch_us", i32), ("max_repeats", i32),
                ("use_graph", i32), ("floor", i32), ("reserved", i32 * 2)]


class tt_timing(C.Structure):
    _fields_ = [("median_us", f32), ("min_us", f32), ("max_us", f32), ("q1_us", f32), ("q3_us", f32),
                ("repeats", i32), ("batches", i32)]


class tt_tune_opts(C.Structure):
    _fields_ = [("timing", tt_timing_opts), ("mode", i32), ("strict_class", i32), ("include_default", i32),
                ("subsample_percent", i32), ("subsample_gain_percent", i32), ("subsample_seed", u32), ("reserved", i32 * 2)]


class tt_tune_result(C.Structure):
    _fields_ = [("chosen", C.POINTER(i32)), ("best_us", C.POINTER(f32)), ("times_us", C.POINTER(f32)),
                ("status", C.POINTER(i32)), ("search_seconds", C.c_double), ("pairs_timed", i32),
                ("pairs_invalid", i32), ("pairs_skipped", i32)]


EXPORTS = {
    "tt_status_string": (C.c_char_p, [i32]),
    "tt_workload_create": (i32, [i32, C.POINTER(tt_shapes), C.POINTER(C.c_void_p)]),
    "tt_workload_destroy": (i32, [C.c_void_p]),
    "tt_workload_key": (i32, [C.c_void_p, C.POINTER(C.c_uint64)]),
    "tt_workload_class": (i32, [C.c_void_p, C.POINTER(C.c_uint64)]),
    "tt_workload_family": (i32, [C.c_void_p, C.POINTER(i32)]),
    "tt_workload_gemm_view": (i32, [C.c_void_p, C.POINTER(tt_gemm_view)]),
    "tt_default_schedule": (i32, [C.c_void_p, C.POINTER(tt_schedule_record)]),
    "tt_schedule_check": (i32, [C.c_void_p, C.POINTER(tt_schedule_record), i32, i32, C.POINTER(tt_apply_info)]),
    "tt_schedule_apply": (i32, [C.c_void_p, C.POINTER(tt_schedule_record), C.POINTER(tt_apply_info)]),
    "tt_schedule_apply_ex": (i32, [C.c_void_p, C.POINTER(tt_schedule_record), i32, i32, C.POINTER(tt_apply_info)]),
    "tt_split_check": (i32, [C.c_int64, C.POINTER(C.c_int64), C.c_size_t, i32, C.POINTER(i32)]),
    "tt_run": (i32, [C.c_void_p, C.POINTER(tt_tensors), C.c_void_p]),
    "tt_run_host": (i32, [C.c_void_p, C.POINTER(tt_tensors), C.c_void_p, C.POINTER(C.c_int64), C.POINTER(C.c_int64)]),
    "tt_run_host_async": (i32, [C.c_void_p, C.POINTER(tt_tensors), C.c_void_p, C.POINTER(C.c_int64), C.POINTER(C.c_int64)]),
    "tt_workload_status": (i32, [C.c_void_p, C.c_void_p]),
    "tt_workload_set_constant_weights": (i32, [C.c_void_p, i32]),
    "tt_workload_set_wait_limit": (i32, [C.c_void_p, C.c_uint64]),
    "tt_workload_test_stall": (i32, [C.c_void_p, C.c_uint32]),
    "tt_time": (i32, [C.c_void_p, C.POINTER(tt_tensors), C.c_size_t, C.c_void_p, C.POINTER(tt_timing_opts),
                      C.POINTER(tt_timing)]),
    "tt_select": (i32, [C.POINTER(f32), C.c_size_t, C.c_size_t, C.POINTER(i32)]),
    "tt_model_latency": (i32, [C.POINTER(f32), C.c_size_t, C.c_size_t, C.POINTER(i32), C.POINTER(i32),
                               C.POINTER(C.c_double)]),
    "tt_rank_pools": (i32, [C.POINTER(C.c_double), C.c_size_t, C.POINTER(i32), C.c_size_t, C.POINTER(C.c_double),
                            C.POINTER(i32)]),
    "tt_transfer_tune": (i32, [C.POINTER(C.c_void_p), C.POINTER(tt_tensors), C.c_size_t, C.POINTER(tt_schedule_record),
                               C.c_size_t, C.POINTER(tt_tune_opts), C.c_void_p, C.POINTER(tt_tune_result)]),
    "tt_transfer_tune_sets": (i32, [C.POINTER(C.c_void_p), C.POINTER(tt_tensors), C.POINTER(C.c_size_t), C.c_size_t,
                                    C.POINTER(tt_schedule_record), C.c_size_t, C.POINTER(tt_tune_opts), C.c_void_p,
                                    C.POINTER(tt_tune_result)]),
    "tt_grid_tune": (i32, [C.c_void_p, C.POINTER(tt_tensors), C.c_void_p, C.POINTER(tt_timing_opts), i32, C.c_size_t,
                           C.POINTER(tt_schedule_record), C.POINTER(f32), C.POINTER(C.c_size_t), C.POINTER(i32)]),
    "tt_record_neighbours": (i32, [C.c_void_p, C.POINTER(tt_schedule_record), C.POINTER(tt_schedule_record), C.c_size_t,
                                   C.POINTER(C.c_size_t)]),
    "tt_refine_with": (i32, [C.c_void_p, C.POINTER(tt_schedule_record), C.c_void_p, C.c_void_p, i32, f32,
                             C.POINTER(tt_schedule_record), C.POINTER(f32), C.POINTER(f32), C.POINTER(i32)]),
    "tt_refine": (i32, [C.c_void_p, C.POINTER(tt_tensors), C.c_void_p, C.POINTER(tt_timing_opts),
                        C.POINTER(tt_schedule_record), i32, f32, C.POINTER(tt_schedule_record), C.POINTER(f32),
                        C.POINTER(f32), C.POINTER(i32)]),
    "tt_pool_subsample": (i32, [C.c_size_t, C.c_size_t, C.c_uint64, C.POINTER(i32)]),
    "tt_pool_save": (i32, [C.c_char_p, C.POINTER(tt_schedule_record), C.POINTER(f32), C.c_size_t]),
    "tt_pool_load": (i32, [C.c_char_p, C.POINTER(tt_schedule_record), C.POINTER(f32), C.c_size_t, C.POINTER(C.c_size_t)]),
    "tt_dense_static_scratch": (i32, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, i32, i32, i32, i32,
                                      C.POINTER(tt_schedule_record), C.c_void_p, C.POINTER(C.c_int64)]),
}

_lib = None


def lib():
    """Load libtt.so (building it with nvcc first if the sources are newer).  Raises if that fails."""
    global _lib
    if _lib is None:
        path = _build.LIB
        if _build.needs_build():
            path = _build.build()
        handle = C.CDLL(path)
        for name, (res, args) in EXPORTS.items():
            fn = getattr(handle, name)          # AttributeError if a declared symbol is missing
            fn.restype, fn.argtypes = res, args
        _lib = handle
    return _lib


class TTError(RuntimeError):
    def __init__(self, status, what=""):
        self.status = int(status)
        msg = lib().tt_status_string(self.status).decode()
        super().__init__(f"{what}: {msg} (tt_status {self.status})" if what else f"{msg} (tt_status {self.status})")


def _check(status, what=""):
    if status != TT_OK:
        raise TTError(status, what)


def status_string(s: int) -> str:
    return lib().tt_status_string(int(s)).decode()


def make_shapes(**kw) -> tt_shapes:
    s = tt_shapes()
    for k, v in kw.items():
        if not hasattr(s, k):
            raise KeyError(k)
        setattr(s, k, v)
    return s


def conv2d_shapes(n, c, h, w, k, r, s, stride=1, pad=0, has_bias=True, act=TT_ACT_RELU, has_residual=False):
    return make_shapes(n=n, c=c, h=h, w=w, k=k, r=r, s=s, stride_h=stride, stride_w=stride, pad_h=pad, pad_w=pad,
                       has_bias=int(has_bias), act=act, has_residual=int(has_residual))


def dense_shapes(m, nn, kk, has_bias=True, act=TT_ACT_NONE):
    return make_shapes(batch=1, m=m, nn=nn, kk=kk, trans_b=1, has_bias=int(has_bias), act=act)


def bmm_shapes(batch, m, nn, kk, trans_b=True):
    return make_shapes(batch=batch, m=m, nn=nn, kk=kk, trans_b=int(trans_b))


def softmax_shapes(batch, m, nn, scale=1.0):
    return make_shapes(batch=batch, m=m, nn=nn, scale=scale)


def make_record(family, **kw) -> tt_schedule_record:
    r = tt_schedule_record()
    r.version = TT_RECORD_VERSION
    r.family = family
    defaults = dict(tile_m=128, tile_n=128, tile_k=32, stages=4, split_k=1, raster=0, block_x=32, block_y=4,
                    items_per_thread=1, vec_width=1, unroll=1, threads=128, mma_m_axis=0, slab_tiles=0, acc_split=1, k_order=0,
                    persistent=0, cta_group=1, ctas_per_sm=0, warp_layout=0, precision=0)
    defaults.update(kw)
    for k, v in defaults.items():
        setattr(r, k, v)
    return r


def split_check(extent, factors, reformulate=False) -> bool:
    arr = (C.c_int64 * len(factors))(*factors)
    v = i32(0)
    _check(lib().tt_split_check(extent, arr, len(factors), int(reformulate), C.byref(v)), "tt_split_check")
    return bool(v.value)


def select(times, n_wl, n_cols):
    arr = (f32 * (n_wl * n_cols))(*[float(t) for t in times])
    out = (i32 * n_wl)()
    _check(lib().tt_select(arr, n_wl, n_cols, out), "tt_select")
    return list(out)


def model_latency(times, n_wl, n_cols, chosen, use_count) -> float:
    arr = (f32 * (n_wl * n_cols))(*[float(t) for t in times])
    ch = (i32 * n_wl)(*chosen)
    uc = (i32 * n_wl)(*use_count)
    out = C.c_double(0)
    _check(lib().tt_model_latency(arr, n_wl, n_cols, ch, uc, C.byref(out)), "tt_model_latency")
    return out.value


def rank_pools(class_share, class_kernels):
    """Equation 1: class_share[c] of the target model, class_kernels[t][c] of each candidate; returns (scores, order)."""
    n_c, n_m = len(class_share), len(class_kernels)
    sh = (C.c_double * n_c)(*[float(v) for v in class_share])
    ck = (i32 * (n_c * max(n_m, 1)))(*[int(v) for row in class_kernels for v in row])
    sc = (C.c_double * max(n_m, 1))()
    od = (i32 * max(n_m, 1))()
    _check(lib().tt_rank_pools(sh, n_c, ck, n_m, sc, od), "tt_rank_pools")
    return list(sc)[:n_m], list(od)[:n_m]


def pool_subsample(n_pool, count, seed):
    """tt_pool_subsample: the first `count` indices of the seeded shuffle of range(n_pool)."""
    out = (i32 * max(count, 1))()
    _check(lib().tt_pool_subsample(n_pool, count, seed, out), "tt_pool_subsample")
    return list(out)[:count]


def pool_save(path, records, us=None):
    """tt_pool_save: write records (and the times they were tuned to) as a text pool file."""
    n = len(records)
    arr = (tt_schedule_record * max(n, 1))(*records)
    uarr = (f32 * max(n, 1))(*[float(v) for v in us]) if us is not None else None
    _check(lib().tt_pool_save(os.fsencode(path), arr, uarr, n), f"tt_pool_save({path})")


def pool_load(path):
    """tt_pool_load: returns (records, times in microseconds)."""
    n = C.c_size_t()
    _check(lib().tt_pool_load(os.fsencode(path), None, None, 0, C.byref(n)), f"tt_pool_load({path})")
    arr = (tt_schedule_record * max(n.value, 1))()
    uarr = (f32 * max(n.value, 1))()
    _check(lib().tt_pool_load(os.fsencode(path), arr, uarr, n.value, C.byref(n)), f"tt_pool_load({path})")
    out = []
    for i in range(n.value):
        r = tt_schedule_record()
        C.memmove(C.byref(r), C.byref(arr[i]), C.sizeof(r))
        out.append(r)
    return out, [float(uarr[i]) for i in range(n.value)]


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def tensors(x, w=None, bias=None, residual=None, y=None) -> tt_tensors:
    """Device pointers of torch CUDA tensors (or host pointers of CPU tensors for tt_run_host)."""
    t = tt_tensors()
    t.x, t.w, t.bias, t.residual, t.y = _ptr(x), _ptr(w), _ptr(bias), _ptr(residual), _ptr(y)
    return t


def _stream():
    import torch
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


class Workload:
    """Owns one tt_workload handle."""

    def __init__(self, op, shapes: tt_shapes, name: str = "", use_count: int = 1):
        self.op, self.shapes, self.name, self.use_count = op, shapes, name, use_count
        h = C.c_void_p()
        _check(lib().tt_workload_create(op, C.byref(shapes), C.byref(h)), f"tt_workload_create({name})")
        self.handle = h

    def close(self):
        if getattr(self, "handle", None):
            lib().tt_workload_destroy(self.handle)
            self.handle = None

    __del__ = close

    def key(self) -> int:
        v = C.c_uint64()
        _check(lib().tt_workload_key(self.handle, C.byref(v)))
        return v.value

    def kernel_class(self) -> int:
        v = C.c_uint64()
        _check(lib().tt_workload_class(self.handle, C.byref(v)))
        return v.value

    def family(self) -> int:
        v = i32()
        _check(lib().tt_workload_family(self.handle, C.byref(v)))
        return v.value

    def gemm_view(self) -> tt_gemm_view:
        v = tt_gemm_view()
        _check(lib().tt_workload_gemm_view(self.handle, C.byref(v)))
        return v

    def default_schedule(self) -> tt_schedule_record:
        r = tt_schedule_record()
        _check(lib().tt_default_schedule(self.handle, C.byref(r)))
        return r

    def check(self, rec, mode=TT_MODE_LEGALISE, strict_class=False):
        """Returns (status, tt_apply_info); never raises for an invalid record."""
        info = tt_apply_info()
        st = lib().tt_schedule_check(self.handle, C.byref(rec), mode, int(strict_class), C.byref(info))
        return st, info

    def apply(self, rec, mode=TT_MODE_LEGALISE, strict_class=False) -> tt_apply_info:
        info = tt_apply_info()
        _check(lib().tt_schedule_apply_ex(self.handle, C.byref(rec), mode, int(strict_class), C.byref(info)),
               f"tt_schedule_apply({self.name})")
        return info

    def try_apply(self, rec, mode=TT_MODE_LEGALISE, strict_class=False):
        info = tt_apply_info()
        st = lib().tt_schedule_apply_ex(self.handle, C.byref(rec), mode, int(strict_class), C.byref(info))
        return st, info

    def run(self, t: tt_tensors):
        _check(lib().tt_run(self.handle, C.byref(t), _stream()), f"tt_run({self.name})")

    def run_host(self, t: tt_tensors):
        up, down = C.c_int64(), C.c_int64()
        _check(lib().tt_run_host(self.handle, C.byref(t), _stream(), C.byref(up), C.byref(down)),
               f"tt_run_host({self.name})")
        return up.value, down.value

    def run_host_async(self, t: tt_tensors, stream=None):
        """tt_run_host_async on `stream` (a torch.cuda.Stream; default: the current one): enqueues only."""
        up, down = C.c_int64(), C.c_int64()
        sp = _stream() if stream is None else C.c_void_p(stream.cuda_stream)
        _check(lib().tt_run_host_async(self.handle, C.byref(t), sp, C.byref(up), C.byref(down)),
               f"tt_run_host_async({self.name})")
        return up.value, down.value

    def status(self, stream=None) -> int:
        sp = _stream() if stream is None else C.c_void_p(stream.cuda_stream)
        return lib().tt_workload_status(self.handle, sp)

    def set_constant_weights(self, on: bool = True):
        _check(lib().tt_workload_set_constant_weights(self.handle, int(bool(on))), "tt_workload_set_constant_weights")

    def set_wait_limit(self, nanoseconds: int):
        _check(lib().tt_workload_set_wait_limit(self.handle, int(nanoseconds)), "tt_workload_set_wait_limit")

    def test_stall(self, extra_bytes: int):
        _check(lib().tt_workload_test_stall(self.handle, int(extra_bytes)), "tt_workload_test_stall")

    def time(self, sets, opts: tt_timing_opts | None = None) -> tt_timing:
        if isinstance(sets, tt_tensors):
            sets = [sets]
        arr = (tt_tensors * len(sets))(*sets)
        out = tt_timing()
        _check(lib().tt_time(self.handle, arr, len(sets), _stream(), C.byref(opts) if opts else None, C.byref(out)),
               f"tt_time({self.name})")
        return out

    def grid_tune(self, t: tt_tensors, opts: tt_timing_opts | None = None, level=0, top_k=1):
        recs = (tt_schedule_record * top_k)()
        us = (f32 * top_k)()
        n = C.c_size_t()
        tried = i32()
        _check(lib().tt_grid_tune(self.handle, C.byref(t), _stream(), C.byref(opts) if opts else None, level, top_k,
                                  recs, us, C.byref(n), C.byref(tried)), f"tt_grid_tune({self.name})")
        out = []
        for i in range(n.value):
            r = tt_schedule_record()
            C.memmove(C.byref(r), C.byref(recs[i]), C.sizeof(r))
            out.append((r, float(us[i])))
        return out, tried.value


    def neighbours(self, rec):
        """tt_record_neighbours: the legalised one-step neighbours of `rec` on this workload."""
        out = (tt_schedule_record * 32)()
        n = C.c_size_t()
        _check(lib().tt_record_neighbours(self.handle, C.byref(rec), out, 32, C.byref(n)), f"tt_record_neighbours({self.name})")
        res = []
        for i in range(n.value):
            r = tt_schedule_record()
            C.memmove(C.byref(r), C.byref(out[i]), C.sizeof(r))
            res.append(r)
        return res

    def refine_with(self, start, time_us, max_rounds=8, min_gain=0.0):
        """tt_refine_with: greedy descent from `start` with a Python timing function rec -> microseconds (negative =
        cannot run).  Returns (best record, best_us, start_us, calls of time_us)."""
        def _cb(_user, rec_ptr):
            return float(time_us(rec_ptr.contents))
        cb = TIME_FN(_cb)
        best, bus, sus, nt = tt_schedule_record(), f32(), f32(), i32()
        _check(lib().tt_refine_with(self.handle, C.byref(start), C.cast(cb, C.c_void_p), None, max_rounds, min_gain,
                                    C.byref(best), C.byref(bus), C.byref(sus), C.byref(nt)), f"tt_refine_with({self.name})")
        return best, bus.value, sus.value, nt.value

    def refine(self, t: tt_tensors, start, opts: tt_timing_opts | None = None, max_rounds=4, min_gain=0.02):
        """tt_refine: the same with device times (median of tt_time); leaves the best record applied."""
        best, bus, sus, nt = tt_schedule_record(), f32(), f32(), i32()
        _check(lib().tt_refine(self.handle, C.byref(t), _stream(), C.byref(opts) if opts else None, C.byref(start),
                               max_rounds, min_gain, C.byref(best), C.byref(bus), C.byref(sus), C.byref(nt)),
               f"tt_refine({self.name})")
        return best, bus.value, sus.value, nt.value


TIME_FN = C.CFUNCTYPE(f32, C.c_void_p, C.POINTER(tt_schedule_record))
TT_STATIC_SCRATCH_BYTES = 8 << 20


def dense_static_scratch(x, w, bias, y, act, rec):
    """tt_dense_static_scratch on torch CUDA tensors x [m,kk], w [nn,kk], bias [nn] or None, y [m,nn]: the dense
    layer under `rec` with its split-K scratch in the library's fixed device array, for callers that cannot
    allocate device memory.  Returns (tt_status, scratch bytes the record needs); never raises."""
    m, kk = x.shape
    nn = w.shape[0]
    used = C.c_int64(0)
    st = lib().tt_dense_static_scratch(_ptr(x), _ptr(w), _ptr(bias), _ptr(y), m, nn, kk, act, C.byref(rec), _stream(),
                                       C.byref(used))
    return st, used.value


def transfer_tune(workloads, tensor_sets, pool, opts: tt_tune_opts | None = None):
    """Evaluate every workload under the default record and every pool record; returns a dict with
    chosen (column index per workload), best_us, times_us [n_wl][n_pool+1], status, search_seconds, counts."""
    n_wl, n_pool = len(workloads), len(pool)
    n_cols = n_pool + 1
    handles = (C.c_void_p * n_wl)(*[w.handle for w in workloads])
    # an entry of tensor_sets may be one tt_tensors or a list of them (several sets, walked round-robin while timing)
    multi = any(not isinstance(t, tt_tensors) for t in tensor_sets)
    groups = [[t] if isinstance(t, tt_tensors) else list(t) for t in tensor_sets]
    flat_sets = [t for g in groups for t in g]
    tens = (tt_tensors * len(flat_sets))(*flat_sets)
    counts = (C.c_size_t * n_wl)(*[len(g) for g in groups])
    parr = (tt_schedule_record * max(n_pool, 1))(*pool)
    chosen = (i32 * n_wl)()
    best = (f32 * n_wl)()
    times = (f32 * (n_wl * n_cols))()
    status = (i32 * (n_wl * n_cols))()
    res = tt_tune_result()
    res.chosen, res.best_us, res.times_us, res.status = chosen, best, times, status
    if opts is None:
        opts = tt_tune_opts()
        opts.include_default = 1
    if multi:
        _check(lib().tt_transfer_tune_sets(handles, tens, counts, n_wl, parr, n_pool, C.byref(opts), _stream(), C.byref(res)),
               "tt_transfer_tune_sets")
    else:
        _check(lib().tt_transfer_tune(handles, tens, n_wl, parr, n_pool, C.byref(opts), _stream(), C.byref(res)),
               "tt_transfer_tune")
    return {
        "chosen": list(chosen), "best_us": list(best),
        "times_us": [[times[i * n_cols + j] for j in range(n_cols)] for i in range(n_wl)],
        "status": [[status[i * n_cols + j] for j in range(n_cols)] for i in range(n_wl)],
        "search_seconds": res.search_seconds, "pairs_timed": res.pairs_timed, "pairs_invalid": res.pairs_invalid,
        "pairs_skipped": res.pairs_skipped,
    }
