// Device-facing half of the C ABI: binding a legalised record to a workload (workspace, tensor maps), running,
// the device-timed evaluator (Section 4.3 of the paper), the native grid tuner that fills pools.
#include <cuda_runtime.h>
#include <cuda.h>
#include <algorithm>
#include <chrono>
#include <cstring>
#include <vector>
#include "tt_internal.h"

namespace tt {

cudaError_t launch_gemm(const tt_apply_info& I, const GemmArgs& g, const void* tmap_a, const void* tmap_b, const void* tmap_x,
                        cudaStream_t st);
cudaError_t launch_dw(const tt_apply_info& I, const DwArgs& dw, cudaStream_t st);
cudaError_t launch_dw_tma(const tt_apply_info& I, const DwArgs& dw, const void* tmap_x, cudaStream_t st);
cudaError_t launch_row(const tt_apply_info& I, const RowArgs& row, cudaStream_t st);
cudaError_t gemm_cluster_fits(int smem_bytes, int cluster, int* fits);
cudaError_t launch_repack(const float* w, float* out, int kout, int C, int RS, int CB, cudaStream_t st);
cudaError_t launch_floor(const tt_apply_info& I, int cluster, cudaStream_t st);
cudaError_t launch_gemm_ps(const tt_apply_info& I, const GemmArgs& g, const void* tmap_a, const void* tmap_b, const void* tmap_x,
                           cudaStream_t st);

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver entry point is looked up through the runtime, so the library links against cudart only and loads
// on machines without a driver.
EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
        else
            cudaGetLastError();
    }
    return fn;
}

bool device_present() {
    int n = 0;
    if (cudaGetDeviceCount(&n) != cudaSuccess) { cudaGetLastError(); return false; }
    return n > 0;
}

// K-major operand [batch][rows][K] -> 3-D tensor map, box = [atom_k, box_rows, 1], swizzle span = one box row.
tt_status encode_operand(void* out, const float* base, int K, int rows, int batch, long long rs, long long bs,
                         bool batched, int atom_k, int box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return TT_ERR_CUDA;
    if ((reinterpret_cast<uintptr_t>(base) & 15u) != 0) return TT_ERR_INVALID_ARG;
    const cuuint64_t nb = batched ? (cuuint64_t)batch : 1;
    cuuint64_t dims[3] = {(cuuint64_t)K, (cuuint64_t)rows, nb};
    cuuint64_t strides[2] = {(cuuint64_t)rs * 4, (cuuint64_t)(batched ? bs : (long long)rows * rs) * 4};
    cuuint32_t box[3] = {(cuuint32_t)atom_k, (cuuint32_t)box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    const int row_bytes = atom_k * 4;
    const CUtensorMapSwizzle swz = row_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                                 : row_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B;
    CUresult r = fn(reinterpret_cast<CUtensorMap*>(out), CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float*>(base),
                    dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? TT_OK : TT_ERR_CUDA;
}

// Row-contiguous operand [batch][K][rows] (element (row, k) at k * ks + row) -> 3-D tensor map without swizzle,
// box = [box_rows, box_k, 1]: the staging boxes of the persistent kernel.
tt_status encode_operand_mn(void* out, const float* base, int rows, int K, int batch, long long ks, long long bs, bool batched,
                            int box_rows, int box_k) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return TT_ERR_CUDA;
    if ((reinterpret_cast<uintptr_t>(base) & 15u) != 0) return TT_ERR_INVALID_ARG;
    const cuuint64_t nb = batched ? (cuuint64_t)batch : 1;
    cuuint64_t dims[3] = {(cuuint64_t)rows, (cuuint64_t)K, nb};
    cuuint64_t strides[2] = {(cuuint64_t)ks * 4, (cuuint64_t)(batched ? bs : (long long)K * ks) * 4};
    cuuint32_t box[3] = {(cuuint32_t)box_rows, (cuuint32_t)box_k, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(reinterpret_cast<CUtensorMap*>(out), CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float*>(base), dims,
                    strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? TT_OK : TT_ERR_CUDA;
}

// NCHW image -> 4-D tensor map (W, H, C, N) without swizzle; box = [W + gap, in_rows, box_ch, 1].  A load that
// starts `gap` columns left of the image and at any (also negative) row gets zeros for everything outside.
tt_status encode_image(void* out, const float* base, int W, int H, int C, int N, int box_w, int box_h, int box_c) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return TT_ERR_CUDA;
    if ((reinterpret_cast<uintptr_t>(base) & 15u) != 0) return TT_ERR_INVALID_ARG;
    cuuint64_t dims[4] = {(cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)C, (cuuint64_t)N};
    cuuint64_t strides[3] = {(cuuint64_t)W * 4, (cuuint64_t)W * H * 4, (cuuint64_t)W * H * C * 4};
    cuuint32_t box[4] = {(cuuint32_t)box_w, (cuuint32_t)box_h, (cuuint32_t)box_c, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = fn(reinterpret_cast<CUtensorMap*>(out), CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, const_cast<float*>(base), dims,
                    strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? TT_OK : TT_ERR_CUDA;
}

// Depthwise input as a 3-D tensor (W, H, planes = N * C), box = [box_w, in_h, tile_c], no swizzle.
tt_status encode_planes(void* out, const float* base, int W, int H, long long planes, int box_w, int box_h, int box_c) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return TT_ERR_CUDA;
    if ((reinterpret_cast<uintptr_t>(base) & 15u) != 0) return TT_ERR_INVALID_ARG;
    cuuint64_t dims[3] = {(cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)planes};
    cuuint64_t strides[2] = {(cuuint64_t)W * 4, (cuuint64_t)W * H * 4};
    cuuint32_t box[3] = {(cuuint32_t)box_w, (cuuint32_t)box_h, (cuuint32_t)box_c};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(reinterpret_cast<CUtensorMap*>(out), CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float*>(base), dims,
                    strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? TT_OK : TT_ERR_CUDA;
}

const void* pick(const tt_tensors* t, int which) { return which == 0 ? t->x : t->w; }

}  // namespace

void release_device(tt_workload* w) {
    if (w->workspace) cudaFree(w->workspace);
    if (w->status_word) cudaFree(w->status_word);
    if (w->ktab_dev) cudaFree(w->ktab_dev);
    w->ktab_dev = nullptr; w->ktab_bytes = 0;
    for (int i = 0; i < 5; ++i) if (w->hbuf[i]) cudaFree(w->hbuf[i]);
    w->workspace = nullptr; w->workspace_bytes = 0; w->status_word = nullptr;
    for (int i = 0; i < 5; ++i) { w->hbuf[i] = nullptr; w->hbytes[i] = 0; }
    cudaGetLastError();
}

tt_status bind_device(tt_workload* w) {
    if (!device_present()) return TT_ERR_CUDA;
    if (w->family == TT_FAMILY_GEMM_TC && w->plan.g.cluster) {
        // a cluster whose CTAs cannot be resident together can never launch: an invalid pair, not a device error
        int fits = 0;
        if (gemm_cluster_fits(w->plan.info.smem_bytes, w->plan.g.cluster, &fits) != cudaSuccess) { cudaGetLastError(); return TT_ERR_CUDA; }
        if (!fits) return TT_ERR_RESOURCE;
    }
    const size_t need = (size_t)w->plan.info.workspace_bytes;
    if (need > w->workspace_bytes) {
        if (w->workspace) cudaFree(w->workspace);
        w->workspace = nullptr; w->workspace_bytes = 0;
        if (cudaMalloc(&w->workspace, need) != cudaSuccess) { cudaGetLastError(); return TT_ERR_OOM; }
        w->workspace_bytes = need;
    }
    if (need > 0 && !w->plan.repack) {
        // arrival counters start at zero; each launch leaves them at zero again
        const size_t off = (size_t)w->plan.partial_bytes;
        if (cudaMemset(static_cast<char*>(w->workspace) + off, 0, need - off) != cudaSuccess) { cudaGetLastError(); return TT_ERR_CUDA; }
    }
    if (!w->status_word) {
        if (cudaMalloc(reinterpret_cast<void**>(&w->status_word), 512) != cudaSuccess) { cudaGetLastError(); return TT_ERR_OOM; }
        if (cudaMemset(w->status_word, 0, 512) != cudaSuccess) return TT_ERR_CUDA;
    }
    if (w->op == TT_OP_CONV2D && !w->plan.g.tap_major && !w->plan.g.persistent) {
        // reduction-index table of the applied record: byte offset of (c, r, s) inside the slab, channel counted
        // from 0 (the kernel rebases it per chunk); indices past K point at the last channel, whose products meet
        // zero-filled filter values
        const GemmArgs& g = w->plan.g;
        const int kpad = g.k_tiles * g.tile_k, RS = g.R * g.S;
        std::vector<int> tab((size_t)kpad);
        for (int k = 0; k < kpad; ++k) {
            if (k < g.K) {
                const int c = k / RS, rem = k - c * RS, fr = rem / g.S, fs = rem - fr * g.S;
                tab[k] = 4 * (c * g.slab_chpitch + fr * g.slab_wp + fs);
            } else {
                tab[k] = 4 * ((g.C - 1) * g.slab_chpitch);
            }
        }
        const size_t bytes = (size_t)kpad * 4;
        if (bytes > w->ktab_bytes) {
            if (w->ktab_dev) cudaFree(w->ktab_dev);
            w->ktab_dev = nullptr; w->ktab_bytes = 0;
            if (cudaMalloc(reinterpret_cast<void**>(&w->ktab_dev), bytes) != cudaSuccess) { cudaGetLastError(); return TT_ERR_OOM; }
            w->ktab_bytes = bytes;
        }
        if (cudaMemcpy(w->ktab_dev, tab.data(), bytes, cudaMemcpyHostToDevice) != cudaSuccess) { cudaGetLastError(); return TT_ERR_CUDA; }
    }
    w->tmaps.clear();
    w->repacked_for = nullptr;
    return TT_OK;
}

static tt_status tensor_maps_for(tt_workload* w, const void* a_ptr, const void* b_ptr, const TmapPair** out) {
    for (const TmapPair& e : w->tmaps)
        if (e.a_ptr == a_ptr && e.b_ptr == b_ptr) { *out = &e; return TT_OK; }
    const GemmArgs& g = w->plan.g;
    TmapPair e;
    std::memset(&e, 0, sizeof e);
    e.a_ptr = a_ptr; e.b_ptr = b_ptr;
    // A gathered operand keeps an all-zero map in its parameter slot; the kernel never issues a TMA load on it.
    tt_status st = TT_OK;
    if (g.a_mode == OPM_TMA)
        st = encode_operand(e.a, static_cast<const float*>(a_ptr), g.K, g.M, g.batch, g.a_rs, g.a_bs, g.a_tma_batched != 0,
                            g.atom_k, kHwTileM);
    if (st != TT_OK) return st;
    if (g.b_mode == OPM_TMA)
        st = encode_operand(e.b, static_cast<const float*>(b_ptr), g.K, g.N, g.batch, g.b_rs, g.b_bs, g.b_tma_batched != 0,
                            g.atom_k, g.b_rows_cta);
    if (st != TT_OK) return st;
    if (g.a_mode == OPM_TMA_MN)
        st = encode_operand_mn(e.a, static_cast<const float*>(a_ptr), g.M, g.K, g.batch, g.a_ks, g.a_bs, g.a_tma_batched != 0,
                               kHwTileM, g.tile_k);
    if (st != TT_OK) return st;
    if (g.b_mode == OPM_TMA_MN)
        st = encode_operand_mn(e.b, static_cast<const float*>(b_ptr), g.N, g.K, g.batch, g.b_ks, g.b_bs, g.b_tma_batched != 0,
                               g.b_rows_cta, g.tile_k);
    if (st != TT_OK) return st;
    if (g.slab_tma) {
        const float* img = static_cast<const float*>(g.a_mode == OPM_IM2COL ? a_ptr : b_ptr);
        if ((reinterpret_cast<uintptr_t>(img) & 15u) != 0) return TT_ERR_INVALID_ARG;   // images must be 16-byte aligned
        st = encode_image(e.x, img, g.W, g.H, g.C, g.batch, g.slab_wp, g.slab_in_rows, g.slab_box_ch);
        if (st != TT_OK) return st;
    }
    if (w->tmaps.size() >= 4096) w->tmaps.clear();
    w->tmaps.push_back(e);
    *out = &w->tmaps.back();
    return TT_OK;
}

tt_status launch(tt_workload* w, const tt_tensors* t, void* stream) {
    if (!w || !t) return TT_ERR_INVALID_ARG;
    if (!w->plan.applied) return TT_ERR_NOT_APPLIED;
    if (!t->x || !t->y) return TT_ERR_INVALID_ARG;
    if (w->op != TT_OP_SOFTMAX && !t->w) return TT_ERR_INVALID_ARG;
    if (w->sh.has_bias && !t->bias) return TT_ERR_INVALID_ARG;
    if (w->sh.has_residual && !t->residual) return TT_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaSuccess;
    const Plan& p = w->plan;
    if (w->family == TT_FAMILY_GEMM_TC) {
        GemmArgs g = p.g;
        const void* a_ptr = pick(t, p.a_tensor);
        const void* b_ptr = pick(t, p.b_tensor);
        bool repacked_now = false;
        if (p.repack) {
            // tap-major convolution: the filters are brought into [filter][32-channel block][tap][channel] order first.
            // Constant weights (the caller's promise) are re-packed once per weight pointer and applied record.
            if (!(w->constant_weights && w->repacked_for == t->w)) {
                if (launch_repack(static_cast<const float*>(t->w), static_cast<float*>(w->workspace), g.M, g.C, g.R * g.S,
                                  p.repack_cb, st) != cudaSuccess) { cudaGetLastError(); return TT_ERR_CUDA; }
                w->repacked_for = t->w;
                repacked_now = true;
            }
            a_ptr = w->workspace;
        }
        const TmapPair* maps = nullptr;
        tt_status s = tensor_maps_for(w, a_ptr, b_ptr, &maps);
        if (s != TT_OK) return s;
        g.a = static_cast<const float*>(a_ptr);
        g.b = static_cast<const float*>(b_ptr);
        g.y = static_cast<float*>(t->y);
        g.bias = w->sh.has_bias ? static_cast<const float*>(t->bias) : nullptr;
        g.residual = w->sh.has_residual ? static_cast<const float*>(t->residual) : nullptr;
        g.partial = static_cast<float*>(w->workspace);
        g.counters = reinterpret_cast<unsigned*>(static_cast<char*>(w->workspace) + p.partial_bytes);
        g.status = w->status_word;
        if ((reinterpret_cast<uintptr_t>(t->y) & 15u) != 0 ||
            (g.residual && (reinterpret_cast<uintptr_t>(g.residual) & 15u) != 0)) g.vec_store = 0;
        if (g.bias && (reinterpret_cast<uintptr_t>(g.bias) & 15u) == 0) g.vec_store |= 2;
        g.ktab_dev = w->ktab_dev;
        g.wait_ns = w->wait_ns;
        g.extra_tx = w->extra_tx;
        g.w_operand = 0;
        if (w->constant_weights && !repacked_now && !g.persistent && (w->op == TT_OP_DENSE || w->op == TT_OP_CONV2D)) {
            if (p.a_tensor == 1 && g.a_mode == OPM_TMA) g.w_operand = 1;
            else if (p.b_tensor == 1 && g.b_mode == OPM_TMA) g.w_operand = 2;
        }
        e = g.persistent ? launch_gemm_ps(p.info, g, maps->a, maps->b, maps->x, st) : launch_gemm(p.info, g, maps->a, maps->b, maps->x, st);
    } else if (w->family == TT_FAMILY_DW_SIMT) {
        DwArgs d = p.dw;
        d.x = static_cast<const float*>(t->x); d.w = static_cast<const float*>(t->w);
        d.bias = w->sh.has_bias ? static_cast<const float*>(t->bias) : nullptr;
        d.y = static_cast<float*>(t->y);
        if ((reinterpret_cast<uintptr_t>(t->y) & 15u) != 0) d.vec = 1;
        if ((reinterpret_cast<uintptr_t>(t->x) & 15u) != 0) d.vec_in = 0;
        if (d.tma_stages > 0) {
            // the image's tensor map, cached per input pointer like the contraction's maps
            const TmapPair* maps = nullptr;
            for (const TmapPair& m : w->tmaps) if (m.a_ptr == t->x) { maps = &m; break; }
            if (!maps) {
                TmapPair m;
                std::memset(&m, 0, sizeof m);
                m.a_ptr = t->x;
                tt_status s = encode_planes(m.x, d.x, d.W, d.H, (long long)d.N * d.C, d.box_w, d.in_h, d.tile_c);
                if (s != TT_OK) return s;
                if (w->tmaps.size() >= 4096) w->tmaps.clear();
                w->tmaps.push_back(m);
                maps = &w->tmaps.back();
            }
            d.status = w->status_word;
            d.wait_ns = w->wait_ns;
            e = launch_dw_tma(p.info, d, maps->x, st);
        } else
        e = launch_dw(p.info, d, st);
    } else {
        RowArgs r = p.row;
        r.x = static_cast<const float*>(t->x); r.y = static_cast<float*>(t->y);
        if (((reinterpret_cast<uintptr_t>(t->y) | reinterpret_cast<uintptr_t>(t->x)) & 15u) != 0) r.vec = 1;
        e = launch_row(p.info, r, st);
    }
    if (e != cudaSuccess) { cudaGetLastError(); return TT_ERR_CUDA; }
    return TT_OK;
}

static tt_status read_status(tt_workload* w, cudaStream_t st) {
    if (!w->status_word) return TT_ERR_NOT_APPLIED;
    if (cudaStreamSynchronize(st) != cudaSuccess) { cudaGetLastError(); return TT_ERR_CUDA; }
    unsigned v = 0;
    if (cudaMemcpy(&v, w->status_word, 4, cudaMemcpyDeviceToHost) != cudaSuccess) { cudaGetLastError(); return TT_ERR_CUDA; }
    if (v != 0) {
        cudaMemset(w->status_word, 0, 4);
        // A CTA that gave up never reported at its tile's arrival counter: the counters of a workspace split-K record
        // are no longer all zero, and the next run would finish tiles from incomplete partial sums.  Clear them.
        const Plan& p = w->plan;
        if (w->family == TT_FAMILY_GEMM_TC && w->workspace && !p.repack && p.info.workspace_bytes > p.partial_bytes)
            cudaMemset(static_cast<char*>(w->workspace) + p.partial_bytes, 0, (size_t)(p.info.workspace_bytes - p.partial_bytes));
        return (tt_status)(v & 0xffu);
    }
    return TT_OK;
}

static void default_timing(tt_timing_opts* o) {
    if (o->warmup_batches <= 0) o->warmup_batches = 3;
    if (o->batches <= 0) o->batches = 10;
    if (o->min_batch_us <= 0) o->min_batch_us = 200;
    if (o->max_repeats <= 0) o->max_repeats = 4096;
}

static float median_of(std::vector<float>& v, float* q1, float* q3) {
    std::sort(v.begin(), v.end());
    const size_t n = v.size();
    auto at = [&](double pos) {
        const size_t lo = (size_t)pos;
        const size_t hi = std::min(lo + 1, n - 1);
        const double f = pos - (double)lo;
        return (float)(v[lo] * (1.0 - f) + v[hi] * f);
    };
    if (q1) *q1 = at(0.25 * (n - 1));
    if (q3) *q3 = at(0.75 * (n - 1));
    // even count: mean of the two middle order statistics
    return (n & 1) ? v[n / 2] : 0.5f * (v[n / 2 - 1] + v[n / 2]);
}

static tt_status time_applied(tt_workload* w, const tt_tensors* sets, size_t n_sets, cudaStream_t st,
                              const tt_timing_opts* oin, tt_timing* out) {
    tt_timing_opts o{};
    if (oin) o = *oin;
    default_timing(&o);
    if (n_sets == 0) return TT_ERR_INVALID_ARG;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    cudaStream_t cap = nullptr;
    cudaGraph_t graph = nullptr;
    cudaGraphExec_t gexec = nullptr;
    tt_status rc = TT_OK;
    size_t next = 0;
    auto fail = [&](tt_status s) { rc = s; };
    auto run_n = [&](int n, cudaStream_t s) -> tt_status {
        for (int i = 0; i < n; ++i) {
            if (o.floor) {
                // the launch floor of the applied record: an empty kernel with the same launch shape
                for (int l = 0; l < w->plan.info.launches; ++l)
                    if (launch_floor(w->plan.info, w->family == TT_FAMILY_GEMM_TC ? w->plan.g.cluster : 0, s) != cudaSuccess) {
                        cudaGetLastError();
                        return TT_ERR_CUDA;
                    }
                continue;
            }
            tt_status r = launch(w, &sets[next], s);
            next = (next + 1) % n_sets;
            if (r != TT_OK) return r;
        }
        return TT_OK;
    };
    do {
        if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) { fail(TT_ERR_CUDA); break; }
        // first launch alone: surfaces launch errors and a tripped wait before anything is timed
        if ((rc = run_n(1, st)) != TT_OK) break;
        if ((rc = read_status(w, st)) != TT_OK) break;
        // calibrate the number of launches per batch
        float ms = 0.f;
        const int probe = 4;
        cudaEventRecord(e0, st);
        if ((rc = run_n(probe, st)) != TT_OK) break;
        cudaEventRecord(e1, st);
        if (cudaEventSynchronize(e1) != cudaSuccess) { fail(TT_ERR_CUDA); break; }
        cudaEventElapsedTime(&ms, e0, e1);
        const double est_us = std::max(0.2, (double)ms * 1000.0 / probe);
        int reps = (int)std::min<double>((double)o.max_repeats, std::max(1.0, std::ceil(o.min_batch_us / est_us)));
        if (o.use_graph) {
            // one batch = one graph of `reps` launches: no CPU launch gaps between them
            reps = (int)((reps + n_sets - 1) / n_sets * n_sets);      // every replay walks the sets identically
            if (cudaStreamCreateWithFlags(&cap, cudaStreamNonBlocking) != cudaSuccess) { fail(TT_ERR_CUDA); break; }
            // tensor maps must exist before capture (encoding is host work, but keep the capture pure launches)
            if (cudaStreamBeginCapture(cap, cudaStreamCaptureModeThreadLocal) != cudaSuccess) { fail(TT_ERR_CUDA); break; }
            tt_status r = run_n(reps, cap);
            cudaError_t ce = cudaStreamEndCapture(cap, &graph);
            if (r != TT_OK) { fail(r); break; }
            if (ce != cudaSuccess || !graph) { fail(TT_ERR_CUDA); break; }
            if (cudaGraphInstantiate(&gexec, graph, 0) != cudaSuccess) { fail(TT_ERR_CUDA); break; }
        }
        std::vector<float> per;
        per.reserve(o.batches);
        for (int b = 0; b < o.warmup_batches + o.batches; ++b) {
            cudaEventRecord(e0, st);
            if (gexec) {
                if (cudaGraphLaunch(gexec, st) != cudaSuccess) { fail(TT_ERR_CUDA); break; }
            } else if ((rc = run_n(reps, st)) != TT_OK) break;
            cudaEventRecord(e1, st);
            if (cudaEventSynchronize(e1) != cudaSuccess) { fail(TT_ERR_CUDA); break; }
            cudaEventElapsedTime(&ms, e0, e1);
            if (b >= o.warmup_batches) per.push_back(ms * 1000.f / (float)reps);
        }
        if (rc != TT_OK) break;
        if ((rc = read_status(w, st)) != TT_OK) break;
        tt_timing t{};
        t.repeats = reps; t.batches = (int)per.size();
        t.median_us = median_of(per, &t.q1_us, &t.q3_us);
        t.min_us = per.front(); t.max_us = per.back();
        *out = t;
    } while (false);
    if (gexec) cudaGraphExecDestroy(gexec);
    if (graph) cudaGraphDestroy(graph);
    if (cap) cudaStreamDestroy(cap);
    if (e0) cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
    if (rc == TT_ERR_CUDA) cudaGetLastError();
    return rc;
}

static tt_status apply_impl(tt_workload* w, const tt_schedule_record* rec, int mode, int strict_class, tt_apply_info* info) {
    if (!w || !rec) return TT_ERR_INVALID_ARG;
    Plan np;
    tt_status s = legalise(w, rec, mode, strict_class, &np);
    if (info && (s == TT_OK || s == TT_ERR_RESOURCE)) *info = np.info;
    if (s != TT_OK) return s;                     // the previously applied record, if any, stays in force
    Plan old = w->plan;
    w->plan = np;
    s = bind_device(w);
    if (s != TT_OK) { w->plan = old; w->plan.applied = false; return s; }
    w->plan.applied = true;
    return TT_OK;
}

}  // namespace tt

using namespace tt;

extern "C" {

tt_status tt_schedule_apply(tt_workload* w, const tt_schedule_record* rec, tt_apply_info* info_out) {
    return apply_impl(w, rec, TT_MODE_LEGALISE, 0, info_out);
}

tt_status tt_schedule_apply_ex(tt_workload* w, const tt_schedule_record* rec, int32_t mode, int32_t strict_class,
                               tt_apply_info* info_out) {
    if (mode != TT_MODE_LEGALISE && mode != TT_MODE_STRICT) return TT_ERR_INVALID_ARG;
    return apply_impl(w, rec, mode, strict_class, info_out);
}

tt_status tt_run(tt_workload* w, const tt_tensors* t, void* cuda_stream) { return launch(w, t, cuda_stream); }


tt_status tt_workload_set_constant_weights(tt_workload* w, int32_t on) {
    if (!w) return TT_ERR_INVALID_ARG;
    w->constant_weights = on != 0;
    return TT_OK;
}

tt_status tt_workload_set_wait_limit(tt_workload* w, uint64_t nanoseconds) {
    if (!w || nanoseconds == 0) return TT_ERR_INVALID_ARG;
    w->wait_ns = nanoseconds;
    return TT_OK;
}

tt_status tt_workload_test_stall(tt_workload* w, uint32_t extra_bytes) {
    if (!w || (extra_bytes & 15u)) return TT_ERR_INVALID_ARG;
    w->extra_tx = extra_bytes;
    return TT_OK;
}

tt_status tt_workload_status(tt_workload* w, void* cuda_stream) {
    if (!w) return TT_ERR_INVALID_ARG;
    return read_status(w, static_cast<cudaStream_t>(cuda_stream));
}

static tt_status run_host_impl(tt_workload* w, const tt_tensors* host, void* cuda_stream, int64_t* bytes_h2d, int64_t* bytes_d2h,
                               bool synchronise) {
    if (!w || !host) return TT_ERR_INVALID_ARG;
    if (!w->plan.applied) return TT_ERR_NOT_APPLIED;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const void* src[4] = {host->x, host->w, host->bias, host->residual};
    int64_t up = 0;
    for (int i = 0; i < 5; ++i) {
        const size_t bytes = tensor_elems(w, i) * 4;
        if (bytes == 0) continue;
        if (i < 4 && !src[i]) return TT_ERR_INVALID_ARG;
        if (bytes > w->hbytes[i]) {
            if (w->hbuf[i]) cudaFree(w->hbuf[i]);
            w->hbuf[i] = nullptr; w->hbytes[i] = 0;
            if (cudaMalloc(&w->hbuf[i], bytes) != cudaSuccess) { cudaGetLastError(); return TT_ERR_OOM; }
            w->hbytes[i] = bytes;
        }
        if (i < 4) {
            if (cudaMemcpyAsync(w->hbuf[i], src[i], bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) { cudaGetLastError(); return TT_ERR_CUDA; }
            up += (int64_t)bytes;
        }
    }
    if (!host->y) return TT_ERR_INVALID_ARG;
    tt_tensors dev{w->hbuf[0], w->hbuf[1], w->hbuf[2], w->hbuf[3], w->hbuf[4]};
    tt_status s = launch(w, &dev, st);
    if (s != TT_OK) return s;
    const size_t ybytes = tensor_elems(w, 4) * 4;
    if (cudaMemcpyAsync(host->y, w->hbuf[4], ybytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) { cudaGetLastError(); return TT_ERR_CUDA; }
    if (synchronise) s = read_status(w, st);
    if (bytes_h2d) *bytes_h2d = up;
    if (bytes_d2h) *bytes_d2h = (int64_t)ybytes;
    return s;
}

tt_status tt_run_host(tt_workload* w, const tt_tensors* host, void* cuda_stream, int64_t* bytes_h2d, int64_t* bytes_d2h) {
    return run_host_impl(w, host, cuda_stream, bytes_h2d, bytes_d2h, true);
}

tt_status tt_run_host_async(tt_workload* w, const tt_tensors* host, void* cuda_stream, int64_t* bytes_h2d, int64_t* bytes_d2h) {
    return run_host_impl(w, host, cuda_stream, bytes_h2d, bytes_d2h, false);
}

tt_status tt_time(tt_workload* w, const tt_tensors* sets, size_t n_sets, void* cuda_stream, const tt_timing_opts* o,
                  tt_timing* out) {
    if (!w || !sets || !out) return TT_ERR_INVALID_ARG;
    if (!w->plan.applied) return TT_ERR_NOT_APPLIED;
    return time_applied(w, sets, n_sets, static_cast<cudaStream_t>(cuda_stream), o, out);
}

static tt_status transfer_tune_impl(tt_workload* const* wls, const tt_tensors* tensors, const size_t* set_counts, size_t n_wl,
                                    const tt_schedule_record* pool, size_t n_pool, const tt_tune_opts* oin, void* cuda_stream,
                                    tt_tune_result* out);

tt_status tt_transfer_tune(tt_workload* const* wls, const tt_tensors* tensors, size_t n_wl, const tt_schedule_record* pool,
                           size_t n_pool, const tt_tune_opts* oin, void* cuda_stream, tt_tune_result* out) {
    return transfer_tune_impl(wls, tensors, nullptr, n_wl, pool, n_pool, oin, cuda_stream, out);
}

tt_status tt_transfer_tune_sets(tt_workload* const* wls, const tt_tensors* tensors, const size_t* set_counts, size_t n_wl,
                                const tt_schedule_record* pool, size_t n_pool, const tt_tune_opts* oin, void* cuda_stream,
                                tt_tune_result* out) {
    if (!set_counts) return TT_ERR_INVALID_ARG;
    for (size_t i = 0; i < n_wl; ++i) if (set_counts[i] == 0) return TT_ERR_INVALID_ARG;
    return transfer_tune_impl(wls, tensors, set_counts, n_wl, pool, n_pool, oin, cuda_stream, out);
}

static tt_status transfer_tune_impl(tt_workload* const* wls, const tt_tensors* tensors, const size_t* set_counts, size_t n_wl,
                                    const tt_schedule_record* pool, size_t n_pool, const tt_tune_opts* oin, void* cuda_stream,
                                    tt_tune_result* out) {
    if (!wls || !tensors || !out || (n_pool && !pool) || !out->chosen || !out->best_us || !out->times_us || !out->status)
        return TT_ERR_INVALID_ARG;
    tt_tune_opts o{};
    o.include_default = 1;
    if (oin) o = *oin;
    if (!device_present()) return TT_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const auto t_begin = std::chrono::steady_clock::now();
    const size_t n_cols = n_pool + 1;
    int timed = 0, invalid = 0, skipped = 0;
    std::vector<tt_schedule_record> cols(n_cols);
    size_t first_set = 0;
    // pool sub-sampling: the order in which a workload's columns are evaluated -- default first, then the seeded
    // subset, then (only if the subset gained too little over the default) the rest of the pool
    const bool sub = o.subsample_percent > 0 && o.subsample_percent < 100 && n_pool > 1;
    size_t n_first = n_pool;
    std::vector<int32_t> order(n_pool);
    for (size_t j = 0; j < n_pool; ++j) order[j] = (int32_t)j;
    if (sub) {
        n_first = std::max<size_t>(1, (n_pool * (size_t)o.subsample_percent + 99) / 100);
        std::vector<int32_t> firsts(n_first);
        if (tt_pool_subsample(n_pool, n_first, o.subsample_seed, firsts.data()) != TT_OK) return TT_ERR_INVALID_ARG;
        std::vector<char> taken(n_pool, 0);
        size_t k = 0;
        for (int32_t f : firsts) { order[k++] = f; taken[(size_t)f] = 1; }
        for (size_t j = 0; j < n_pool; ++j) if (!taken[j]) order[k++] = (int32_t)j;
    }
    for (size_t i = 0; i < n_wl; ++i) {
        tt_workload* w = wls[i];
        if (!w) return TT_ERR_INVALID_ARG;
        const size_t n_sets = set_counts ? set_counts[i] : 1;
        const tt_tensors* sets = tensors + first_set;
        first_set += n_sets;
        tt_default_schedule(w, &cols[0]);
        for (size_t j = 0; j < n_pool; ++j) cols[j + 1] = pool[j];
        bool stop_early = false;
        float best_first = -1.f;                         // fastest time among the subset's records
        for (size_t step = 0; step < n_cols; ++step) {
            const size_t j = step == 0 ? 0 : (size_t)order[step - 1] + 1;
            float& cell = out->times_us[i * n_cols + j];
            int32_t& cst = out->status[i * n_cols + j];
            cell = -1.f;
            if (sub && step == n_first + 1) {
                // the subset is done: go on only if it did not beat the default record by the asked-for margin
                const float def = out->times_us[i * n_cols];
                stop_early = best_first >= 0.f && def >= 0.f && best_first <= def * (1.f - 0.01f * (float)o.subsample_gain_percent);
            }
            if (stop_early) { cst = TT_SKIPPED; ++skipped; continue; }
            if (j == 0 && !o.include_default) { cst = TT_ERR_INVALID_SCHEDULE; continue; }
            // the default record is the workload's own: never subject to the class rule
            tt_status s = apply_impl(w, &cols[j], j == 0 ? TT_MODE_LEGALISE : o.mode, j == 0 ? 0 : o.strict_class, nullptr);
            if (s == TT_OK) {
                tt_timing tm{};
                s = time_applied(w, sets, n_sets, st, &o.timing, &tm);
                if (s == TT_OK) {
                    cell = tm.median_us; ++timed;
                    if (step >= 1 && step <= n_first && (best_first < 0.f || cell < best_first)) best_first = cell;
                }
            }
            cst = s;
            if (s != TT_OK) {
                if (s == TT_ERR_CUDA || s == TT_ERR_OOM) return s;   // the device is unwell: stop, do not mislabel
                ++invalid;                                          // an invalid pair is a result, not a failure
            }
        }
        tt_select(&out->times_us[i * n_cols], 1, n_cols, &out->chosen[i]);
        const int c = out->chosen[i];
        out->best_us[i] = c >= 0 ? out->times_us[i * n_cols + c] : -1.f;
        if (c >= 0) {
            tt_status s = apply_impl(w, &cols[c], c == 0 ? TT_MODE_LEGALISE : o.mode, c == 0 ? 0 : o.strict_class, nullptr);
            if (s != TT_OK) return s;
        }
    }
    out->pairs_timed = timed; out->pairs_invalid = invalid; out->pairs_skipped = skipped;
    out->search_seconds = std::chrono::duration<double>(std::chrono::steady_clock::now() - t_begin).count();
    return TT_OK;
}

tt_status tt_grid_tune(tt_workload* w, const tt_tensors* t, void* cuda_stream, const tt_timing_opts* o, int32_t level,
                       size_t top_k, tt_schedule_record* out_records, float* out_us, size_t* n_out, int32_t* n_tried) {
    if (!w || !t || !out_records || !out_us || !n_out || top_k == 0) return TT_ERR_INVALID_ARG;
    if (!device_present()) return TT_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    tt_schedule_record base;
    tt_default_schedule(w, &base);
    std::vector<tt_schedule_record> cand;
    auto push = [&](const tt_schedule_record& r) -> bool {
        // keep only records that are legal as written: a record that needs rounding duplicates another candidate
        tt_apply_info info;
        if (tt_schedule_check(w, &r, TT_MODE_LEGALISE, 0, &info) != TT_OK) return false;
        // (a pipeline made shallower to fit short reductions or shared memory is kept: exact duplicates are dropped below)
        if (info.changed & ~(TT_CHG_TILE_M | TT_CHG_STAGES)) return false;      // (includes a reformulated reduction order)
        cand.push_back(info.legal);
        return true;
    };
    const bool full = level > 0;
    if (w->family == TT_FAMILY_GEMM_TC) {
        const std::vector<int> tns = full ? std::vector<int>{16, 32, 48, 64, 96, 128, 192, 256} : std::vector<int>{32, 64, 128, 256};
        const std::vector<int> tks = full ? std::vector<int>{8, 16, 32, 64, 128} : std::vector<int>{32, 64, 128};
        const std::vector<int> sts = full ? std::vector<int>{2, 3, 4, 6, 8} : std::vector<int>{2, 3, 4};
        const std::vector<int> sks = full ? std::vector<int>{1, 2, 3, 4, 5, 6, 7, 8, 12, 16, 24, 32} : std::vector<int>{1, 2, 3, 4, 6, 8};
        const std::vector<int> ras = full ? std::vector<int>{0, 1} : std::vector<int>{0};
        for (int ax : {1, 2}) for (int tn : tns) for (int tk : tks) for (int sg : sts) for (int sk : sks) for (int ra : ras) {
            tt_schedule_record r = base;
            r.mma_m_axis = ax; r.tile_m = kHwTileM; r.tile_n = tn; r.tile_k = tk; r.stages = sg; r.split_k = sk; r.raster = ra;
            push(r);
        }
        // the persistent form (alone and as CTA pairs) and the two-CTAs-per-SM build of the one-tile form; on kernels
        // without them these legalise back and are dropped as duplicates-to-be
        for (int ax : {1, 2}) for (int tn : full ? std::vector<int>{32, 64, 128, 192, 240, 256} : std::vector<int>{64, 128, 256})
            for (int tk : {32, 64}) for (int sg : full ? std::vector<int>{2, 3, 4, 6} : std::vector<int>{2, 4, 6}) for (int cg : {1, 2}) {
                tt_schedule_record r = base;
                r.mma_m_axis = ax; r.tile_m = kHwTileM; r.tile_n = tn; r.tile_k = tk; r.stages = sg; r.split_k = 1; r.raster = 0;
                r.persistent = 1; r.cta_group = cg;
                push(r);
            }
        for (int ax : {1, 2}) for (int tn : {64, 128, 256}) for (int sg : {2, 3}) {
            tt_schedule_record r = base;
            r.mma_m_axis = ax; r.tile_m = kHwTileM; r.tile_n = tn; r.tile_k = 32; r.stages = sg; r.split_k = 1; r.raster = 0;
            r.ctas_per_sm = 2;
            push(r);
        }
        if (w->op == TT_OP_CONV2D) {
            for (int tn : {128, 224, 256}) for (int sg : {2, 4}) {
                tt_schedule_record r = base;
                r.mma_m_axis = 1; r.tile_m = kHwTileM; r.tile_n = tn; r.tile_k = 32; r.stages = sg; r.split_k = 1; r.raster = 0;
                r.k_order = 1; r.persistent = 1;
                push(r);
            }
            // a slab that serves one reduction tile per staging: the smallest shared-memory footprint (two CTAs may
            // then share an SM)
            for (int ax : {1, 2}) for (int tn : full ? std::vector<int>{32, 64, 128, 256} : std::vector<int>{64, 128}) for (int sg : {2, 3}) {
                tt_schedule_record r = base;
                r.mma_m_axis = ax; r.tile_m = kHwTileM; r.tile_n = tn; r.tile_k = 32; r.stages = sg; r.split_k = 1; r.raster = 0;
                r.slab_tiles = 1;
                push(r);
            }
            // the tap-major reduction order (records that ask for it on a kernel that has none are legalised back
            // to the stored order and dropped here as duplicates-to-be)
            for (int tn : full ? std::vector<int>{32, 64, 96, 128, 160, 192, 224, 256} : std::vector<int>{64, 128, 224, 256})
                for (int sg : full ? std::vector<int>{1, 2, 3, 4, 5, 6, 8} : std::vector<int>{2, 3, 5}) {
                    tt_schedule_record r = base;
                    r.mma_m_axis = 1; r.tile_m = kHwTileM; r.tile_n = tn; r.tile_k = 32; r.stages = sg; r.split_k = 1; r.raster = 0;
                    r.k_order = 1;
                    push(r);
                }
        }
    } else if (w->family == TT_FAMILY_DW_SIMT) {
        const std::vector<int> tcs = full ? std::vector<int>{1, 2, 4, 8, 16, 32} : std::vector<int>{1, 4, 16};
        const std::vector<int> bys = full ? std::vector<int>{1, 2, 4, 7, 8, 14, 16, 28} : std::vector<int>{4, 8, 16};
        const std::vector<int> bxs = full ? std::vector<int>{8, 16, 28, 32, 56, 64, 112} : std::vector<int>{16, 32, 64};
        const std::vector<int> its = full ? std::vector<int>{1, 2, 4, 8} : std::vector<int>{1, 4};
        for (int tc : tcs) for (int by : bys) for (int bx : bxs) for (int it : its) for (int vw : {1, 4}) for (int th : {128, 256}) {
            tt_schedule_record r = base;
            r.tile_m = tc; r.block_y = by; r.block_x = bx; r.items_per_thread = it; r.vec_width = vw; r.threads = th;
            r.unroll = 0;                               // staged kernel
            push(r);
        }
        // register-window kernel: rows per thread x CTA tile
        const std::vector<int> wys = full ? std::vector<int>{1, 2, 4, 7, 8, 14, 16, 28, 56} : std::vector<int>{4, 8, 16};
        const std::vector<int> wxs = full ? std::vector<int>{8, 16, 28, 32, 56, 64, 112} : std::vector<int>{16, 32, 64, 112};
        for (int it : {4, 8}) for (int ro : {1, 2, 4}) for (int tc : tcs) for (int by : wys) for (int bx : wxs) for (int th : {64, 128, 256}) {
            if (it == 8 && ro == 4) continue;
            tt_schedule_record r = base;
            r.tile_m = tc; r.block_y = by; r.block_x = bx; r.items_per_thread = it; r.threads = th;
            r.unroll = ro;
            for (int vw : {4, 2, 1}) {                  // the widest store the output rows allow
                r.vec_width = vw;
                if (push(r)) break;
            }
        }
        // TMA-staged persistent kernel (raster = 1): strips of 4 or 8 columns, 1-4 rows; tiles span the image width
        // where they can (a box then needs no columns of a neighbouring tile)
        const std::vector<int> pcs = full ? std::vector<int>{1, 2, 4, 8, 16, 32} : std::vector<int>{2, 4, 8, 16};
        const std::vector<int> pys = full ? std::vector<int>{2, 4, 7, 8, 14, 16, 28, 56} : std::vector<int>{4, 8, 14, 28};
        const std::vector<int> pxs = full ? std::vector<int>{16, 28, 32, 56, 64, 112} : std::vector<int>{32, 56, 112};
        for (int it : full ? std::vector<int>{4, 8} : std::vector<int>{4}) for (int ro : {2, 4}) for (int tc : pcs) for (int by : pys)
            for (int bx : pxs) for (int sg : full ? std::vector<int>{2, 3, 4} : std::vector<int>{2, 3}) {
                if (it == 8 && ro == 4) continue;
                tt_schedule_record r = base;
                r.tile_m = tc; r.block_y = by; r.block_x = bx; r.items_per_thread = it; r.threads = 256;
                r.unroll = ro; r.raster = 1; r.stages = sg;
                for (int vw : {4, 2, 1}) {
                    r.vec_width = vw;
                    if (push(r)) break;
                }
            }
    } else {
        for (int bx : {4, 8, 16, 32}) for (int by : {1, 2, 4, 8, 16}) for (int vw : {1, 2, 4}) {
            tt_schedule_record r = base;
            r.block_x = bx; r.block_y = by; r.vec_width = vw;
            push(r);
        }
    }
    if (cand.empty()) {
        // nothing of the grid fits this shape as written: tune around the legalised default record
        tt_apply_info info;
        if (tt_schedule_check(w, &base, TT_MODE_LEGALISE, 0, &info) == TT_OK) cand.push_back(info.legal);
    }
    // drop exact duplicates (legalisation can map different inputs to one record)
    std::vector<tt_schedule_record> uniq;
    for (const auto& r : cand) {
        bool dup = false;
        for (const auto& u : uniq) if (std::memcmp(&u, &r, sizeof r) == 0) { dup = true; break; }
        if (!dup) uniq.push_back(r);
    }
    std::vector<std::pair<float, size_t>> timed;
    for (size_t i = 0; i < uniq.size(); ++i) {
        tt_status s = apply_impl(w, &uniq[i], TT_MODE_LEGALISE, 0, nullptr);
        if (s == TT_ERR_OOM || s == TT_ERR_CUDA) return s;
        if (s != TT_OK) continue;
        tt_timing tm{};
        s = time_applied(w, t, 1, st, o, &tm);
        if (s == TT_ERR_CUDA || s == TT_ERR_OOM) return s;
        if (s == TT_OK) timed.emplace_back(tm.median_us, i);
    }
    if (n_tried) *n_tried = (int32_t)uniq.size();
    std::stable_sort(timed.begin(), timed.end(), [](const auto& a, const auto& b) { return a.first < b.first; });
    const size_t n = std::min(top_k, timed.size());
    for (size_t i = 0; i < n; ++i) {
        out_records[i] = uniq[timed[i].second];
        out_records[i].origin_op = w->op;
        out_records[i].origin = w->sh;
        out_us[i] = timed[i].first;
    }
    *n_out = n;
    if (n > 0) return apply_impl(w, &out_records[0], TT_MODE_LEGALISE, 0, nullptr);
    return TT_ERR_INVALID_SCHEDULE;
}

namespace {
struct RefineCtx { tt_workload* w; const tt_tensors* t; cudaStream_t st; const tt_timing_opts* o; tt_status fatal; };
float refine_time(void* user, const tt_schedule_record* rec) {
    RefineCtx* c = static_cast<RefineCtx*>(user);
    if (c->fatal != TT_OK) return -1.f;
    tt_status s = tt::apply_impl(c->w, rec, TT_MODE_LEGALISE, 0, nullptr);
    if (s == TT_ERR_OOM || s == TT_ERR_CUDA) { c->fatal = s; return -1.f; }
    if (s != TT_OK) return -1.f;
    tt_timing tm{};
    s = tt::time_applied(c->w, c->t, 1, c->st, c->o, &tm);
    if (s == TT_ERR_OOM || s == TT_ERR_CUDA) { c->fatal = s; return -1.f; }
    return s == TT_OK ? tm.median_us : -1.f;
}
}  // namespace

tt_status tt_refine(tt_workload* w, const tt_tensors* t, void* cuda_stream, const tt_timing_opts* o,
                    const tt_schedule_record* start, int32_t max_rounds, float min_gain, tt_schedule_record* best,
                    float* best_us, float* start_us, int32_t* n_timed) {
    if (!w || !t || !start || !best || !best_us) return TT_ERR_INVALID_ARG;
    if (!device_present()) return TT_ERR_CUDA;
    RefineCtx c{w, t, static_cast<cudaStream_t>(cuda_stream), o, TT_OK};
    const tt_status s = tt_refine_with(w, start, refine_time, &c, max_rounds, min_gain, best, best_us, start_us, n_timed);
    if (c.fatal != TT_OK) return c.fatal;
    if (s != TT_OK) return s;
    return tt::apply_impl(w, best, TT_MODE_LEGALISE, 0, nullptr);
}

}  // extern "C"

// ------------------------------------------------------------------------------------------------------------
// Split-K dense layer for callers that must not allocate device memory.
//
// Some hosts of this library cannot call cudaMalloc at the point where they need a kernel: code running inside
// a memory pool that owns the whole device, a real-time loop that may not take the allocator's lock, a plug-in
// whose host application forbids allocations after start-up.  For them the split-K partial sums, the arrival
// counters and the status word live in one fixed array that is part of the library image: every device that
// loads the library carries it until the process exits.
// ------------------------------------------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_tt_static_scratch[TT_STATIC_SCRATCH_BYTES];

namespace tt {
namespace {
constexpr int kMaxDevices = 64;
constexpr int64_t kStaticStatusBytes = 512;   // the status area, sized like the one tt_schedule_apply allocates
unsigned char* g_scratch_addr[kMaxDevices] = {};

// In host code the array's name only stands for the symbol; the device address is asked for once per device,
// with that device current.
tt_status static_scratch(unsigned char** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { cudaGetLastError(); return TT_ERR_CUDA; }
    if (!g_scratch_addr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_tt_static_scratch) != cudaSuccess || !p) { cudaGetLastError(); return TT_ERR_CUDA; }
        g_scratch_addr[dev] = static_cast<unsigned char*>(p);
    }
    *out = g_scratch_addr[dev];
    return TT_OK;
}
}  // namespace
}  // namespace tt

extern "C" tt_status tt_dense_static_scratch(const void* x, const void* w, const void* bias, void* y, int32_t m,
                                             int32_t nn, int32_t kk, int32_t act, const tt_schedule_record* rec,
                                             void* cuda_stream, int64_t* scratch_bytes_used) {
    if (!x || !w || !y || !rec || m <= 0 || nn <= 0 || kk <= 0 || act < TT_ACT_NONE || act > TT_ACT_GELU_ERF)
        return TT_ERR_INVALID_ARG;
    if (!device_present()) return TT_ERR_CUDA;
    // the kernel description, built in place (no handle is created)
    tt_workload wl;
    wl.op = TT_OP_DENSE;
    std::memset(&wl.sh, 0, sizeof wl.sh);
    wl.sh.batch = 1; wl.sh.m = m; wl.sh.nn = nn; wl.sh.kk = kk; wl.sh.trans_b = 1;
    wl.sh.has_bias = bias != nullptr; wl.sh.act = act;
    wl.family = TT_FAMILY_GEMM_TC;
    wl.P = wl.Q = 0;
    wl.view = tt_gemm_view{1, m, nn, kk, 2.0 * m * (double)nn * kk, 0.0};
    Plan plan;
    tt_schedule_record r1 = *rec;
    r1.persistent = 0; r1.cta_group = 1;        // the one-tile-per-CTA form: the persistent one has no split-K, hence no scratch
    tt_status s = legalise(&wl, &r1, TT_MODE_LEGALISE, 0, &plan);
    if (s != TT_OK) return s;
    // layout of the fixed array: status word | arrival counters | partial sums
    const int64_t counters_bytes = ((int64_t)plan.info.grid_x * plan.info.grid_z * 4 + 255) / 256 * 256;
    const int64_t need = kStaticStatusBytes + counters_bytes + (plan.g.split_k > 1 ? plan.partial_bytes : 0);
    if (scratch_bytes_used) *scratch_bytes_used = need;
    if (need > (int64_t)TT_STATIC_SCRATCH_BYTES) return TT_ERR_RESOURCE;   // this record's partial sums do not fit
    if (plan.g.cluster) {
        // as in tt_schedule_apply: a split-K cluster whose CTAs cannot be resident together is an invalid pair
        int fits = 0;
        if (gemm_cluster_fits(plan.info.smem_bytes, plan.g.cluster, &fits) != cudaSuccess) { cudaGetLastError(); return TT_ERR_CUDA; }
        if (!fits) return TT_ERR_RESOURCE;
    }
    unsigned char* base = nullptr;
    if ((s = static_scratch(&base)) != TT_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    // the array keeps what the previous call left: the status word and the counters must start at zero
    if (cudaMemsetAsync(base, 0, (size_t)(kStaticStatusBytes + counters_bytes), st) != cudaSuccess) { cudaGetLastError(); return TT_ERR_CUDA; }
    GemmArgs g = plan.g;
    const void* tens[2] = {x, w};
    const void* a_ptr = tens[plan.a_tensor];
    const void* b_ptr = tens[plan.b_tensor];
    g.a = static_cast<const float*>(a_ptr);
    g.b = static_cast<const float*>(b_ptr);
    g.y = static_cast<float*>(y);
    g.bias = static_cast<const float*>(bias);
    g.residual = nullptr;
    g.status = reinterpret_cast<unsigned*>(base);
    g.counters = reinterpret_cast<unsigned*>(base + kStaticStatusBytes);
    g.partial = reinterpret_cast<float*>(base + kStaticStatusBytes + counters_bytes);
    g.wait_ns = 1000000000ull;
    g.extra_tx = 0;
    g.w_operand = 0;
    if ((reinterpret_cast<uintptr_t>(y) & 15u) != 0) g.vec_store = 0;
    if (g.bias && (reinterpret_cast<uintptr_t>(g.bias) & 15u) == 0) g.vec_store |= 2;
    TmapPair maps;
    std::memset(&maps, 0, sizeof maps);
    if (g.a_mode == OPM_TMA)
        s = encode_operand(maps.a, g.a, g.K, g.M, g.batch, g.a_rs, g.a_bs, g.a_tma_batched != 0, g.atom_k, kHwTileM);
    if (s == TT_OK && g.b_mode == OPM_TMA)
        s = encode_operand(maps.b, g.b, g.K, g.N, g.batch, g.b_rs, g.b_bs, g.b_tma_batched != 0, g.atom_k, g.tile_n);
    if (s != TT_OK) return s;
    if (launch_gemm(plan.info, g, maps.a, maps.b, maps.x, st) != cudaSuccess) { cudaGetLastError(); return TT_ERR_CUDA; }
    if (cudaStreamSynchronize(st) != cudaSuccess) { cudaGetLastError(); return TT_ERR_CUDA; }
    unsigned v = 0;
    if (cudaMemcpy(&v, base, 4, cudaMemcpyDeviceToHost) != cudaSuccess) { cudaGetLastError(); return TT_ERR_CUDA; }
    return v ? (tt_status)(v & 0xffu) : TT_OK;
}
