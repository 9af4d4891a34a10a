// Device code of libtt for sm_100a: the schedule-parameterised kernel families.
//
//   GEMM_TC  tcgen05.mma kind::tf32, accumulator in tensor memory, operands staged in shared memory by TMA
//            (K-major tensors) or by gather warps (im2col of NCHW activations, strided views), `stages`-deep
//            mbarrier pipeline, bias/activation fused into the accumulator read-out, deterministic split-K.
//   DW_SIMT  depthwise convolution, shared-memory halo tile, fp32 FMA.
//   ROW_SIMT row softmax with sub-warp shuffles.
//
// Every tile size, the pipeline depth, split-K and the tile order are run-time values taken from the applied
// schedule record, so applying a record never recompiles anything.
//
// Every wait on an mbarrier is bounded: when it expires the CTA records TT_ERR_TIMEOUT in the workload's status
// word, all roles leave their loops, tensor memory is released and the kernel returns normally.
#include <cuda_runtime.h>
#include <cuda.h>
#include <cstdint>
#include <cstring>
#include "tt_internal.h"

namespace tt {

// ------------------------------------------------------------------------------------------------------------
// PTX wrappers
// ------------------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok;
}
__device__ __forceinline__ unsigned long long global_timer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

constexpr unsigned long long kWaitLimitNs = 1000000000ull;   // one second per wait, then give up

// Bounded wait.  Returns false when the CTA is aborting (this wait or another one expired).
__device__ __noinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, unsigned* status,
                                       unsigned where) {
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_timer_ns();
    unsigned spins = 0;
    for (;;) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((++spins & 31u) == 0u) {
            if (*abort_flag) return false;
            if (global_timer_ns() - t0 > kWaitLimitNs) {
                *abort_flag = 1;
                atomicCAS(status, 0u, (unsigned)TT_ERR_TIMEOUT | (where << 8));
                return false;
            }
        }
    }
}

__device__ __forceinline__ void fence_proxy_async_shared() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void fence_mbar_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const void* tmap, uint32_t bar, int c0, int c1, int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(tmap), "r"(bar), "r"(c0), "r"(c1), "r"(c2) : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t slot_smem, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot_smem), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]^T, one 128 x N x 8 TF32 step.
__device__ __forceinline__ void mma_tf32(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// Arrive on an mbarrier once every MMA issued so far by this thread has completed.
__device__ __forceinline__ void mma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// 32 lanes x 16 consecutive 32-bit columns: thread i of the warp receives lane (base + i).
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major tile whose rows are `row_bytes` long and hardware-swizzled with
// the span of one row: start address >> 4 in bits 0-13, leading byte offset >> 4 in bits 16-29 (not used by
// swizzled K-major tiles; set to 1), stride byte offset (distance between 8-row groups) >> 4 in bits 32-45,
// constant 0b001 in bits 46-48, swizzle mode in bits 61-63 (2 = 128 B, 4 = 64 B, 6 = 32 B).
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, int row_bytes) {
    const uint64_t swz = row_bytes == 128 ? 2ull : (row_bytes == 64 ? 4ull : 6ull);
    uint64_t d = (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= 1ull << 16;
    d |= (uint64_t)((8u * (uint32_t)row_bytes) >> 4) << 32;
    d |= 1ull << 46;
    d |= swz << 61;
    return d;
}

__device__ __forceinline__ float apply_act(float v, int act) {
    switch (act) {
        case TT_ACT_RELU: return fmaxf(v, 0.f);
        case TT_ACT_RELU6: return fminf(fmaxf(v, 0.f), 6.f);
        case TT_ACT_GELU_ERF: return 0.5f * v * (1.f + erff(v * 0.70710678118654752440f));
        default: return v;
    }
}

// Byte offset of element (row, kk) inside one swizzle atom block of a K-major tile: rows are row_bytes apart
// and the 16-byte chunk index is XORed with bits 7.. of the linear offset (the TMA swizzle patterns).
__device__ __forceinline__ uint32_t swz_off(uint32_t row, uint32_t kbyte, uint32_t row_bytes, uint32_t mask) {
    const uint32_t off = row * row_bytes + kbyte;
    return off ^ (((off >> 7) & mask) << 4);
}

// ------------------------------------------------------------------------------------------------------------
// Gather producers: fill one operand tile of one pipeline stage with generic-proxy stores.
// `rows` tile rows starting at global row row0 (valid below row_extent), reduction indices k0 .. k0 + tile_k.
// ------------------------------------------------------------------------------------------------------------
struct Im2col { int C, H, W, R, S, Q, sh, sw, ph, pw; };

__device__ __forceinline__ void gather_tile(int mode, uint32_t tile_smem, int rows, int row0, int row_extent,
                                            const float* __restrict__ src, long long rs, long long ks,
                                            const Im2col& ic, int k0, int K, int tile_k, int atom_k, int row_bytes,
                                            int swz_mask, int gw, int n_gw, int lane) {
    const uint32_t atom_bytes = (uint32_t)rows * (uint32_t)row_bytes;
    if (mode == OPM_GATHER_K) {
        // lanes walk k (contiguous in memory): 4-byte stores, conflict-free inside a row
        for (int r = gw; r < rows; r += n_gw) {
            const int grow = row0 + r;
            const bool rv = grow < row_extent;
            for (int kk = lane; kk < tile_k; kk += 32) {
                const int k = k0 + kk;
                float v = 0.f;
                if (rv && k < K) v = __ldg(src + (long long)grow * rs + (long long)k * ks);
                const int atom = kk / atom_k, ka = kk - atom * atom_k;
                const uint32_t addr = tile_smem + atom * atom_bytes + swz_off(r, ka * 4, row_bytes, swz_mask);
                asm volatile("st.shared.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
            }
        }
        return;
    }
    // lanes walk rows; each thread assembles 4 consecutive k of its row and writes one 16-byte chunk
    const int row_groups = (rows + 31) >> 5;
    const int k_chunks = tile_k >> 2;
    const int units = row_groups * k_chunks;
    const int RS = ic.R * ic.S;
    for (int u = gw; u < units; u += n_gw) {
        const int rg = u % row_groups, kc = u / row_groups;
        const int r = rg * 32 + lane;
        if (r >= rows) continue;
        const int grow = row0 + r;
        const int kb = k0 + kc * 4;
        float v[4] = {0.f, 0.f, 0.f, 0.f};
        if (grow < row_extent) {
            if (mode == OPM_IM2COL) {
                const int p = grow / ic.Q, q = grow - p * ic.Q;
                const int ih0 = p * ic.sh - ic.ph, iw0 = q * ic.sw - ic.pw;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int k = kb + j;
                    if (k < K) {
                        const int c = k / RS, rs_ = k - c * RS;
                        const int fr = rs_ / ic.S, fs = rs_ - fr * ic.S;
                        const int ih = ih0 + fr, iw = iw0 + fs;
                        if (ih >= 0 && ih < ic.H && iw >= 0 && iw < ic.W)
                            v[j] = __ldg(src + ((long long)c * ic.H + ih) * ic.W + iw);
                    }
                }
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int k = kb + j;
                    if (k < K) v[j] = __ldg(src + (long long)grow * rs + (long long)k * ks);
                }
            }
        }
        const int kk = kc * 4;
        const int atom = kk / atom_k, ka = kk - atom * atom_k;
        const uint32_t addr = tile_smem + atom * atom_bytes + swz_off(r, ka * 4, row_bytes, swz_mask);
        asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]) : "memory");
    }
}

// ------------------------------------------------------------------------------------------------------------
// GEMM_TC kernel.  grid = (tiles_m * tiles_n, split_k, batch), block = 192 threads.
// ------------------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kGemmThreads, 1)
tt_gemm_tc_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b, const GemmArgs g) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t full_bar[kMaxStages];
    __shared__ uint64_t empty_bar[kMaxStages];
    __shared__ uint64_t accum_bar;
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int* abortp = &abort_flag;

    // tile coordinates
    int tm, tn;
    if (g.raster == 0) { tm = blockIdx.x % g.tiles_m; tn = blockIdx.x / g.tiles_m; }
    else               { tn = blockIdx.x % g.tiles_n; tm = blockIdx.x / g.tiles_n; }
    const int m0 = tm * kHwTileM, n0 = tn * g.tile_n;
    const int split = blockIdx.y, bz = blockIdx.z;
    const int kt_begin = split * g.k_tiles_per_split;
    const int kt_end = min(g.k_tiles, kt_begin + g.k_tiles_per_split);
    const int iters = kt_end - kt_begin;

    const uint32_t tiles_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t stage_bytes = g.a_stage_bytes + g.b_stage_bytes;
    const bool a_tma = g.a_mode == OPM_TMA, b_tma = g.b_mode == OPM_TMA;
    const bool any_tma = a_tma || b_tma, any_gather = !a_tma || !b_tma;
    constexpr int kGatherWarps = 4;

    if (threadIdx.x == 0) {
        const uint32_t full_count = (any_tma ? 1u : 0u) + (any_gather ? (uint32_t)kGatherWarps : 0u);
        for (int s = 0; s < g.stages; ++s) {
            mbar_init(smem_u32(&full_bar[s]), full_count);
            mbar_init(smem_u32(&empty_bar[s]), 1u);
        }
        mbar_init(smem_u32(&accum_bar), 1u);
        abort_flag = 0;
        fence_mbar_init();
        fence_proxy_async_shared();
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&tmem_slot), g.tmem_cols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *(volatile uint32_t*)&tmem_slot;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0 && any_tma) {
            int armed = 0;   // stages whose loads were issued
            for (int it = 0; it < iters; ++it) {
                const int s = it % g.stages;
                const uint32_t ph = (uint32_t)(it / g.stages) & 1u;
                if (!mbar_wait(smem_u32(&empty_bar[s]), ph ^ 1u, abortp, g.status, 1u)) break;
                const uint32_t fb = smem_u32(&full_bar[s]);
                mbar_expect_tx(fb, g.tx_bytes);
                const uint32_t a_s = tiles_base + s * stage_bytes, b_s = a_s + g.a_stage_bytes;
                const int k0 = (kt_begin + it) * g.tile_k;
                for (int at = 0; at < g.n_atoms; ++at) {
                    if (a_tma) tma_load_3d(a_s + at * (kHwTileM * g.row_bytes), &tmap_a, fb, k0 + at * g.atom_k, m0, g.a_tma_batched ? bz : 0);
                    if (b_tma) tma_load_3d(b_s + at * (g.tile_n * g.row_bytes), &tmap_b, fb, k0 + at * g.atom_k, n0, g.b_tma_batched ? bz : 0);
                }
                armed = it + 1;
            }
            if (*abortp) {
                // let copies in flight land before shared memory is given back (bounded)
                const int first = max(0, armed - g.stages);
                for (int it = first; it < armed; ++it) {
                    const unsigned long long t0 = global_timer_ns();
                    while (!mbar_try_wait(smem_u32(&full_bar[it % g.stages]), (uint32_t)(it / g.stages) & 1u)) {
                        if (global_timer_ns() - t0 > 2000000ull) break;
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            bool ok = true;
            for (int it = 0; it < iters && ok; ++it) {
                const int s = it % g.stages;
                const uint32_t ph = (uint32_t)(it / g.stages) & 1u;
                if (!mbar_wait(smem_u32(&full_bar[s]), ph, abortp, g.status, 2u)) { ok = false; break; }
                tc_fence_after();
                const uint32_t a_s = tiles_base + s * stage_bytes, b_s = a_s + g.a_stage_bytes;
                const int k8_per_atom = g.atom_k >> 3;
                for (int at = 0; at < g.n_atoms; ++at) {
                    const uint64_t ad = make_desc(a_s + at * (kHwTileM * g.row_bytes), g.row_bytes);
                    const uint64_t bd = make_desc(b_s + at * (g.tile_n * g.row_bytes), g.row_bytes);
                    for (int k8 = 0; k8 < k8_per_atom; ++k8) {
                        // 8 TF32 = 32 bytes further along K inside the swizzle atom: start address + 2 (16-byte units)
                        mma_tf32(tmem_base, ad + (uint64_t)(k8 * 2), bd + (uint64_t)(k8 * 2), g.idesc,
                                 (it > 0 || at > 0 || k8 > 0) ? 1u : 0u);
                    }
                }
                mma_commit(smem_u32(&empty_bar[s]));     // stage reusable once these MMAs have read it
            }
            if (ok) mma_commit(smem_u32(&accum_bar));    // accumulator complete
        }
    } else {
        // ---------------- gather producers, then epilogue ----------------
        const int gw = warp - 2;
        if (any_gather) {
            Im2col ic{g.C, g.H, g.W, g.R, g.S, g.Q, g.sh, g.sw, g.ph, g.pw};
            const float* a_src = g.a + (long long)bz * g.a_bs;
            const float* b_src = g.b + (long long)bz * g.b_bs;
            for (int it = 0; it < iters; ++it) {
                const int s = it % g.stages;
                const uint32_t ph = (uint32_t)(it / g.stages) & 1u;
                if (!mbar_wait(smem_u32(&empty_bar[s]), ph ^ 1u, abortp, g.status, 3u)) break;
                const uint32_t a_s = tiles_base + s * stage_bytes, b_s = a_s + g.a_stage_bytes;
                const int k0 = (kt_begin + it) * g.tile_k;
                if (!a_tma) gather_tile(g.a_mode, a_s, kHwTileM, m0, g.M, a_src, g.a_rs, g.a_ks, ic, k0, g.K, g.tile_k,
                                        g.atom_k, g.row_bytes, g.swz_mask, gw, kGatherWarps, lane);
                if (!b_tma) gather_tile(g.b_mode, b_s, g.tile_n, n0, g.N, b_src, g.b_rs, g.b_ks, ic, k0, g.K, g.tile_k,
                                        g.atom_k, g.row_bytes, g.swz_mask, gw, kGatherWarps, lane);
                fence_proxy_async_shared();              // generic-proxy stores -> visible to the tensor core's reads
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&full_bar[s]));
            }
        }
        // epilogue: warp (warp % 4) owns tensor-memory lanes 32*(warp % 4) .. +31
        const bool have_acc = mbar_wait(smem_u32(&accum_bar), 0u, abortp, g.status, 4u);
        if (have_acc) {
            tc_fence_after();
            const int quad = warp & 3;
            const int m = m0 + quad * 32 + lane;
            const bool m_ok = m < g.M;
            const uint32_t t_row = tmem_base + ((uint32_t)(quad * 32) << 16);
            const bool to_partial = g.split_k > 1;
            float bias_m = 0.f;
            if (!to_partial && g.bias_mode == 1 && m_ok) bias_m = __ldg(g.bias + m);
            float* yrow;
            long long ns;
            if (to_partial) {
                yrow = g.partial + (((long long)split * g.batch + bz) * g.M + m) * (long long)g.N;
                ns = 1;
            } else {
                yrow = g.y + (long long)bz * g.y_bs + (long long)m * g.y_ms;
                ns = g.y_ns;
            }
            const float* rrow = (!to_partial && g.residual) ? g.residual + (long long)bz * g.y_bs + (long long)m * g.y_ms : nullptr;
            const bool vec = to_partial ? ((g.N & 3) == 0) : (g.vec_store != 0);
            for (int c0 = 0; c0 < g.tile_n; c0 += 16) {
                uint32_t r[16];
                tmem_ld16(t_row + (uint32_t)c0, r);
                tmem_wait_ld();
                if (!m_ok) continue;
                const int nb = n0 + c0;
                if (nb >= g.N) continue;
                float v[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) v[j] = __uint_as_float(r[j]);
                if (!to_partial) {
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const int n = nb + j;
                        if (n < g.N) {
                            float t = v[j] + bias_m;
                            if (g.bias_mode == 2) t += __ldg(g.bias + n);
                            if (rrow) t += __ldg(rrow + (long long)n * ns);
                            v[j] = apply_act(t, g.act);
                        }
                    }
                }
                if (vec && nb + 16 <= g.N) {
#pragma unroll
                    for (int j = 0; j < 16; j += 4)
                        *reinterpret_cast<float4*>(yrow + nb + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                } else {
#pragma unroll
                    for (int j = 0; j < 16; ++j)
                        if (nb + j < g.N) yrow[(long long)(nb + j) * ns] = v[j];
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, g.tmem_cols);
    }
}

// ------------------------------------------------------------------------------------------------------------
// Split-K reduction + bias/activation epilogue (fixed summation order: bit-identical from run to run).
// ------------------------------------------------------------------------------------------------------------
__global__ void tt_splitk_reduce_kernel(const ReduceArgs a) {
    const long long per = (long long)a.batch * a.M * a.N;
    const int step = a.vec ? 4 : 1;
    const long long total = per / step;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        const long long e = i * step;
        const int n = (int)(e % a.N);
        const long long bm = e / a.N;
        const int m = (int)(bm % a.M);
        const int b = (int)(bm / a.M);
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        for (int s = 0; s < a.split_k; ++s) {
            const float* p = a.partial + (long long)s * per + e;
            if (a.vec) {
                const float4 t = __ldg(reinterpret_cast<const float4*>(p));
                acc[0] += t.x; acc[1] += t.y; acc[2] += t.z; acc[3] += t.w;
            } else {
                acc[0] += __ldg(p);
            }
        }
        const long long ybase = (long long)b * a.y_bs + (long long)m * a.y_ms;
        const float bm_ = a.bias_mode == 1 ? __ldg(a.bias + m) : 0.f;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (j < step) {
                float t = acc[j] + bm_;
                if (a.bias_mode == 2) t += __ldg(a.bias + n + j);
                if (a.residual) t += __ldg(a.residual + ybase + (long long)(n + j) * a.y_ns);
                acc[j] = apply_act(t, a.act);
            }
        }
        if (a.vec) *reinterpret_cast<float4*>(a.y + ybase + n) = make_float4(acc[0], acc[1], acc[2], acc[3]);
        else a.y[ybase + (long long)n * a.y_ns] = acc[0];
    }
}

// ------------------------------------------------------------------------------------------------------------
// DW_SIMT: depthwise conv + bias + activation.  One CTA = tile_c channels x tile_h x tile_w outputs of one image.
// The input halo tile is staged in shared memory with coalesced row reads; each thread then produces `items`
// consecutive outputs along the width and stores them with vec-wide stores.
// ------------------------------------------------------------------------------------------------------------
__global__ void tt_dwconv_kernel(const DwArgs d) {
    extern __shared__ float dsm[];
    const int n = blockIdx.y;
    int t = blockIdx.x;
    const int tw = t % d.tiles_w; t /= d.tiles_w;
    const int th = t % d.tiles_h; t /= d.tiles_h;
    const int tc = t;
    const int c0 = tc * d.tile_c, p0 = th * d.tile_h, q0 = tw * d.tile_w;
    const int nc = min(d.tile_c, d.C - c0);
    const int in_hw = d.in_h * d.in_w;
    const int RS = d.R * d.S;
    float* s_in = dsm;                                   // [tile_c][in_h][in_w]
    float* s_w = dsm + (size_t)d.tile_c * in_hw;         // [tile_c][R*S]
    float* s_b = s_w + (size_t)d.tile_c * RS;            // [tile_c]
    const int ih0 = p0 * d.sh - d.ph, iw0 = q0 * d.sw - d.pw;

    for (int i = threadIdx.x; i < nc * in_hw; i += blockDim.x) {
        const int c = i / in_hw, rem = i - c * in_hw;
        const int r = rem / d.in_w, col = rem - r * d.in_w;
        const int ih = ih0 + r, iw = iw0 + col;
        float v = 0.f;
        if (ih >= 0 && ih < d.H && iw >= 0 && iw < d.W)
            v = __ldg(d.x + (((long long)n * d.C + c0 + c) * d.H + ih) * d.W + iw);
        s_in[i] = v;
    }
    for (int i = threadIdx.x; i < nc * RS; i += blockDim.x) s_w[i] = __ldg(d.w + (long long)c0 * RS + i);
    for (int i = threadIdx.x; i < nc; i += blockDim.x) s_b[i] = d.bias ? __ldg(d.bias + c0 + i) : 0.f;
    __syncthreads();

    const int groups_w = d.tile_w / d.items;             // tile_w is a multiple of items
    const int work = nc * d.tile_h * groups_w;
    for (int i = threadIdx.x; i < work; i += blockDim.x) {
        const int gwi = i % groups_w;
        const int rest = i / groups_w;
        const int r = rest % d.tile_h, c = rest / d.tile_h;
        const int p = p0 + r, q = q0 + gwi * d.items;
        if (p >= d.P || q >= d.Q) continue;
        float acc[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[j] = s_b[c];
        const float* wi = s_w + c * RS;
        const float* xi = s_in + c * in_hw + (r * d.sh) * d.in_w + gwi * d.items * d.sw;
        for (int fr = 0; fr < d.R; ++fr) {
            for (int fs = 0; fs < d.S; ++fs) {
                const float wv = wi[fr * d.S + fs];
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    if (j < d.items) acc[j] = fmaf(xi[fr * d.in_w + fs + j * d.sw], wv, acc[j]);
            }
        }
        float* yo = d.y + (((long long)n * d.C + c0 + c) * d.P + p) * d.Q + q;
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[j] = apply_act(acc[j], d.act);
        if (d.vec == 4 && q + d.items <= d.Q) {
#pragma unroll
            for (int j = 0; j < 8; j += 4)
                if (j < d.items) *reinterpret_cast<float4*>(yo + j) = make_float4(acc[j], acc[j + 1], acc[j + 2], acc[j + 3]);
        } else if (d.vec == 2 && q + d.items <= d.Q) {
#pragma unroll
            for (int j = 0; j < 8; j += 2)
                if (j < d.items) *reinterpret_cast<float2*>(yo + j) = make_float2(acc[j], acc[j + 1]);
        } else {
#pragma unroll
            for (int j = 0; j < 8; ++j)
                if (j < d.items && q + j < d.Q) yo[j] = acc[j];
        }
    }
}

// ------------------------------------------------------------------------------------------------------------
// ROW_SIMT: softmax(scale * x) per row; `lanes_per_row` threads of one warp share a row.
// ------------------------------------------------------------------------------------------------------------
__global__ void tt_softmax_kernel(const RowArgs a) {
    const int lpr = a.lanes_per_row;
    const int sub = threadIdx.x % lpr;
    const long long row = (long long)blockIdx.x * a.rows_per_cta + threadIdx.x / lpr;
    const bool live = row < a.rows;
    const float* xr = a.x + (live ? row : 0) * (long long)a.cols;
    float* yr = a.y + (live ? row : 0) * (long long)a.cols;
    const int vec = a.vec;
    float mx = -INFINITY;
    if (live) {
        for (int j = sub * vec; j < a.cols; j += lpr * vec)
            for (int e = 0; e < vec; ++e) mx = fmaxf(mx, a.scale * __ldg(xr + j + e));
    }
    for (int o = lpr >> 1; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    float sum = 0.f;
    if (live) {
        for (int j = sub * vec; j < a.cols; j += lpr * vec)
            for (int e = 0; e < vec; ++e) sum += expf(a.scale * __ldg(xr + j + e) - mx);
    }
    for (int o = lpr >> 1; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    if (live) {
        const float inv = 1.f / sum;
        for (int j = sub * vec; j < a.cols; j += lpr * vec) {
            float o4[4];
            for (int e = 0; e < vec; ++e) o4[e] = expf(a.scale * __ldg(xr + j + e) - mx) * inv;
            if (vec == 4) *reinterpret_cast<float4*>(yr + j) = make_float4(o4[0], o4[1], o4[2], o4[3]);
            else if (vec == 2) *reinterpret_cast<float2*>(yr + j) = make_float2(o4[0], o4[1]);
            else yr[j] = o4[0];
        }
    }
}

// ------------------------------------------------------------------------------------------------------------
// Launchers (called from tt_device.cu)
// ------------------------------------------------------------------------------------------------------------
cudaError_t launch_gemm(const tt_apply_info& I, const GemmArgs& g, const ReduceArgs& red, const void* tmap_a,
                        const void* tmap_b, cudaStream_t st) {
    static int attr_set_for = -1;
    int dev = 0;
    cudaGetDevice(&dev);
    if (attr_set_for != dev) {
        cudaError_t e = cudaFuncSetAttribute(tt_gemm_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kDynSmemLimit);
        if (e != cudaSuccess) return e;
        attr_set_for = dev;
    }
    CUtensorMap ta, tb;
    memcpy(&ta, tmap_a, sizeof ta);
    memcpy(&tb, tmap_b, sizeof tb);
    dim3 grid(I.grid_x, I.grid_y, I.grid_z);
    tt_gemm_tc_kernel<<<grid, kGemmThreads, I.smem_bytes, st>>>(ta, tb, g);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    if (g.split_k > 1) {
        const long long total = (long long)red.batch * red.M * red.N / (red.vec ? 4 : 1);
        long long blocks = (total + 255) / 256;
        if (blocks > 148 * 8) blocks = 148 * 8;
        tt_splitk_reduce_kernel<<<(int)blocks, 256, 0, st>>>(red);
        e = cudaGetLastError();
    }
    return e;
}

cudaError_t launch_dw(const tt_apply_info& I, const DwArgs& dw, cudaStream_t st) {
    static int attr_set_for = -1;
    int dev = 0;
    cudaGetDevice(&dev);
    if (attr_set_for != dev) {
        cudaError_t e = cudaFuncSetAttribute(tt_dwconv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kDynSmemLimit);
        if (e != cudaSuccess) return e;
        attr_set_for = dev;
    }
    dim3 grid(I.grid_x, I.grid_y, 1);
    tt_dwconv_kernel<<<grid, I.threads, I.smem_bytes, st>>>(dw);
    return cudaGetLastError();
}

cudaError_t launch_row(const tt_apply_info& I, const RowArgs& row, cudaStream_t st) {
    tt_softmax_kernel<<<I.grid_x, I.threads, 0, st>>>(row);
    return cudaGetLastError();
}

}  // namespace tt
