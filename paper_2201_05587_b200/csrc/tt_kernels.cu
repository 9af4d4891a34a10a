// Device code of libtt for sm_100a: the schedule-parameterised kernel families.
//
//   GEMM_TC  tcgen05.mma kind::tf32, accumulator in tensor memory, `stages`-deep mbarrier pipeline.  Operands reach
//            shared memory by TMA (K-major tensors), by expansion from a slab of input rows that TMA (or cp.async)
//            staged once per CTA (im2col of NCHW activations), or by gathers (strided views).  Bias/activation are
//            fused into the accumulator read-out.  Split-K of 2..8 runs as a thread-block cluster that reduces
//            through distributed shared memory; more splits go through a workspace and the last-arriving CTA adds
//            them up, both in fixed split order.  Launched with programmatic stream serialization.  Built twice:
//            with all registers (one CTA per SM) and capped so that two CTAs share an SM on large grids.
//   DW_SIMT  depthwise convolution, fp32 FMA: a persistent kernel whose tiles' input boxes arrive by TMA (3x3 / 5x5,
//            16-byte image rows), a register-window kernel (3x3 / 5x5) and a shared-memory staged kernel.
//   ROW_SIMT row softmax with sub-warp shuffles, register-resident rows when they fit.
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
#include <algorithm>
#include <utility>
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
// Raise the byte count the barrier's current phase expects, without arriving on it.
__device__ __forceinline__ void mbar_expect_tx_only(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
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
// Non-blocking test of a barrier phase.
__device__ __forceinline__ uint32_t mbar_test_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok;
}
__device__ __forceinline__ unsigned long long global_timer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}



// Bounded wait.  Returns false when the CTA is aborting (this wait or another one expired).
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile int* abort_flag, unsigned* status,
                                            unsigned where, unsigned long long limit_ns) {
    const unsigned long long t0 = global_timer_ns();
    unsigned spins = 0;
    for (;;) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((++spins & 31u) == 0u) {
            if (*abort_flag) return false;
            if (global_timer_ns() - t0 > limit_ns) {
                *abort_flag = 1;
                atomicCAS(status, 0u, (unsigned)TT_ERR_TIMEOUT | (where << 8));
                return false;
            }
        }
    }
}

__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, unsigned* status,
                                          unsigned where, unsigned long long limit_ns) {
    if (mbar_try_wait(bar, parity)) return true;         // the common case costs one instruction
    return mbar_wait_slow(bar, parity, abort_flag, status, where, limit_ns);
}

// Programmatic dependent launch.  A kernel launched with programmatic stream serialization may become resident while
// its predecessor in the stream is still running; it must wait here before its first access to global memory.  The
// kernel after it is allowed to do the same from this kernel's entry on.  (Without the launch attribute both
// instructions do nothing.)
__device__ __forceinline__ void pdl_allow_next() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait_prev() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// One lane of a converged warp (the same lane every time): it issues the warp's asynchronous instructions.
__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "elect.sync _|p, 0xffffffff;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(pred));
    return pred != 0u;
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

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const void* tmap, uint32_t bar, int c0, int c1, int c2, int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst), "l"(tmap), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
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
// All 8-wide reduction steps of one pipeline stage into one accumulator: ATOMS swizzle atoms of K8 steps each.
// Inside an atom a step advances both descriptors by 2 (32 bytes); the next atom starts a_atom / b_atom later.
template <int ATOMS, int K8>
__device__ __forceinline__ void issue_steps(uint32_t d_tmem, uint32_t d_hi, uint32_t a_lo, uint32_t b_lo, uint32_t a_atom,
                                            uint32_t b_atom, uint32_t idesc, uint32_t accumulate) {
#pragma unroll
    for (int at = 0; at < ATOMS; ++at) {
#pragma unroll
        for (int k8 = 0; k8 < K8; ++k8) {
            mma_tf32(d_tmem, ((uint64_t)d_hi << 32) | (uint64_t)(a_lo + (uint32_t)at * a_atom + 2u * (uint32_t)k8),
                     ((uint64_t)d_hi << 32) | (uint64_t)(b_lo + (uint32_t)at * b_atom + 2u * (uint32_t)k8), idesc,
                     (at == 0 && k8 == 0) ? accumulate : 1u);
        }
    }
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

// GELU in its erf form, 0.5 x (1 + erf(x / sqrt 2)).  erf through the rational approximation 7.1.26 of Abramowitz and
// Stegun (absolute error below 1.5e-7, far inside what a TF32 product carries): a dozen instructions instead of
// the library routine's, which matters in a read-out that is a long serial instruction stream per thread.
__device__ __forceinline__ float gelu_erf(float x) {
    const float z = fabsf(x) * 0.70710678118654752440f;
    const float t = __fdividef(1.f, fmaf(0.3275911f, z, 1.f));
    float poly = fmaf(1.061405429f, t, -1.453152027f);
    poly = fmaf(poly, t, 1.421413741f);
    poly = fmaf(poly, t, -0.284496736f);
    poly = fmaf(poly, t, 0.254829592f);
    const float erf_abs = 1.f - poly * t * __expf(-z * z);
    return 0.5f * x * (1.f + copysignf(erf_abs, x));
}

__device__ __forceinline__ float apply_act(float v, int act) {
    switch (act) {
        case TT_ACT_RELU: return fmaxf(v, 0.f);
        case TT_ACT_RELU6: return fminf(fmaxf(v, 0.f), 6.f);
        case TT_ACT_GELU_ERF: return gelu_erf(v);
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
// Operand producers that do not go through TMA.
//
// im2col operand of conv2d (rows = output pixels, k = (c, r, s), gathered from an NCHW image).  The input rows a
// CTA's pixels need are staged ONCE per chunk of reduction tiles in a shared-memory slab by cp.async: per
// channel, the rows [ih_lo, ih_lo + in_rows) one after the other, each followed by `gap` zeros, so that the
// left/right padding of a row and rows outside the image read as zero without any test.  A pipeline stage is
// then expanded from the slab: element (pixel, k) sits at rowoff[pixel] + koff[k], two table look-ups, and a
// lane assembles four consecutive k of its pixel and writes one 16-byte chunk of the swizzled K-major tile.
// Global memory is read once per CTA (not once per filter tap), and no load of the main loop waits on DRAM or L2.
//
// Strided views (the NN operand of batch_matmul) and K-contiguous operands with K % 4 != 0 are gathered from
// global memory directly: the 8 gather warps form 1, 2 or 4 groups, group g fills stages g, g + groups, ...
// ------------------------------------------------------------------------------------------------------------
__device__ __forceinline__ void st_shared_v4(uint32_t addr, float a, float b, float c, float d) {
    asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}
__device__ __forceinline__ void st_shared_f32(uint32_t addr, float a) {
    asm volatile("st.shared.f32 [%0], %1;" ::"r"(addr), "f"(a) : "memory");
}
__device__ __forceinline__ void st_shared_u32(uint32_t addr, uint32_t a) {
    asm volatile("st.shared.u32 [%0], %1;" ::"r"(addr), "r"(a) : "memory");
}
__device__ __forceinline__ float ld_shared_f32(uint32_t addr) {
    float v;
    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint32_t ld_shared_u32(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint4 ld_shared_v4u(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ void cp_async_16(uint32_t dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_4(uint32_t dst, const void* src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// Thread-block cluster primitives (split-K over a cluster: the splits of one output tile are the CTAs of a cluster
// and exchange their partial tiles through distributed shared memory).
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
__device__ __forceinline__ uint32_t map_to_peer(uint32_t saddr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
    return r;
}
__device__ __forceinline__ float ld_peer_f32(uint32_t caddr) {
    float v;
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(caddr) : "memory");
    return v;
}
__device__ __forceinline__ void st_peer_v4(uint32_t caddr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(caddr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ void st_peer_u32(uint32_t caddr, uint32_t a) {
    asm volatile("st.shared::cluster.b32 [%0], %1;" ::"r"(caddr), "r"(a) : "memory");
}
__device__ __forceinline__ float4 ld_shared_v4f(uint32_t addr) {
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr) : "memory");
    return v;
}
// Split-K over a cluster.  The output tile is cut into one band per CTA, along the direction in which the output is
// NOT contiguous (bands of rows when outputs are contiguous along columns, bands of columns otherwise).  Every CTA
// first writes its partial tile into its own shared memory (the pipeline buffers, idle by then) in the layout of the
// reduction area, so that a band is one contiguous run of bytes; one thread per peer then sends that peer's band with
// a single bulk copy (cp.async.bulk, shared::cta -> shared::cluster) into the peer's reduction area, which is not part
// of the pipeline buffers (a fast peer cannot disturb a slower one's main loop).  The copy reports its bytes to a
// barrier of the receiving CTA, which expects the bands of all other splits: a CTA starts adding as soon as ITS bands
// have landed, in split order, its own band read from its own staging copy.  Area layout, per source split (the
// CTA's own split has no slot):
//   bands of rows:    [row in band][col], pitch tile_n + 4 floats;   bands of columns: [col in band][row], pitch 128.
constexpr int kRedColPitch = kHwTileM;
// One band of this CTA's staged partial tile -> the same band's slot in a peer's reduction area; the bytes are counted
// on the peer's barrier (both destination addresses are shared::cluster addresses of the same peer).
__device__ __forceinline__ void bulk_copy_to_peer(uint32_t dst_caddr, uint32_t src_saddr, uint32_t bytes, uint32_t bar_caddr) {
    asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst_caddr), "r"(src_saddr), "r"(bytes), "r"(bar_caddr) : "memory");
}
// Wait until every bulk copy this thread issued has been written at its destination.
__device__ __forceinline__ void bulk_copies_done() {
    asm volatile("cp.async.bulk.commit_group;\n\tcp.async.bulk.wait_group 0;" ::: "memory");
}

// All gather threads meet and learn whether every one of them is still healthy (named barrier 1).
__device__ __forceinline__ bool gather_vote(bool ok) {
    uint32_t all;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 q, %1, 0;\n\t"
        "bar.red.and.pred p, 1, %2, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(all) : "r"((uint32_t)ok), "n"(kGatherThreads) : "memory");
    return all != 0u;
}

// n / d for the small ranges of the slab loader: magic = ceil(2^32 / d) is exact while n * d < 2^32; d == 1 has magic 0.
__device__ __forceinline__ int small_div(int n, unsigned magic) { return magic ? (int)__umulhi((unsigned)n, magic) : n; }

// Stage the input rows of channels [c_first, c_first + nch) that this CTA's pixels need into one slab buffer.
// Pieces (16 bytes when the rows allow it, else 4) are dealt round-robin to the gather threads; rows outside the
// image or beyond the CTA's own range are skipped and keep the zeros written at kernel start.
__device__ __forceinline__ void slab_load_chunk(const GemmArgs& g, const float* __restrict__ img, uint32_t buf, int c_first,
                                                int nch, int ih_lo, int in_rows_cta, bool vec16, int gt) {
    const int wpieces = vec16 ? g.W >> 2 : g.W;
    const bool use_magic = vec16 == (g.slab_vec16 != 0);  // the host's magic number is for its own piece width
    if (wpieces <= 16) {
        // short rows (small images): one thread copies a whole row, so the row's address arithmetic is done once
        const int n_rows = nch * g.slab_in_rows;
        for (int row = gt; row < n_rows; row += kGatherThreads) {
            const int cl = small_div(row, g.magic_in_rows);
            const int rl = row - cl * g.slab_in_rows;
            int ih = ih_lo + rl;
            if (g.sh > g.R) {
                const int po = small_div(rl, g.magic_rstep);
                ih = ih_lo + po * g.sh + (rl - po * g.slab_rstep);
            }
            if (rl >= in_rows_cta || (unsigned)ih >= (unsigned)g.H) continue;
            const float* src = img + ((long long)(c_first + cl) * g.H + ih) * g.W;
            const uint32_t dst = buf + 4u * (uint32_t)(cl * g.slab_chpitch + rl * g.slab_wp + g.slab_gap);
            if (vec16) {
                for (int pc = 0; pc < wpieces; ++pc) cp_async_16(dst + 16u * (uint32_t)pc, src + 4 * pc);
            } else {
                for (int pc = 0; pc < wpieces; ++pc) cp_async_4(dst + 4u * (uint32_t)pc, src + pc);
            }
        }
        return;
    }
    const int total = nch * g.slab_in_rows * wpieces;
    for (int idx = gt; idx < total; idx += kGatherThreads) {
        const int t1 = use_magic ? small_div(idx, g.magic_wpieces) : idx / wpieces;
        const int pc = idx - t1 * wpieces;
        const int cl = small_div(t1, g.magic_in_rows);
        const int rl = t1 - cl * g.slab_in_rows;
        // slab row -> image row: consecutive rows when stride <= filter height, else r rows per output row
        int ih = ih_lo + rl;
        if (g.sh > g.R) {
            const int po = small_div(rl, g.magic_rstep);
            ih = ih_lo + po * g.sh + (rl - po * g.slab_rstep);
        }
        if (rl >= in_rows_cta || (unsigned)ih >= (unsigned)g.H) continue;
        const int col = vec16 ? pc << 2 : pc;
        const float* src = img + ((long long)(c_first + cl) * g.H + ih) * g.W + col;
        const uint32_t dst = buf + 4u * (uint32_t)(cl * g.slab_chpitch + rl * g.slab_wp + g.slab_gap + col);
        if (vec16) cp_async_16(dst, src); else cp_async_4(dst, src);
    }
}

// The chunks c0, c0 + step, ... of one tile row per lane, KB at a time, in three rounds without a branch between
// loads: all table entries, all slab values, then the stores (chunks past the tile re-read the last one and are
// not stored).
template <int KB>
__device__ __forceinline__ void expand_chunks(int c0, int step, int n_ch, uint32_t origin, uint32_t ktab_smem, uint32_t dst_row,
                                              uint32_t swz, int atom_shift, int atom_k, uint32_t atom_bytes, bool in_tile) {
    for (; c0 < n_ch; c0 += step * KB) {
        uint4 e[KB];
        float val[KB][4];
#pragma unroll
        for (int b = 0; b < KB; ++b)
            e[b] = ld_shared_v4u(ktab_smem + 16u * (uint32_t)min(c0 + b * step, n_ch - 1));   // same address in every lane
#pragma unroll
        for (int b = 0; b < KB; ++b) {
            val[b][0] = ld_shared_f32(origin + e[b].x);
            val[b][1] = ld_shared_f32(origin + e[b].y);
            val[b][2] = ld_shared_f32(origin + e[b].z);
            val[b][3] = ld_shared_f32(origin + e[b].w);
        }
#pragma unroll
        for (int b = 0; b < KB; ++b) {
            const int ci = c0 + b * step;
            if (ci < n_ch && in_tile) {
                const int kk = ci << 2;
                st_shared_v4(dst_row + (uint32_t)(kk >> atom_shift) * atom_bytes + ((uint32_t)((kk & (atom_k - 1)) << 2) ^ swz),
                             val[b][0], val[b][1], val[b][2], val[b][3]);
            }
        }
    }
}

// What a gather thread needs to expand its share of any stage, worked out once per kernel: which tile row it
// serves, where that row's window starts in a slab channel, where the row lands in a K-major tile, which
// chunks of four reduction indices it takes.
struct ExpandPlan {
    bool fast, in_tile;          // fast: 1, 2, 4 or 8 row blocks, so a warp keeps one row block for the whole kernel
    uint32_t row_origin;         // byte offset of the row's window origin inside a slab channel
    uint32_t dst_row, swz;       // byte offset of the row inside a tile; its swizzle term
    int c0, step, n_ch, mine;    // first chunk, chunk stride, chunks per tile, chunks this warp takes
    int atom_shift, atom_k;
    uint32_t atom_bytes;
};

__device__ __forceinline__ ExpandPlan make_expand_plan(int rows, uint32_t rowoff_smem, int tile_k, int atom_k, int row_bytes,
                                                       int swz_mask, int gw, int lane) {
    ExpandPlan p;
    const int n_rb = (rows + 31) >> 5;
    p.fast = (kGatherWarps % n_rb) == 0;
    p.atom_shift = atom_k == 32 ? 5 : (atom_k == 16 ? 4 : 3);
    p.atom_k = atom_k;
    p.atom_bytes = (uint32_t)rows * (uint32_t)row_bytes;
    p.n_ch = tile_k >> 2;
    const int shift = row_bytes == 128 ? 0 : (row_bytes == 64 ? 1 : 2);
    const int rb = p.fast ? gw % n_rb : 0;
    p.step = p.fast ? kGatherWarps / n_rb : 1;
    p.c0 = p.fast ? gw / n_rb : 0;
    p.mine = (p.n_ch - p.c0 + p.step - 1) / p.step;
    const int row = rb * 32 + lane;
    p.in_tile = row < rows;
    p.row_origin = ld_shared_u32(rowoff_smem + 4u * (uint32_t)(p.in_tile ? row : rows - 1));
    p.dst_row = (uint32_t)row * (uint32_t)row_bytes;
    p.swz = (uint32_t)((row >> shift) & swz_mask) << 4;
    return p;
}

// Expand one pipeline stage of the im2col operand from the slab.  A warp takes (32-row block, 4-wide k chunk)
// tasks gw, gw + 8, ...; the loads of four tasks are issued before the first store.
// rowoff_smem: per tile row, the byte offset of its pixel's window origin inside a channel of the slab;
// ktab_smem: per reduction index of this tile, the byte offset of (channel, tap) relative to that origin.
__device__ __forceinline__ void expand_stage(const ExpandPlan& xp, uint32_t tile_smem, int rows, uint32_t slab, uint32_t rowoff_smem,
                                             uint32_t ktab_smem, int tile_k, int atom_k, int row_bytes, int swz_mask,
                                             int gw, int lane) {
    if (xp.fast) {
        const uint32_t origin = slab + xp.row_origin, dst_row = tile_smem + xp.dst_row;
        if (xp.mine <= 2) expand_chunks<2>(xp.c0, xp.step, xp.n_ch, origin, ktab_smem, dst_row, xp.swz, xp.atom_shift, xp.atom_k, xp.atom_bytes, xp.in_tile);
        else if (xp.mine <= 4) expand_chunks<4>(xp.c0, xp.step, xp.n_ch, origin, ktab_smem, dst_row, xp.swz, xp.atom_shift, xp.atom_k, xp.atom_bytes, xp.in_tile);
        else expand_chunks<8>(xp.c0, xp.step, xp.n_ch, origin, ktab_smem, dst_row, xp.swz, xp.atom_shift, xp.atom_k, xp.atom_bytes, xp.in_tile);
        return;
    }
    const int atom_shift = atom_k == 32 ? 5 : (atom_k == 16 ? 4 : 3);
    const int shift = row_bytes == 128 ? 0 : (row_bytes == 64 ? 1 : 2);
    const uint32_t atom_bytes = (uint32_t)rows * (uint32_t)row_bytes;
    const int n_rb = (rows + 31) >> 5;
    const int n_tasks = n_rb * (tile_k >> 2);
    const uint32_t inv_rb = (65536u + (uint32_t)n_rb - 1u) / (uint32_t)n_rb;     // t / n_rb == (t * inv_rb) >> 16 for small t
    constexpr int kBatch = 4;
    for (int t0 = gw; t0 < n_tasks; t0 += kGatherWarps * kBatch) {
        float val[kBatch][4];
        uint32_t dst[kBatch];
#pragma unroll
        for (int b = 0; b < kBatch; ++b) {
            const int t = t0 + b * kGatherWarps;
            const bool live = t < n_tasks;               // warp-uniform
            const int tt = live ? t : 0;
            const int ci = (int)(((uint32_t)tt * inv_rb) >> 16);
            const int rb = tt - ci * n_rb;
            const int kk = ci << 2;
            const int row = rb * 32 + lane;
            const bool in_tile = live && row < rows;
            dst[b] = in_tile ? tile_smem + (uint32_t)(kk >> atom_shift) * atom_bytes + (uint32_t)row * (uint32_t)row_bytes +
                                   ((uint32_t)((kk & (atom_k - 1)) << 2) ^ ((uint32_t)((row >> shift) & swz_mask) << 4))
                             : 0xffffffffu;
            const uint32_t origin = slab + ld_shared_u32(rowoff_smem + 4u * (uint32_t)(row < rows ? row : rows - 1));
            const uint4 e = ld_shared_v4u(ktab_smem + 16u * (uint32_t)ci);       // same address in every lane
            val[b][0] = ld_shared_f32(origin + e.x);
            val[b][1] = ld_shared_f32(origin + e.y);
            val[b][2] = ld_shared_f32(origin + e.z);
            val[b][3] = ld_shared_f32(origin + e.w);
        }
#pragma unroll
        for (int b = 0; b < kBatch; ++b)
            if (dst[b] != 0xffffffffu) st_shared_v4(dst[b], val[b][0], val[b][1], val[b][2], val[b][3]);
    }
}

// One stage of a strided view whose rows are contiguous across lanes (unit row stride): lanes walk rows
// (coalesced loads), each lane assembles four consecutive reduction indices of its row in registers and writes
// one 16-byte chunk into the swizzled K-major tile.  Loads of eight tasks are issued before the first store.
__device__ __forceinline__ void gather_rows_stage(uint32_t tile_smem, int rows, const float* __restrict__ src,
                                                  long long rs, long long ks, int row0, int row_extent, int k0, int K,
                                                  int tile_k, int atom_k, int row_bytes, int swz_mask, int wig, int wpg,
                                                  int lane) {
    const int atom_shift = atom_k == 32 ? 5 : (atom_k == 16 ? 4 : 3);
    const int shift = row_bytes == 128 ? 0 : (row_bytes == 64 ? 1 : 2);
    const uint32_t atom_bytes = (uint32_t)rows * (uint32_t)row_bytes;
    const int n_rb = (rows + 31) >> 5;
    const int n_ch = tile_k >> 2;
    const int my_ch = (n_ch - wig + wpg - 1) / wpg;      // chunks wig, wig + wpg, ... belong to this warp
    const int n_tasks = my_ch > 0 ? my_ch * n_rb : 0;    // task = (chunk, 32-row block)
    const uint32_t inv_rb = (65536u + (uint32_t)n_rb - 1u) / (uint32_t)n_rb;
    constexpr int kBatch = 8;
    for (int t0 = 0; t0 < n_tasks; t0 += kBatch) {
        float val[kBatch][4];
        uint32_t dst[kBatch];
#pragma unroll
        for (int b = 0; b < kBatch; ++b) {
            const int t = t0 + b;
            const bool live = t < n_tasks;               // warp-uniform
            const int tt = live ? t : 0;
            const int ci = (int)(((uint32_t)tt * inv_rb) >> 16);
            const int rb = tt - ci * n_rb;
            const int kk = (wig + ci * wpg) * 4;
            const int row = rb * 32 + lane;
            const bool in_tile = live && row < rows;
            dst[b] = in_tile ? tile_smem + (uint32_t)(kk >> atom_shift) * atom_bytes + (uint32_t)row * (uint32_t)row_bytes +
                                   ((uint32_t)((kk & (atom_k - 1)) << 2) ^ ((uint32_t)((row >> shift) & swz_mask) << 4))
                             : 0xffffffffu;
            const int grow = row0 + row;
            const bool rv = in_tile && grow < row_extent;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int k = k0 + kk + j;
                val[b][j] = (rv && k < K) ? __ldg(src + (long long)grow * rs + (long long)k * ks) : 0.f;
            }
        }
#pragma unroll
        for (int b = 0; b < kBatch; ++b)
            if (dst[b] != 0xffffffffu) st_shared_v4(dst[b], val[b][0], val[b][1], val[b][2], val[b][3]);
    }
}

// One stage of an operand whose reduction index is contiguous in memory but cannot go through TMA (K % 4 != 0):
// a warp takes rows, its lanes walk k; 4-byte stores stay inside one swizzled row (conflict-free).
__device__ __forceinline__ void gather_k_stage(uint32_t tile_smem, int rows, const float* __restrict__ src, long long rs,
                                               long long ks, int row0, int row_extent, int k0, int K, int tile_k,
                                               int atom_k, int row_bytes, int swz_mask, int wig, int wpg, int lane) {
    const int atom_shift = atom_k == 32 ? 5 : (atom_k == 16 ? 4 : 3);
    const int shift = row_bytes == 128 ? 0 : (row_bytes == 64 ? 1 : 2);
    const uint32_t atom_bytes = (uint32_t)rows * (uint32_t)row_bytes;
    for (int kk = lane; kk < tile_k; kk += 32) {
        const int k = k0 + kk;
        const uint32_t kterm = (uint32_t)(kk >> atom_shift) * atom_bytes;
        const uint32_t kb = (uint32_t)((kk & (atom_k - 1)) << 2);
        for (int r0 = wig; r0 < rows; r0 += wpg * 4) {
            float val[4];
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                const int r = r0 + b * wpg;
                const int grow = row0 + r;
                val[b] = (r < rows && grow < row_extent && k < K) ? __ldg(src + (long long)grow * rs + (long long)k * ks) : 0.f;
            }
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                const int r = r0 + b * wpg;
                if (r < rows)
                    st_shared_f32(tile_smem + kterm + (uint32_t)r * (uint32_t)row_bytes + (kb ^ ((uint32_t)((r >> shift) & swz_mask) << 4)), val[b]);
            }
        }
    }
}

__device__ __forceinline__ void gather_stage(int mode, uint32_t tile_smem, int rows, const float* __restrict__ src,
                                             long long rs, long long ks, int row0, int row_extent, int k0, int K,
                                             int tile_k, int atom_k, int row_bytes, int swz_mask, int wig, int wpg,
                                             int lane) {
    if (mode == OPM_GATHER_ROWS)
        gather_rows_stage(tile_smem, rows, src, rs, ks, row0, row_extent, k0, K, tile_k, atom_k, row_bytes, swz_mask, wig, wpg, lane);
    else
        gather_k_stage(tile_smem, rows, src, rs, ks, row0, row_extent, k0, K, tile_k, atom_k, row_bytes, swz_mask, wig, wpg, lane);
}

// ------------------------------------------------------------------------------------------------------------
// Epilogue helpers
// ------------------------------------------------------------------------------------------------------------
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr) : "memory");
}

constexpr int kStagePitch = 36;                          // floats per staged row: 16-byte accesses stay conflict-free
constexpr int kStageBytesPerWarp = 32 * kStagePitch * 4;

// ReLU, ReLU6 and "none" are one clamp with per-kernel bounds (no branch per element); GELU is a separate path.
struct EpiArgs {
    float* ybase; const float* rbase; long long y_ms, y_ns; int M; float lo, hi; bool gelu, vec;
    int lin_wp, lin_q, lin_p;   // lin_wp > 0: column n is the padded-linear pixel p * lin_wp + q', stored at p * lin_q + q' if q' < lin_q
};

__device__ __forceinline__ float finish_one(float v, const EpiArgs& e) {
    if (e.gelu) return gelu_erf(v);              // uniform per kernel
    return fminf(fmaxf(v, e.lo), e.hi);
}

// Store one 32-row x 32-column block of pre-activation values (bias already added) whose rows are this warp's
// lanes.  Row-major outputs (y_ns == 1) are transposed through the warp's shared-memory staging area so that
// eight lanes write one 128-byte row segment; otherwise lanes are contiguous in memory and each column is one
// coalesced store.  FULL: all 32 rows and 32 columns exist and 16-byte accesses are aligned.
// POST: a residual is added, so the activation runs here, after it; otherwise the values arrive activated.
template <bool FULL, bool POST>
__device__ __forceinline__ void epilogue_block(float (&v)[32], const EpiArgs& e, int m_first, int nb, int cnt,
                                               uint32_t stg, int lane, bool transposed) {
    if (transposed) {
#pragma unroll
        for (int j = 0; j < 32; j += 4) st_shared_v4(stg + (uint32_t)(lane * kStagePitch + j) * 4u, v[j], v[j + 1], v[j + 2], v[j + 3]);
        __syncwarp();
        const int cc = (lane & 7) * 4;
        if (e.lin_wp > 0) {
            // tap-major convolution: column n is the padded-linear pixel p * wp + q'.  A lane's four columns lie in one
            // padded row (wp is a multiple of 4); when Q is one too, all four are outputs or all four fall into the gap.
            const int n = nb + cc;
            const int p = n / e.lin_wp, q = n - p * e.lin_wp;
            const bool col_ok = cc < cnt && q < e.lin_q && p < e.lin_p;
            const int nq = min(4, e.lin_q - q);          // outputs among the four (4 whenever Q is a multiple of 4)
            const long long coff = (long long)p * e.lin_q + q;
#pragma unroll
            for (int itr = 0; itr < 8; ++itr) {
                const int rr = itr * 4 + (lane >> 3);
                const int m = m_first + rr;
                float4 t;
                asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(t.x), "=f"(t.y), "=f"(t.z), "=f"(t.w)
                             : "r"(stg + (uint32_t)(rr * kStagePitch + cc) * 4u));
                if (col_ok && m < e.M) {
                    const long long o = (long long)m * e.y_ms + coff;
                    if (POST) {
                        t.x = finish_one(t.x + __ldg(e.rbase + o), e);
                        if (nq > 1) t.y = finish_one(t.y + __ldg(e.rbase + o + 1), e);
                        if (nq > 2) t.z = finish_one(t.z + __ldg(e.rbase + o + 2), e);
                        if (nq > 3) t.w = finish_one(t.w + __ldg(e.rbase + o + 3), e);
                    }
                    if (e.vec) *reinterpret_cast<float4*>(e.ybase + o) = t;      // (vec implies Q % 4 == 0)
                    else {
                        e.ybase[o] = t.x;
                        if (nq > 1) e.ybase[o + 1] = t.y;
                        if (nq > 2) e.ybase[o + 2] = t.z;
                        if (nq > 3) e.ybase[o + 3] = t.w;
                    }
                }
            }
            __syncwarp();
            return;
        }
#pragma unroll
        for (int itr = 0; itr < 8; ++itr) {
            const int rr = itr * 4 + (lane >> 3);
            const int m = m_first + rr;
            float4 t;
            asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(t.x), "=f"(t.y), "=f"(t.z), "=f"(t.w)
                         : "r"(stg + (uint32_t)(rr * kStagePitch + cc) * 4u));
            const long long o = (long long)m * e.y_ms + nb + cc;
            if (FULL) {
                if (POST) {
                    const float4 r4 = __ldg(reinterpret_cast<const float4*>(e.rbase + o));
                    t.x = finish_one(t.x + r4.x, e); t.y = finish_one(t.y + r4.y, e);
                    t.z = finish_one(t.z + r4.z, e); t.w = finish_one(t.w + r4.w, e);
                }
                *reinterpret_cast<float4*>(e.ybase + o) = t;
            } else {
                const float tv[4] = {t.x, t.y, t.z, t.w};
                const bool row_ok = m < e.M;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const bool ok = row_ok && cc + j < cnt;
                    float out = tv[j];
                    if (POST) out = finish_one(out + (ok ? __ldg(e.rbase + o + j) : 0.f), e);
                    if (ok) e.ybase[o + j] = out;
                }
            }
        }
        __syncwarp();
    } else {
        const int m = m_first + lane;
        const bool row_ok = FULL || m < e.M;
        long long o = (long long)m * e.y_ms + (long long)nb * e.y_ns;
#pragma unroll
        for (int j = 0; j < 32; ++j, o += e.y_ns) {
            const bool ok = row_ok && (FULL || j < cnt);
            float out = v[j];
            if (POST) out = finish_one(out + (ok ? __ldg(e.rbase + o) : 0.f), e);
            if (ok) e.ybase[o] = out;
        }
    }
}

// ------------------------------------------------------------------------------------------------------------
// GEMM_TC kernel.  grid = (tiles_m * tiles_n, split_k, batch), block = 320 threads:
// warp 0 TMA producer, warp 1 MMA issuer + tensor-memory owner, warps 2-9 gather producers, then epilogue.
// Two builds: MIN_CTAS = 1 (all registers), and MIN_CTAS = 2 (registers capped so that two CTAs share an SM when a
// record's shared memory and tensor memory allow it: one CTA's set-up and read-out then overlap the other's main loop).
// ------------------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok;
}
// Bounded wait on a barrier that CTAs of the cluster arrive on (acquire at cluster scope).
__device__ __noinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, volatile int* abort_flag, unsigned* status,
                                               unsigned where, unsigned long long limit_ns) {
    if (mbar_try_wait_cluster(bar, parity)) return true;
    const unsigned long long t0 = global_timer_ns();
    unsigned spins = 0;
    for (;;) {
        if (mbar_try_wait_cluster(bar, parity)) return true;
        if ((++spins & 31u) == 0u) {
            if (*abort_flag) return false;
            if (global_timer_ns() - t0 > limit_ns) {
                *abort_flag = 1;
                atomicCAS(status, 0u, (unsigned)TT_ERR_TIMEOUT | (where << 8));
                return false;
            }
        }
    }
}

// Split-K over a cluster: extent (rows or columns) and bytes of the band of the output tile that split `owner` finishes.
__device__ __forceinline__ int red_band_extent(const GemmArgs& g, int owner) {
    const int whole = g.y_ns == 1 ? kHwTileM : g.tile_n;
    const int per = (whole + g.split_k - 1) / g.split_k;
    return max(0, min(whole, (owner + 1) * per) - owner * per);
}
__device__ __forceinline__ uint32_t red_band_bytes(const GemmArgs& g, int owner) {
    return (uint32_t)red_band_extent(g, owner) * 4u * (uint32_t)(g.y_ns == 1 ? g.tile_n + 4 : kRedColPitch);
}

template <int MIN_CTAS>
__global__ void __launch_bounds__(kGemmThreads, MIN_CTAS)
tt_gemm_tc_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                  const __grid_constant__ CUtensorMap tmap_x, const GemmArgs g) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t full_bar[kMaxStages];
    __shared__ uint64_t empty_bar[kMaxStages];
    __shared__ uint64_t accum_bar;
    __shared__ uint64_t slab_full[2];     // a slab chunk has landed (TMA)
    __shared__ uint64_t slab_empty[2];    // all gather warps are done with a slab buffer
    __shared__ uint64_t pm_full[2];       // tap-major convolution: a pixel-major slab buffer has been written
    __shared__ uint64_t pm_empty[2];      // ... and every multiply-accumulate that reads it has completed
    __shared__ uint64_t red_bar;          // split-K over a cluster: the other splits' bands of this CTA's output have landed
    __shared__ uint64_t lo_bar[kMaxStages];   // error-compensated products: the remainders of a stage's operand tiles are written
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ int last_split_flag;
    __shared__ __align__(16) float s_bias[256];
    __shared__ int s_rowoff[256];

    // the warp index is broadcast from lane 0 so that the compiler knows it is the same in all lanes of a warp and
    // keeps the role loops (addresses, descriptors, counters) on the uniform datapath
    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
    volatile int* abortp = &abort_flag;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the next kernel of the stream may begin its set-up

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
    // (error-compensated products: a stage holds the two operand tiles and, behind them, their remainders)
    const uint32_t lo_off = g.a_stage_bytes + g.b_stage_bytes;
    const uint32_t stage_bytes = g.x3 ? 2u * lo_off : lo_off;
    const bool a_tma = g.a_mode == OPM_TMA, b_tma = g.b_mode == OPM_TMA;
    const bool any_tma = a_tma || b_tma, any_gather = !a_tma || !b_tma;
    const bool im2col = g.a_mode == OPM_IM2COL || g.b_mode == OPM_IM2COL;
    const bool tapm = g.tap_major != 0;               // conv2d, reduction walked by channel block and tap
    const bool slab_tma = (im2col || tapm) && g.slab_tma != 0;
    // im2col geometry of this CTA: first output row of its pixels, the image row its slab starts at, slab chunks
    int ic_p_first = 0, ic_ih_lo = 0, ic_chunks = 0;
    if (im2col) {
        const int row0 = g.a_mode == OPM_IM2COL ? m0 : n0;
        ic_p_first = row0 / g.Q;
        ic_ih_lo = ic_p_first * g.sh - g.ph;
        ic_chunks = (iters + g.slab_tiles - 1) / g.slab_tiles;
    }
    if (tapm) {
        // the tile's columns are padded-linear pixels n = p * wp + q'
        ic_p_first = n0 / g.slab_wp;
        ic_ih_lo = ic_p_first - g.ph;
        ic_chunks = (iters + g.slab_tiles - 1) / g.slab_tiles;
    }
    // gather groups (global gathers only): 4 groups of 2 warps from 4 stages up, 2 groups of 4 warps for 2-3 stages,
    // else one group; the im2col expansion keeps all eight warps on one stage
    const int n_groups = im2col ? 1 : (g.stages >= 4 ? 4 : (g.stages >= 2 ? 2 : 1));
    const int wpg = kGatherWarps / n_groups;

    if (threadIdx.x == 32) {
        // the tensor maps are fetched ahead of their first use (they are kernel parameters: nothing the previous
        // kernel of the stream could still be writing)
        if (g.a_mode == OPM_TMA) asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_a) : "memory");
        if (g.b_mode == OPM_TMA) asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_b) : "memory");
        if (g.slab_tma) asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_x) : "memory");
    }
    if (threadIdx.x == 0) {
        const uint32_t full_count = tapm ? 1u : (any_tma ? 1u : 0u) + (any_gather ? (uint32_t)wpg : 0u);
        for (int s = 0; s < g.stages; ++s) {
            mbar_init(smem_u32(&full_bar[s]), full_count);
            mbar_init(smem_u32(&empty_bar[s]), 1u);
        }
        mbar_init(smem_u32(&accum_bar), 1u);
        if (g.x3) for (int s = 0; s < g.stages; ++s) mbar_init(smem_u32(&lo_bar[s]), (uint32_t)kGatherWarps);
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&slab_full[b]), 1u);
            mbar_init(smem_u32(&slab_empty[b]), (uint32_t)kGatherWarps);
            mbar_init(smem_u32(&pm_full[b]), (uint32_t)kGatherWarps);
            mbar_init(smem_u32(&pm_empty[b]), 1u);
        }
        if (g.cluster) {
            // the bands this CTA finishes arrive from the other splits: rows x (tile_n + 4) or columns x 128 floats each
            mbar_init(smem_u32(&red_bar), 1u);
            mbar_expect_tx(smem_u32(&red_bar), (uint32_t)(g.split_k - 1) * red_band_bytes(g, split));
        }
        abort_flag = 0;
        last_split_flag = 0;
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
    // A CTA's reduction area and its barrier may be used by a peer only once they exist: every thread announces
    // itself here (the barrier above is initialised) and checks, just before the first copy to a peer could be issued,
    // that all peers have done the same.
    if (g.cluster) cluster_arrive();
    // Programmatic dependent launch: everything above (barriers, tensor memory) touched no global memory and may
    // run while the previous kernel of the stream is still draining; from here on its results are needed.  The
    // kernel that follows this one was allowed to start its own set-up at this kernel's entry.  (Without the launch
    // attribute both instructions do nothing.)
    // (The TMA warp waits a little later: it first requests the constant operand's first stages, see below.)
    if (warp != 0) asm volatile("griddepcontrol.wait;" ::: "memory");

    // Warps 0 and 1 run their loops with all 32 lanes: waits, counters and descriptor arithmetic stay
    // warp-uniform, and one elected lane issues the asynchronous instructions.
    if (warp == 0) {
        // ---------------- TMA producer ----------------
        const bool leader = elect_one();                 // this lane arms the barriers and issues every load
        const uint32_t a_atom = (uint32_t)(kHwTileM * g.row_bytes), b_atom = (uint32_t)(g.tile_n * g.row_bytes);
        const int a_bz = g.a_tma_batched ? bz : 0, b_bz = g.b_tma_batched ? bz : 0;
        // Constant operand (the caller promised that the weights are not written by the kernel in front of this one): its
        // tiles for the first pipeline stages are requested before the wait on that kernel, so they stream in while
        // it is still running.  The barrier only learns of the bytes here; the arrival comes with the stage's other operand.
        int n_pref = 0;
        if (g.w_operand) {
            n_pref = min(g.stages, iters);
            if (leader) {
                int kc0 = kt_begin * g.tile_k;
                for (int it = 0; it < n_pref; ++it, kc0 += g.tile_k) {
                    const uint32_t bar = smem_u32(&full_bar[it]);
                    uint32_t dst = tiles_base + (uint32_t)it * stage_bytes + (g.w_operand == 2 ? g.a_stage_bytes : 0u);
                    mbar_expect_tx_only(bar, g.w_operand == 2 ? g.b_stage_bytes : g.a_stage_bytes);
                    int kc = kc0;
#pragma unroll 1
                    for (int at = 0; at < g.n_atoms; ++at, kc += g.atom_k) {
                        if (g.w_operand == 1) { tma_load_3d(dst, &tmap_a, bar, kc, m0, a_bz); dst += a_atom; }
                        else { tma_load_3d(dst, &tmap_b, bar, kc, n0, b_bz); dst += b_atom; }
                    }
                }
            }
            __syncwarp();
        }
        asm volatile("griddepcontrol.wait;" ::: "memory");
        if (any_tma || slab_tma) {
            int armed = n_pref;   // stages whose loads were issued
            uint32_t st = 0, ph = 0;
            const uint32_t full0 = smem_u32(&full_bar[0]), empty0 = smem_u32(&empty_bar[0]);
            int k0 = kt_begin * g.tile_k;
            uint32_t a_stage = tiles_base, full_addr = full0, empty_addr = empty0;
            // conv2d: slab chunk j (the input rows behind reduction tiles j*T .. j*T+T-1) goes to buffer j & 1 as one
            // box that starts `gap` columns left of the image: the zero fill writes gaps and rows outside the image
            const int RS = g.R * g.S, T = g.slab_tiles;
            const uint32_t slab0 = tiles_base + g.slab_off;
            int slab_issued = 0;
            // (the tap-major path has one staging buffer -- it is transposed away at once --, the other two)
            const int sbufs = tapm ? 1 : 2;
            auto issue_chunk = [&](int j) {
                const int b = tapm ? 0 : (j & 1);
                const uint32_t bar = smem_u32(&slab_full[b]);
                mbar_expect_tx(bar, g.slab_box_bytes);
                tma_load_4d(slab0 + (uint32_t)b * g.slab_buf_bytes, &tmap_x, bar, -g.slab_gap, ic_ih_lo,
                            (kt_begin * g.tile_k + j * T * g.tile_k) / RS, bz);
            };
            if (slab_tma) {
                if (leader) { issue_chunk(0); if (sbufs > 1 && ic_chunks > 1) issue_chunk(1); }
                slab_issued = min(ic_chunks, sbufs);
            }
            int next_slab_it = slab_tma ? (slab_issued - 1) * T : 0x7fffffff;   // chunk `slab_issued` is requested when chunk slab_issued-1 starts
            bool ok = true;
            for (int it = 0; it < iters; ++it, k0 += g.tile_k) {
                if (it == next_slab_it) {
                    next_slab_it += T;
                    if (slab_issued < ic_chunks) {
                        // its buffer is free once the gather warps have left chunk slab_issued - 2
                        const int j = slab_issued;
                        const bool freed = tapm ? mbar_wait(smem_u32(&slab_empty[0]), (uint32_t)(j - 1) & 1u, abortp, g.status, 5u, g.wait_ns)
                                                : mbar_wait(smem_u32(&slab_empty[j & 1]), (uint32_t)((j - 2) >> 1) & 1u, abortp, g.status, 5u, g.wait_ns);
                        if (!__all_sync(0xffffffffu, freed)) { ok = false; break; }
                        if (leader) issue_chunk(j);
                        ++slab_issued;
                    }
                }
                if (!any_tma) continue;
                const bool got = mbar_wait(empty_addr, ph ^ 1u, abortp, g.status, 1u, g.wait_ns);
                if (!__all_sync(0xffffffffu, got)) { ok = false; break; }
                if (leader) {
                    // (test facility: split 0 may be told to expect more than arrives, see tt_workload_test_stall)
                    const bool a_here = a_tma && !(it < n_pref && g.w_operand == 1), b_here = b_tma && !(it < n_pref && g.w_operand == 2);
                    mbar_expect_tx(full_addr, (a_here ? g.a_stage_bytes : 0u) + (b_here ? g.b_stage_bytes : 0u) +
                                                  ((it == 0 && split == 0) ? g.extra_tx : 0u));
                    if (a_here) {
                        uint32_t dst = a_stage;
                        int kc = k0;
#pragma unroll 1
                        for (int at = 0; at < g.n_atoms; ++at, dst += a_atom, kc += g.atom_k) tma_load_3d(dst, &tmap_a, full_addr, kc, m0, a_bz);
                    }
                    if (b_here) {
                        uint32_t dst = a_stage + g.a_stage_bytes;
                        int kc = k0;
#pragma unroll 1
                        for (int at = 0; at < g.n_atoms; ++at, dst += b_atom, kc += g.atom_k) tma_load_3d(dst, &tmap_b, full_addr, kc, n0, b_bz);
                    }
                }
                __syncwarp();
                armed = max(armed, it + 1);
                a_stage += stage_bytes; full_addr += 8u; empty_addr += 8u;
                if (++st == (uint32_t)g.stages) { st = 0; ph ^= 1u; a_stage = tiles_base; full_addr = full0; empty_addr = empty0; }
            }
            if ((!ok || *abortp) && lane == 0) {
                // let copies in flight land before shared memory is given back (bounded)
                const int first = max(0, armed - g.stages);
                for (int it = first; it < armed; ++it) {
                    const unsigned long long t0 = global_timer_ns();
                    while (!mbar_try_wait(smem_u32(&full_bar[it % g.stages]), (uint32_t)(it / g.stages) & 1u)) {
                        if (global_timer_ns() - t0 > 2000000ull) break;
                    }
                }
                for (int j = max(0, slab_issued - sbufs); j < slab_issued; ++j) {
                    const unsigned long long t0 = global_timer_ns();
                    while (!mbar_try_wait(smem_u32(&slab_full[tapm ? 0 : (j & 1)]), (uint32_t)(tapm ? j : (j >> 1)) & 1u)) {
                        if (global_timer_ns() - t0 > 2000000ull) break;
                    }
                }
            }
            __syncwarp();
        }
        if (g.cluster) cluster_wait();
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        {
            bool ok = true;
            uint32_t st = 0, ph = 0;
            const uint32_t full0 = smem_u32(&full_bar[0]), empty0 = smem_u32(&empty_bar[0]);
            // descriptors differ only in their 14-bit start-address field: keep the constant upper word, step the
            // lower word by (bytes >> 4) per stage, per atom and per 8-wide K slice
            const uint64_t d0 = make_desc(0u, g.row_bytes);
            const uint32_t d_hi = (uint32_t)(d0 >> 32), d_lo = (uint32_t)d0;
            const uint32_t a_lo0 = d_lo + ((tiles_base & 0x3FFFFu) >> 4);
            const uint32_t b_lo0 = a_lo0 + (g.a_stage_bytes >> 4);
            const uint32_t stage_step = stage_bytes >> 4;
            const uint32_t a_atom = (uint32_t)(kHwTileM * g.row_bytes) >> 4, b_atom = (uint32_t)(g.tile_n * g.row_bytes) >> 4;
            const int k8_per_atom = g.atom_k >> 3;
            const uint32_t a_next_atom = a_atom - 2u * (uint32_t)k8_per_atom, b_next_atom = b_atom - 2u * (uint32_t)k8_per_atom;
            const bool leader = elect_one();             // this lane issues every multiply-accumulate and every commit
            // accumulators: reduction steps are dealt round-robin; an accumulator's first step overwrites
            uint32_t d_tmem = tmem_base;
            const uint32_t d_end = tmem_base + (uint32_t)(g.n_acc * g.tile_n);
            int fresh = g.n_acc;                         // accumulators not written yet
            uint32_t a_stage = a_lo0, b_stage = b_lo0, full_addr = full0, empty_addr = empty0;
            if (tapm) {
                // Tap-major convolution: the B tile of reduction tile `it` = (channel block, tap (r, s)) is the
                // pixel-major slab of that block read from row lin0 + r * wp + s on (128-byte rows, one per
                // padded-linear pixel; the hardware swizzles on absolute addresses, so any start row works).
                const uint32_t pm0 = tiles_base + g.pm_off;
                const int RS = g.R * g.S;
                const int lin0 = (n0 - ic_p_first * g.slab_wp) + g.slab_gap - g.pw;
                int chunk = 0, tap = 0, fr = 0, fs = 0;
                for (int it = 0; it < iters; ++it) {
                    bool got = mbar_wait(full_addr, ph, abortp, g.status, 2u, g.wait_ns);                       // the filter tile
                    if (tap == 0) got = mbar_wait(smem_u32(&pm_full[chunk & 1]), (uint32_t)(chunk >> 1) & 1u, abortp, g.status, 7u, g.wait_ns) && got;
                    if (!__all_sync(0xffffffffu, got)) { ok = false; break; }
                    tc_fence_after();
                    if (leader) {
                        // the stage holds n_atoms taps of this channel block, one 128 x 32 filter atom each
                        uint32_t a_lo = a_stage;
                        int r2 = fr, s2 = fs;
#pragma unroll 1
                        for (int t = 0; t < g.n_atoms; ++t, a_lo += a_atom) {
                            const uint32_t row = (uint32_t)(lin0 + r2 * g.slab_wp + s2);
                            const uint32_t b_lo = d_lo + (((pm0 + (uint32_t)(chunk & 1) * g.pm_buf_bytes + row * 128u) & 0x3FFFFu) >> 4);
                            issue_steps<1, 4>(tmem_base, d_hi, a_lo, b_lo, a_atom, b_atom, g.idesc, (it > 0 || t > 0) ? 1u : 0u);
                            if (++s2 == g.S) { s2 = 0; ++r2; }
                        }
                        mma_commit(empty_addr);                                                  // filter stage reusable
                        if (tap + g.n_atoms == RS) mma_commit(smem_u32(&pm_empty[chunk & 1]));      // slab buffer reusable
                    }
                    __syncwarp();
                    for (int t = 0; t < g.n_atoms; ++t) if (++fs == g.S) { fs = 0; ++fr; }
                    tap += g.n_atoms;
                    if (tap == RS) { tap = 0; fr = 0; fs = 0; ++chunk; }
                    a_stage += stage_step; full_addr += 8u; empty_addr += 8u;
                    if (++st == (uint32_t)g.stages) { st = 0; ph ^= 1u; a_stage = a_lo0; full_addr = full0; empty_addr = empty0; }
                }
            } else
            for (int it = 0; it < iters; ++it) {
                bool got = mbar_wait(full_addr, ph, abortp, g.status, 2u, g.wait_ns);
                if (g.x3) got = mbar_wait(smem_u32(&lo_bar[st]), ph, abortp, g.status, 16u, g.wait_ns) && got;   // the remainders too
                if (!__all_sync(0xffffffffu, got)) { ok = false; break; }
                tc_fence_after();
                if (leader) {
                    // descriptors step by 2 (32 bytes = 8 TF32 along K) inside a swizzle atom, then to the next atom
                    uint32_t a_lo = a_stage, b_lo = b_stage;
                    if (g.n_acc == 1) {
                        // one accumulator: nothing to rotate.  The common tile_k values are unrolled completely, so
                        // that an issue is two additions and the instruction.
                        auto issue_stage = [&](uint32_t a0, uint32_t b0, uint32_t accumulate) {
                            if (g.tile_k == 64) issue_steps<2, 4>(tmem_base, d_hi, a0, b0, a_atom, b_atom, g.idesc, accumulate);
                            else if (g.tile_k == 32) issue_steps<1, 4>(tmem_base, d_hi, a0, b0, a_atom, b_atom, g.idesc, accumulate);
                            else if (g.tile_k == 128) issue_steps<4, 4>(tmem_base, d_hi, a0, b0, a_atom, b_atom, g.idesc, accumulate);
                            else if (g.tile_k == 16) issue_steps<1, 2>(tmem_base, d_hi, a0, b0, a_atom, b_atom, g.idesc, accumulate);
                            else issue_steps<1, 1>(tmem_base, d_hi, a0, b0, a_atom, b_atom, g.idesc, accumulate);
                        };
                        const uint32_t accumulate = it > 0 ? 1u : 0u;
                        if (g.x3) {
                            // the two cross terms first (small), then the product of what the tensor core sees of a and b
                            const uint32_t lo = lo_off >> 4;
                            issue_stage(a_lo + lo, b_lo, accumulate);
                            issue_stage(a_lo, b_lo + lo, 1u);
                            issue_stage(a_lo, b_lo, 1u);
                        } else {
                            issue_stage(a_lo, b_lo, accumulate);
                        }
                    } else
#pragma unroll 1
                    for (int at = 0; at < g.n_atoms; ++at) {
#pragma unroll 4
                        for (int k8 = 0; k8 < k8_per_atom; ++k8) {
                            mma_tf32(d_tmem, ((uint64_t)d_hi << 32) | (uint64_t)a_lo, ((uint64_t)d_hi << 32) | (uint64_t)b_lo, g.idesc,
                                     fresh > 0 ? 0u : 1u);
                            a_lo += 2u; b_lo += 2u;
                            if (fresh > 0) --fresh;
                            d_tmem += (uint32_t)g.tile_n;
                            if (d_tmem == d_end) d_tmem = tmem_base;
                        }
                        a_lo += a_next_atom; b_lo += b_next_atom;
                    }
                    mma_commit(empty_addr);              // stage reusable once these MMAs have read it
                }
                __syncwarp();
                a_stage += stage_step; b_stage += stage_step; full_addr += 8u; empty_addr += 8u;
                if (++st == (uint32_t)g.stages) { st = 0; ph ^= 1u; a_stage = a_lo0; b_stage = b_lo0; full_addr = full0; empty_addr = empty0; }
            }
            if (ok && leader) mma_commit(smem_u32(&accum_bar));    // accumulator complete
            __syncwarp();
        }
        if (g.cluster) cluster_wait();
    } else {
        // ---------------- gather producers, then epilogue ----------------
        const int gw = warp - 2;
        const int gt = (int)threadIdx.x - 64;
        const int quad = warp & 3;                       // tensor-memory lane quadrant this warp may read
        const int m = m0 + quad * 32 + lane;
        // bias is fetched now so that its latency hides behind the main loop
        if (g.bias_mode == 2 && gt < g.tile_n) s_bias[gt] = (n0 + gt < g.N) ? __ldg(g.bias + n0 + gt) : 0.f;
        if (g.bias_mode == 1 && g.cluster && gt < kHwTileM) s_bias[gt] = (m0 + gt < g.M) ? __ldg(g.bias + m0 + gt) : 0.f;   // for the cluster reduction
        const float bias_row = (g.bias_mode == 1 && m < g.M) ? __ldg(g.bias + m) : 0.f;
        if (im2col) {
            // ---- conv2d: slab staging + expansion; all eight warps work on the same stage ----
            const bool on_a = g.a_mode == OPM_IM2COL;
            const int rows = on_a ? kHwTileM : g.tile_n, row0 = on_a ? m0 : n0, ext = on_a ? g.M : g.N;
            const float* img = (on_a ? g.a : g.b) + (long long)bz * (on_a ? g.a_bs : g.b_bs);
            const float* o_src = on_a ? g.b + (long long)bz * g.b_bs : g.a + (long long)bz * g.a_bs;   // the other operand
            const bool o_gather = on_a ? !b_tma : !a_tma;
            const uint32_t ktab = tiles_base + g.ktab_off;
            const uint32_t slab0 = tiles_base + g.slab_off;
            const uint32_t rowoff = smem_u32(s_rowoff);
            const int RS = g.R * g.S, T = g.slab_tiles;
            const int last = min(row0 + rows, ext) - 1;
            const int p_first = ic_p_first, p_last = last / g.Q;
            const int ih_lo = ic_ih_lo;
            const int in_rows_cta = (p_last - p_first) * g.slab_rstep + g.R;
            const int kbeg = kt_begin * g.tile_k;
            const bool vec16 = g.slab_vec16 && ((reinterpret_cast<uintptr_t>(img) & 15u) == 0);
            // per tile row: byte offset of its pixel's window origin inside a slab channel
            if (gt < rows) {
                const int grow = min(row0 + gt, ext - 1);    // rows past the extent repeat the last pixel (never stored)
                const int p = grow / g.Q, q = grow - p * g.Q;
                s_rowoff[gt] = 4 * ((p - p_first) * g.slab_rstep * g.slab_wp + q * g.sw + (g.slab_gap - g.pw));
            }
            // per reduction index of this CTA: byte offset of (c, r, s) inside the slab, channel counted from 0
            // (made by the host when the record was applied); four entries per copy
            for (int i = gt * 4; i < iters * g.tile_k; i += kGatherThreads * 4)
                cp_async_16(ktab + 4u * (uint32_t)i, g.ktab_dev + kbeg + i);
            cp_async_commit();
            // zeros that no copy ever writes: the tail behind each buffer's last row, and, when the gather warps stage
            // the slab themselves, every gap and every row outside the image
            if (slab_tma) {
                const uint32_t tail = 4u * (uint32_t)(g.slab_box_ch * g.slab_chpitch);
                for (int b = 0; b < g.slab_nbuf; ++b)
                    for (uint32_t o = tail + (uint32_t)gt * 4u; o < g.slab_buf_bytes; o += (uint32_t)kGatherThreads * 4u)
                        st_shared_u32(slab0 + (uint32_t)b * g.slab_buf_bytes + o, 0u);
            } else {
                const uint32_t slab_bytes = (uint32_t)g.slab_nbuf * g.slab_buf_bytes;
                for (uint32_t o = (uint32_t)gt * 16u; o < slab_bytes; o += (uint32_t)kGatherThreads * 16u)
                    st_shared_v4(slab0 + o, 0.f, 0.f, 0.f, 0.f);
            }
            bool ok = gather_vote(true);                 // row table and zeros are in place (the k-table may still be in flight)
            const int n_chunks = ic_chunks;
            const ExpandPlan xplan = make_expand_plan(rows, rowoff, g.tile_k, g.atom_k, g.row_bytes, g.swz_mask, gw, lane);   // after the vote: reads s_rowoff
            auto chunk_first_channel = [&](int j) { return (kbeg + j * T * g.tile_k) / RS; };
            auto chunk_load = [&](int j) {               // the gather warps stage chunk j themselves (no TMA)
                const int k_lo = kbeg + j * T * g.tile_k;
                const int k_hi = min(g.K, kbeg + min((j + 1) * T, iters) * g.tile_k);
                if (k_hi > k_lo) {
                    const int c_first = k_lo / RS, c_last = (k_hi - 1) / RS;
                    slab_load_chunk(g, img, slab0 + (uint32_t)(j & 1) * g.slab_buf_bytes, c_first, c_last - c_first + 1, ih_lo,
                                    in_rows_cta, vec16, gt);
                }
                cp_async_commit();
            };
            if (!slab_tma) {
                chunk_load(0);
                if (n_chunks > 1) chunk_load(1);
            }
            const uint32_t full0 = smem_u32(&full_bar[0]), empty0 = smem_u32(&empty_bar[0]);
            uint32_t st = 0, ph = 0;
            for (int j = 0; j < n_chunks; ++j) {
                if (slab_tma) {
                    if (ok && !mbar_wait(smem_u32(&slab_full[j & 1]), (uint32_t)(j >> 1) & 1u, abortp, g.status, 6u, g.wait_ns)) ok = false;
                    if (j == 0) {
                        cp_async_wait<0>();              // the k-table copies of this thread ...
                        ok = gather_vote(ok);            // ... and of every other gather thread have landed
                        if (!ok) break;
                    }
                } else {
                    if (j + 1 < n_chunks) cp_async_wait<1>(); else cp_async_wait<0>();
                    ok = gather_vote(ok);                // every thread's copies of chunk j are visible to all
                    if (!ok) break;
                }
                // table offsets count channels from 0: rebase the buffer by the chunk's first channel
                const uint32_t slab = slab0 + (uint32_t)(j & 1) * g.slab_buf_bytes - 4u * (uint32_t)(chunk_first_channel(j) * g.slab_chpitch);
                const int it_end = min((j + 1) * T, iters);
                for (int it = j * T; it < it_end; ++it) {
                    if (ok && !mbar_wait(empty0 + st * 8u, ph ^ 1u, abortp, g.status, 3u, g.wait_ns)) ok = false;
                    if (ok) {
                        const uint32_t a_s = tiles_base + st * stage_bytes, b_s = a_s + g.a_stage_bytes;
                        const uint32_t kt = ktab + 4u * (uint32_t)(it * g.tile_k);
                        expand_stage(xplan, on_a ? a_s : b_s, rows, slab, rowoff, kt, g.tile_k, g.atom_k, g.row_bytes, g.swz_mask, gw, lane);
                        if (o_gather) {
                            const int k0 = (kt_begin + it) * g.tile_k;
                            if (on_a) gather_stage(g.b_mode, b_s, g.tile_n, o_src, g.b_rs, g.b_ks, n0, g.N, k0, g.K, g.tile_k,
                                                   g.atom_k, g.row_bytes, g.swz_mask, gw, kGatherWarps, lane);
                            else gather_stage(g.a_mode, a_s, kHwTileM, o_src, g.a_rs, g.a_ks, m0, g.M, k0, g.K, g.tile_k,
                                              g.atom_k, g.row_bytes, g.swz_mask, gw, kGatherWarps, lane);
                        }
                        fence_proxy_async_shared();      // generic-proxy stores -> visible to the tensor core's reads
                        __syncwarp();
                        if (lane == 0) mbar_arrive(full0 + st * 8u);
                    }
                    if (++st == (uint32_t)g.stages) { st = 0; ph ^= 1u; }
                }
                if (slab_tma) {
                    // this warp is done with the buffer: the producer may refill it
                    __syncwarp();
                    if (lane == 0 && j + 2 < n_chunks) mbar_arrive(smem_u32(&slab_empty[j & 1]));
                } else if (j + 2 < n_chunks) {
                    ok = gather_vote(ok);                // everyone is done reading this buffer
                    if (!ok) break;
                    chunk_load(j + 2);
                }
            }
            cp_async_wait<0>();
        } else if (tapm) {
            // ---- conv2d, tap-major: transpose every 32-channel block of input rows, once, into a pixel-major slab ----
            // staging buffer (TMA): [32 channels][in_rows][wp] floats; pixel-major slab: one 128-byte row per staged
            // position (32 channels), 16-byte chunks swizzled by the row's absolute address like a TMA 128-byte tile.
            const uint32_t st0 = tiles_base + g.slab_off, pm0 = tiles_base + g.pm_off;
            const int npix = g.slab_in_rows * g.slab_wp;
            // rows a view can touch beyond the transposed range must hold finite numbers: clear both buffers once
            for (uint32_t o = (uint32_t)gt * 16u; o < (uint32_t)g.pm_nbuf * g.pm_buf_bytes; o += (uint32_t)kGatherThreads * 16u)
                st_shared_v4(pm0 + o, 0.f, 0.f, 0.f, 0.f);
            if (g.slab_box_ch < 32)                      // channels beyond the TMA box (which may already be landing) read as zero
                for (uint32_t o = g.slab_box_bytes + (uint32_t)gt * 16u; o < g.slab_buf_bytes; o += (uint32_t)kGatherThreads * 16u)
                    st_shared_v4(st0 + o, 0.f, 0.f, 0.f, 0.f);
            bool ok = gather_vote(true);
            const uint32_t ch_bytes = 4u * (uint32_t)g.slab_chpitch;
            for (int j = 0; j < ic_chunks; ++j) {
                const int b = j & 1;                     // pixel-major buffer; the staging buffer is always the same one
                if (ok && !mbar_wait(smem_u32(&slab_full[0]), (uint32_t)j & 1u, abortp, g.status, 6u, g.wait_ns)) ok = false;
                if (ok && j >= 2 && !mbar_wait(smem_u32(&pm_empty[b]), (uint32_t)((j - 2) >> 1) & 1u, abortp, g.status, 8u, g.wait_ns)) ok = false;
                if (ok) {
                    // warp gw moves channels 4 gw .. 4 gw + 3 of every staged position; lanes walk positions
                    const uint32_t src = st0 + (uint32_t)(4 * gw) * ch_bytes;
                    const uint32_t dst = pm0 + (uint32_t)b * g.pm_buf_bytes;
                    for (int p0 = lane; p0 < npix; p0 += 128) {
                        float v[4][4];
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const int pix = min(p0 + 32 * u, npix - 1);
                            const uint32_t a = src + 4u * (uint32_t)pix;
                            v[u][0] = ld_shared_f32(a);
                            v[u][1] = ld_shared_f32(a + ch_bytes);
                            v[u][2] = ld_shared_f32(a + 2u * ch_bytes);
                            v[u][3] = ld_shared_f32(a + 3u * ch_bytes);
                        }
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const int pix = p0 + 32 * u;
                            if (pix < npix) {
                                const uint32_t rowa = dst + 128u * (uint32_t)pix;
                                st_shared_v4(rowa + ((((uint32_t)gw) ^ ((rowa >> 7) & 7u)) << 4), v[u][0], v[u][1], v[u][2], v[u][3]);
                            }
                        }
                    }
                    fence_proxy_async_shared();          // generic-proxy stores -> visible to the tensor core's reads
                    __syncwarp();
                    if (lane == 0) {
                        mbar_arrive(smem_u32(&pm_full[b]));
                        if (j + 1 < ic_chunks) mbar_arrive(smem_u32(&slab_empty[0]));   // the staging buffer may be refilled
                    }
                }
            }
        } else if (any_gather) {
            const float* a_src = g.a + (long long)bz * g.a_bs;
            const float* b_src = g.b + (long long)bz * g.b_bs;
            const int grp = gw / wpg, wig = gw - grp * wpg;
            const uint32_t full0 = smem_u32(&full_bar[0]), empty0 = smem_u32(&empty_bar[0]);
            int st = grp % g.stages;
            uint32_t ph = (uint32_t)(grp / g.stages) & 1u;
            for (int it = grp; it < iters; it += n_groups) {
                if (!mbar_wait(empty0 + (uint32_t)st * 8u, ph ^ 1u, abortp, g.status, 3u, g.wait_ns)) break;
                const uint32_t a_s = tiles_base + (uint32_t)st * stage_bytes, b_s = a_s + g.a_stage_bytes;
                const int k0 = (kt_begin + it) * g.tile_k;
                if (!a_tma) gather_stage(g.a_mode, a_s, kHwTileM, a_src, g.a_rs, g.a_ks, m0, g.M, k0, g.K, g.tile_k,
                                         g.atom_k, g.row_bytes, g.swz_mask, wig, wpg, lane);
                if (!b_tma) gather_stage(g.b_mode, b_s, g.tile_n, b_src, g.b_rs, g.b_ks, n0, g.N, k0, g.K, g.tile_k,
                                         g.atom_k, g.row_bytes, g.swz_mask, wig, wpg, lane);
                fence_proxy_async_shared();              // generic-proxy stores -> visible to the tensor core's reads
                __syncwarp();
                if (lane == 0) mbar_arrive(full0 + (uint32_t)st * 8u);
                st += n_groups;
                while (st >= g.stages) { st -= g.stages; ph ^= 1u; }
            }
        }
        if (g.x3) {
            // ---- error-compensated products: once a stage's operand tiles have landed, the eight warps write, 16 bytes
            // per thread and step, what the tensor core will NOT see of every value (x minus x truncated to TF32's ten
            // mantissa bits: exact in fp32) into the second half of the stage, in the same swizzled layout ----
            const uint32_t full0 = smem_u32(&full_bar[0]);
            uint32_t st = 0, ph = 0;
            for (int it = 0; it < iters; ++it) {
                if (!mbar_wait(full0 + st * 8u, ph, abortp, g.status, 15u, g.wait_ns)) break;
                const uint32_t hi = tiles_base + st * stage_bytes;
                for (uint32_t off = 16u * (uint32_t)gt; off < lo_off; off += 16u * (uint32_t)kGatherThreads) {
                    const float4 v = ld_shared_v4f(hi + off);
                    st_shared_v4(hi + lo_off + off, v.x - __uint_as_float(__float_as_uint(v.x) & 0xFFFFE000u),
                                 v.y - __uint_as_float(__float_as_uint(v.y) & 0xFFFFE000u),
                                 v.z - __uint_as_float(__float_as_uint(v.z) & 0xFFFFE000u),
                                 v.w - __uint_as_float(__float_as_uint(v.w) & 0xFFFFE000u));
                }
                fence_proxy_async_shared();              // generic-proxy stores -> visible to the tensor core's reads
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&lo_bar[st]));
                if (++st == (uint32_t)g.stages) { st = 0; ph ^= 1u; }
            }
        }
        // split-K over a cluster: everything the reduction needs that does not depend on the accumulator is worked out
        // here, while the main loop is still running (divisions, 64-bit products, first reads of kernel parameters)
        struct {
            int sk, whole, per; uint32_t line, slot, red; bool along_cols, gelu, clamp, vec_ok; int bias_mode;
            float lo, hi; float* ybase; const float* rbase; long long y_ms, y_ns;
        } cr;
        if (g.cluster) {
            cr.sk = g.split_k;
            cr.along_cols = g.y_ns == 1;                                 // bands of rows
            cr.whole = cr.along_cols ? kHwTileM : g.tile_n;
            cr.per = (cr.whole + cr.sk - 1) / cr.sk;                     // lines (rows or columns) per band
            cr.line = 4u * (uint32_t)(cr.along_cols ? g.tile_n + 4 : kRedColPitch);   // bytes per line
            cr.slot = (uint32_t)cr.per * cr.line;                        // bytes between the bands of two consecutive splits
            cr.red = tiles_base + g.red_off;
            cr.ybase = g.y + (long long)bz * g.y_bs;
            cr.rbase = g.residual ? g.residual + (long long)bz * g.y_bs : nullptr;
            cr.lo = g.act == TT_ACT_NONE || g.act == TT_ACT_GELU_ERF ? -INFINITY : 0.f;
            cr.hi = g.act == TT_ACT_RELU6 ? 6.f : INFINITY;
            cr.gelu = g.act == TT_ACT_GELU_ERF; cr.clamp = g.act == TT_ACT_RELU || g.act == TT_ACT_RELU6;
            cr.bias_mode = g.bias_mode; cr.y_ms = g.y_ms; cr.y_ns = g.y_ns;
            const long long lead = cr.along_cols ? g.y_ms : g.y_ns;      // stride of the other output axis
            cr.vec_ok = (lead & 3) == 0 && (g.y_bs & 3) == 0 && (reinterpret_cast<uintptr_t>(cr.ybase) & 15u) == 0 &&
                        (cr.rbase == nullptr || (reinterpret_cast<uintptr_t>(cr.rbase) & 15u) == 0);
            if constexpr (MIN_CTAS == 1) {               // (kept in registers; the register-capped build works them out again)
                int pin = cr.per;
                asm volatile("" : "+r"(pin), "+r"(cr.slot), "+r"(cr.red), "+l"(cr.ybase), "+l"(cr.rbase), "+l"(cr.y_ms), "+l"(cr.y_ns));
                cr.per = pin;
            }
        }
        // epilogue: warp w owns tensor-memory lanes 32*(w % 4) .. +31; the two warps of a lane quadrant take
        // alternate 32-column blocks
        const bool have_acc = mbar_wait(smem_u32(&accum_bar), 0u, abortp, g.status, 4u, g.wait_ns);
        // every epilogue thread takes the same decision (named barrier 1 over the epilogue threads); the barrier
        // also orders the bias staging above against its readers below
        uint32_t all_acc;
        asm volatile(
            "{\n\t.reg .pred p, q;\n\t"
            "setp.ne.u32 q, %1, 0;\n\t"
            "bar.red.and.pred p, 1, %2, q;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(all_acc) : "r"((uint32_t)have_acc), "n"(kGatherThreads) : "memory");
        if (g.cluster) cluster_wait();                   // every peer is set up: its reduction area and barrier may be used
        if (all_acc) {
            tc_fence_after();
            const int half = gw >> 2;
            const bool m_ok = m < g.M;
            const uint32_t t_row = tmem_base + ((uint32_t)(quad * 32) << 16);
            const bool split_mode = g.split_k > 1 && g.cluster == 0;   // splits beyond a cluster go through the workspace
            // a split with fewer reduction steps than accumulators leaves the last ones unwritten
            const int n_acc = min(g.n_acc, iters * (g.tile_k >> 3));
            // split-K workspace [split][batch][N][M]: a column of the tile is contiguous across lanes
            const long long per_split = (long long)g.batch * g.M * (long long)g.N;
            float* pcol = g.partial + (long long)bz * g.M * (long long)g.N + m;
            if (g.cluster) {
                // split-K over a cluster, step 1: this split's partial tile goes to the pipeline buffers (idle: every
                // multiply-accumulate has completed) in the layout of the reduction area, a band being one run of bytes
                const int row = quad * 32 + lane;
                const uint32_t row_dst = tiles_base + 4u * (uint32_t)(g.y_ns == 1 ? row * (g.tile_n + 4) : row);
#pragma unroll 1
                for (int c0 = half * 32; c0 < g.tile_n; c0 += 64) {
                    uint32_t r[32];
                    tmem_ld32(t_row + (uint32_t)c0, r);
                    tmem_wait_ld();
#pragma unroll 1
                    for (int j = 1; j < n_acc; ++j) {        // the other accumulators, in fixed order
                        uint32_t t2[32];
                        tmem_ld32(t_row + (uint32_t)(j * g.tile_n + c0), t2);
                        tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) + __uint_as_float(t2[i]));
                    }
                    if (g.y_ns == 1) {
                        // bands of rows: [row][col], pitch tile_n + 4
                        const uint32_t dst = row_dst + 4u * (uint32_t)c0;
#pragma unroll
                        for (int j = 0; j < 32; j += 4)
                            if (c0 + j < g.tile_n)           // tile_n is a multiple of 16: groups of four are whole
                                st_shared_v4(dst + 4u * (uint32_t)j, __uint_as_float(r[j]), __uint_as_float(r[j + 1]),
                                             __uint_as_float(r[j + 2]), __uint_as_float(r[j + 3]));
                    } else {
                        // bands of columns: [col][row], pitch 128 -- the lanes of a warp write 128 contiguous bytes
                        uint32_t dst = row_dst + 4u * (uint32_t)(c0 * kRedColPitch);
#pragma unroll
                        for (int j = 0; j < 32; ++j, dst += 4u * (uint32_t)kRedColPitch)
                            if (c0 + j < g.tile_n) st_shared_u32(dst, r[j]);
                    }
                }
                fence_proxy_async_shared();              // generic-proxy stores -> visible to the bulk copies below
            } else if (split_mode) {
                // 1. park this split's partial tile in the workspace
                float* pmine = pcol + (long long)split * per_split;
#pragma unroll 1
                for (int c0 = half * 32; c0 < g.tile_n; c0 += 64) {
                    uint32_t r[32];
                    tmem_ld32(t_row + (uint32_t)c0, r);
                    tmem_wait_ld();
#pragma unroll 1
                    for (int j = 1; j < n_acc; ++j) {        // the other accumulators, in fixed order
                        uint32_t t2[32];
                        tmem_ld32(t_row + (uint32_t)(j * g.tile_n + c0), t2);
                        tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) + __uint_as_float(t2[i]));
                    }
                    const int nb = n0 + c0;
                    const int cnt = min(g.N - nb, g.tile_n - c0);
                    if (!m_ok || cnt <= 0) continue;
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (j < cnt) __stcg(pmine + (long long)(nb + j) * g.M, __uint_as_float(r[j]));
                }
                // 2. the split that arrives last at this tile's counter reduces all of them, in split order
                __threadfence();
                asm volatile("bar.sync 1, %0;" ::"n"(kGatherThreads) : "memory");
                if (threadIdx.x == 64) {
                    unsigned* ctr = g.counters + (size_t)bz * gridDim.x + blockIdx.x;
                    const unsigned old = atomicAdd(ctr, 1u);
                    const int last = old == (unsigned)(g.split_k - 1);
                    if (last) *ctr = 0u;                 // all splits have arrived: ready for the next launch
                    last_split_flag = last;
                }
                asm volatile("bar.sync 1, %0;" ::"n"(kGatherThreads) : "memory");
            }
            const bool finish = g.cluster == 0 && (!split_mode || (*(volatile int*)&last_split_flag != 0));
            if (finish) {
                if (split_mode) __threadfence();
                EpiArgs e;
                e.ybase = g.y + (long long)bz * g.y_bs;
                e.rbase = g.residual ? g.residual + (long long)bz * g.y_bs : nullptr;
                e.y_ms = g.y_ms; e.y_ns = g.y_ns; e.M = g.M;
                e.lo = g.act == TT_ACT_NONE || g.act == TT_ACT_GELU_ERF ? -INFINITY : 0.f;
                e.hi = g.act == TT_ACT_RELU6 ? 6.f : INFINITY;
                e.gelu = g.act == TT_ACT_GELU_ERF;
                e.vec = (g.vec_store & 1) != 0;
                e.lin_wp = tapm ? g.slab_wp : 0; e.lin_q = g.Q; e.lin_p = g.Pout;
                const bool transposed = g.y_ns == 1 && g.y_ms != 1;
                const uint32_t stg = tiles_base + (uint32_t)gw * (uint32_t)kStageBytesPerWarp;   // pipeline buffers are idle now
                const int m_first = m0 + quad * 32;
                uint32_t r[32];
                int c0 = half * 32;
                if (!split_mode && c0 < g.tile_n) tmem_ld32(t_row + (uint32_t)c0, r);
#pragma unroll 1
                for (; c0 < g.tile_n; c0 += 64) {
                    float v[32];
                    const int nb = n0 + c0;
                    const int cnt = min(g.N - nb, g.tile_n - c0);
                    if (!split_mode) {
                        // read-out is software-pipelined: the next block's tensor-memory load is in flight while
                        // this block is biased, activated and stored
                        tmem_wait_ld();
#pragma unroll
                        for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]);
#pragma unroll 1
                        for (int a = 1; a < n_acc; ++a) {        // the other accumulators, in fixed order
                            tmem_ld32(t_row + (uint32_t)(a * g.tile_n + c0), r);
                            tmem_wait_ld();
#pragma unroll
                            for (int j = 0; j < 32; ++j) v[j] += __uint_as_float(r[j]);
                        }
                        if (c0 + 64 < g.tile_n) tmem_ld32(t_row + (uint32_t)(c0 + 64), r);
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j) v[j] = 0.f;
                        if (m_ok && cnt > 0) {
#pragma unroll 2
                            for (int sp = 0; sp < g.split_k; ++sp) {
                                const float* ps = pcol + (long long)sp * per_split + (long long)nb * g.M;
#pragma unroll
                                for (int j = 0; j < 32; ++j)
                                    if (j < cnt) v[j] += __ldcg(ps + (long long)j * g.M);
                            }
                        }
                    }
                    if (cnt <= 0) continue;              // warp-uniform
                    if (g.bias_mode == 1) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) v[j] += bias_row;
                    } else if (g.bias_mode == 2) {
#pragma unroll
                        for (int j = 0; j < 32; j += 4) {
                            const float4 b = *reinterpret_cast<const float4*>(s_bias + c0 + j);
                            v[j] += b.x; v[j + 1] += b.y; v[j + 2] += b.z; v[j + 3] += b.w;
                        }
                    }
                    // full blocks take the unguarded path (16-byte accesses need the aligned layout when transposed)
                    const bool full = !tapm && cnt >= 32 && m_first + 32 <= g.M && (e.vec || !transposed);
                    if (e.rbase == nullptr) {
                        // no residual: activate here, once, outside the store loops
                        if (e.gelu) {
#pragma unroll
                            for (int j = 0; j < 32; ++j) v[j] = gelu_erf(v[j]);
                        } else if (g.act != TT_ACT_NONE) {
#pragma unroll
                            for (int j = 0; j < 32; ++j) v[j] = fminf(fmaxf(v[j], e.lo), e.hi);
                        }
                        if (full) epilogue_block<true, false>(v, e, m_first, nb, cnt, stg, lane, transposed);
                        else epilogue_block<false, false>(v, e, m_first, nb, cnt, stg, lane, transposed);
                    } else {
                        if (full) epilogue_block<true, true>(v, e, m_first, nb, cnt, stg, lane, transposed);
                        else epilogue_block<false, true>(v, e, m_first, nb, cnt, stg, lane, transposed);
                    }
                }
            }
        }
        if (g.cluster) {
            // step 2: once every read-out warp has staged its part, one thread per peer sends that peer's band
            asm volatile("bar.sync 1, %0;" ::"n"(kGatherThreads) : "memory");
            if (all_acc && lane == 0 && gw < cr.sk && gw != split) {
                const uint32_t bytes = (uint32_t)max(0, min(cr.whole, (gw + 1) * cr.per) - gw * cr.per) * cr.line;
                if (bytes != 0u) {
                    // (a CTA keeps no slot for its own split: the splits after it move down by one)
                    bulk_copy_to_peer(map_to_peer(cr.red + (uint32_t)(split < gw ? split : split - 1) * cr.slot, (uint32_t)gw),
                                      tiles_base + (uint32_t)gw * cr.slot, bytes, map_to_peer(smem_u32(&red_bar), (uint32_t)gw));
                    bulk_copies_done();                  // (this CTA's shared memory is no longer read, the peer's no longer written)
                }
            }
            __syncwarp();
            cluster_arrive();                            // second round: this warp sends nothing to a peer any more
            // step 3: add up the bands of this CTA once the other splits' copies of them have landed
            const bool landed = __all_sync(0xffffffffu, mbar_wait_cluster(smem_u32(&red_bar), 0u, abortp, g.status, 14u, g.wait_ns));
            // four outputs that are neighbours in memory, first one (mm, nn), `off` bytes into the band: the partial
            // sums of all splits (this split's own from the staging copy, the others' from the reduction area)
            auto load_sums = [&](uint32_t off, float4 (&p)[8]) {
#pragma unroll
                for (int q = 0; q < 8; ++q)
                    if (q < cr.sk) p[q] = ld_shared_v4f((q == split ? tiles_base + (uint32_t)q * cr.slot : cr.red + (uint32_t)(q < split ? q : q - 1) * cr.slot) + off);
            };
            // ... are added in split order, then bias, residual, activation, one 16-byte store
            auto finish4 = [&](const float4 (&p)[8], int mm, int nn, int valid) {
                float4 acc = p[0];
#pragma unroll
                for (int q = 1; q < 8; ++q)
                    if (q < cr.sk) { acc.x += p[q].x; acc.y += p[q].y; acc.z += p[q].z; acc.w += p[q].w; }
                float v[4] = {acc.x, acc.y, acc.z, acc.w};
                const long long o = (long long)mm * cr.y_ms + (long long)nn * cr.y_ns;   // the four are o, o+1, o+2, o+3
                // the tile's bias values were staged in shared memory before the main loop
                if (cr.bias_mode == 1) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) v[i] += s_bias[mm - m0 + (cr.along_cols ? 0 : i)];
                } else if (cr.bias_mode == 2) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) v[i] += s_bias[nn - n0 + (cr.along_cols ? i : 0)];
                }
                if (cr.rbase) {
#pragma unroll
                    for (int i = 0; i < 4; ++i)
                        if (i < valid) v[i] += __ldg(cr.rbase + o + i);
                }
                if (cr.gelu) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) v[i] = gelu_erf(v[i]);
                } else if (cr.clamp) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) v[i] = fminf(fmaxf(v[i], cr.lo), cr.hi);
                }
                if (valid == 4 && cr.vec_ok) *reinterpret_cast<float4*>(cr.ybase + o) = make_float4(v[0], v[1], v[2], v[3]);
                else {
#pragma unroll
                    for (int i = 0; i < 4; ++i)
                        if (i < valid) cr.ybase[o + i] = v[i];
                }
            };
            // a warp takes two lines (rows or columns) of the band at a time, the loads of both under way together (one
            // line in the register-capped build)
            constexpr int kLines = MIN_CTAS == 1 ? 2 : 1;
            if (!landed) {
                // (the wait recorded the time-out; nothing is stored)
            } else if (cr.along_cols) {
                // this CTA's band of rows; the lanes of a warp walk a row's columns four at a time
                const int rows_here = min(min(kHwTileM, (split + 1) * cr.per), g.M - m0) - split * cr.per;
                const int c_end = min(g.tile_n, g.N - n0);
                for (int rl = gw; rl < rows_here; rl += kLines * kGatherWarps) {
                    const bool two = kLines == 2 && rl + kGatherWarps < rows_here;
                    for (int col = lane * 4; col < c_end; col += 128) {
                        float4 pa[8], pb[8];
                        load_sums((uint32_t)rl * cr.line + 4u * (uint32_t)col, pa);
                        if (two) load_sums((uint32_t)(rl + kGatherWarps) * cr.line + 4u * (uint32_t)col, pb);
                        finish4(pa, m0 + split * cr.per + rl, n0 + col, min(4, c_end - col));
                        if (two) finish4(pb, m0 + split * cr.per + rl + kGatherWarps, n0 + col, min(4, c_end - col));
                    }
                }
            } else {
                // this CTA's band of columns; the lanes of a warp walk a column's 128 rows four at a time
                const int cols_here = min(min(g.tile_n, (split + 1) * cr.per), g.N - n0) - split * cr.per;
                const int r_end = min(kHwTileM, g.M - m0);
                if (lane * 4 < r_end)
                    for (int cl = gw; cl < cols_here; cl += kLines * kGatherWarps) {
                        const bool two = kLines == 2 && cl + kGatherWarps < cols_here;
                        float4 pa[8], pb[8];
                        load_sums((uint32_t)cl * cr.line + 16u * (uint32_t)lane, pa);
                        if (two) load_sums((uint32_t)(cl + kGatherWarps) * cr.line + 16u * (uint32_t)lane, pb);
                        finish4(pa, m0 + lane * 4, n0 + split * cr.per + cl, min(4, r_end - lane * 4));
                        if (two) finish4(pb, m0 + lane * 4, n0 + split * cr.per + cl + kGatherWarps, min(4, r_end - lane * 4));
                    }
            }
        }
    }
    if (g.cluster) {
        // Every thread of every CTA of the cluster takes part in both rounds of the cluster barrier, also after a
        // tripped wait: the second round completes when no CTA sends any more, so none leaves while a copy into its
        // shared memory could still be under way.
        if (warp < 2) cluster_arrive();
        cluster_wait();
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
// GEMM_TC, persistent form (record field `persistent` = 1).  grid = resident CTAs; every CTA walks output tiles
// t = unit, unit + units, ... (a unit is a CTA, or a pair of CTAs when CG = 2) with
//   - the operand pipeline running on across tile boundaries (the loads of the next tile are in flight while this
//     tile's last multiply-accumulates run),
//   - TWO accumulators in tensor memory, used alternately: the read-out warps drain tile t (bias, activation,
//     stores) while the MMA warp already accumulates tile t + 1,
//   - barriers and tensor memory set up once per CTA instead of once per tile.
// Operands: K-major tensors arrive by TMA straight into the swizzled pipeline stage.  Operands whose ROW index is
// the contiguous one in memory (the image of a 1x1 convolution: pixels; the second operand of an NN batch_matmul)
// arrive by TMA as [tile_k][rows] boxes in a staging ring and four warps transpose them into the K-major stage
// (kind::tf32 has no MN-major operands on this part).  No split-K, one accumulator per tile.
// Warps: 0 TMA producer, 1 MMA issuer + tensor-memory owner, 2-5 transposers, 6-9 read-out.
// CG = 2: two CTAs of a cluster work on one 256-row tile.  Each loads its own 128 rows of A and its half of B's
// rows with ordinary (non-multicast) TMA; the CTA of rank 0 issues tcgen05.mma.cta_group::2, which reads both
// CTAs' shared memory and writes each CTA's half of the accumulator into that CTA's tensor memory, so an SM reads
// only half of B per multiply-accumulate.  Both CTAs' loads report their bytes to the stage barrier of rank 0 (which
// expects the pair's total), a multicast tcgen05.commit frees the stage and publishes the accumulator in both CTAs.
// ------------------------------------------------------------------------------------------------------------
template <int CG>
__device__ __forceinline__ void mma_tf32_cg(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    if constexpr (CG == 1) {
        mma_tf32(d_tmem, adesc, bdesc, idesc, accumulate);
    } else {
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "setp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::2.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
            ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
    }
}
// Arrive on the barrier at this shared-memory offset once every MMA issued so far has completed: in this CTA (CG 1),
// or in both CTAs of the pair (CG 2; the arrival is multicast, no data moves).
template <int CG>
__device__ __forceinline__ void mma_commit_cg(uint32_t bar) {
    if constexpr (CG == 1) {
        mma_commit(bar);
    } else {
        const uint16_t mask = 3;
        asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                     ::"r"(bar), "h"(mask) : "memory");
    }
}
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// Arrive on the barrier at the same offset in the CTA of rank `rank` of this cluster.
__device__ __forceinline__ void mbar_arrive_remote(uint32_t bar, uint32_t rank) {
    asm volatile(
        "{\n\t.reg .b32 ra;\n\t"
        "mapa.shared::cluster.u32 ra, %0, %1;\n\t"
        "mbarrier.arrive.release.cluster.shared::cluster.b64 _, [ra];\n\t}"
        ::"r"(bar), "r"(rank) : "memory");
}
// TMA load whose completion is reported to a barrier given by its cluster-wide address, which may lie in the other
// CTA of the pair (no multicast: the data goes to this CTA's shared memory only).
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const void* tmap, uint32_t bar_cluster, int c0, int c1, int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(tmap), "r"(bar_cluster), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
__device__ __forceinline__ void tma_load_3d_plain(uint32_t dst, const void* tmap, uint32_t bar, int c0, int c1, int c2) {
    tma_load_3d(dst, tmap, bar, c0, c1, c2);
}

constexpr int kPsTransposeWarps = 4;
constexpr int kPsEpilogueWarps = 4;

// Transpose one staged box [tile_k][rows] (row index contiguous) into the K-major swizzled stage tile.  A task is a
// (32-row block, four consecutive reduction indices) pair: lanes walk rows (conflict-free 4-byte loads), each lane
// assembles its row's four values and writes one 16-byte chunk.  What bounds this routine is its instruction count, so
// a warp keeps a row block (or shares one with other warps, taking alternate chunks) and everything that depends on the
// row is worked out once; per chunk there are four loads, one store and a few additions.
template <int KB>
__device__ __forceinline__ void ps_transpose_chunks(uint32_t src, uint32_t src_step, uint32_t dst_row, uint32_t swz, int c0, int step, int n_ch,
                                                    uint32_t k_bytes, int atom_shift, int atom_k, uint32_t atom_bytes, bool in_tile) {
    for (; c0 < n_ch; c0 += step * KB, src += src_step * KB) {
        float val[KB][4];
#pragma unroll
        for (int b = 0; b < KB; ++b) {
            const uint32_t a = src + (c0 + b * step < n_ch ? (uint32_t)b * src_step : 0u);
            val[b][0] = ld_shared_f32(a);
            val[b][1] = ld_shared_f32(a + k_bytes);
            val[b][2] = ld_shared_f32(a + 2u * k_bytes);
            val[b][3] = ld_shared_f32(a + 3u * k_bytes);
        }
#pragma unroll
        for (int b = 0; b < KB; ++b) {
            const int ci = c0 + b * step;
            if (ci < n_ch && in_tile) {
                const int kk = ci << 2;
                st_shared_v4(dst_row + (uint32_t)(kk >> atom_shift) * atom_bytes + ((uint32_t)((kk & (atom_k - 1)) << 2) ^ swz),
                             val[b][0], val[b][1], val[b][2], val[b][3]);
            }
        }
    }
}

__device__ __forceinline__ void ps_transpose(uint32_t stg, uint32_t tile, int rows, int tile_k, int atom_k, int row_bytes,
                                             int swz_mask, int tw, int nw, int lane) {
    const int atom_shift = atom_k == 32 ? 5 : (atom_k == 16 ? 4 : 3);
    const int shift = row_bytes == 128 ? 0 : (row_bytes == 64 ? 1 : 2);
    const uint32_t atom_bytes = (uint32_t)rows * (uint32_t)row_bytes;
    const int n_rb = (rows + 31) >> 5, n_ch = tile_k >> 2;
    const uint32_t k_bytes = 4u * (uint32_t)rows;                  // distance between consecutive reduction indices in the box
    // row blocks to the nw warps that work on this machine: with nw or more blocks (or a count that does not divide nw) a warp
    // takes blocks tw, tw + nw, ... and every chunk of them; with fewer, nw / n_rb warps share a block and take alternate chunks
    int rb_first, rb_step, c_first, c_step;
    const bool shared_block = n_rb < nw && (nw % n_rb) == 0;
    if (!shared_block) { rb_first = tw; rb_step = nw; c_first = 0; c_step = 1; }
    else { rb_first = tw % n_rb; rb_step = n_rb; c_first = tw / n_rb; c_step = nw / n_rb; }   // (rb_step only ends the loop)
    for (int rb = rb_first; rb < n_rb; rb += rb_step) {
        const int row = rb * 32 + lane;
        const bool in_tile = row < rows;
        const uint32_t src = stg + 4u * (uint32_t)(in_tile ? row : rows - 1) + (uint32_t)c_first * 4u * k_bytes;
        const uint32_t dst_row = tile + (uint32_t)row * (uint32_t)row_bytes;
        const uint32_t swz = (uint32_t)((row >> shift) & swz_mask) << 4;
        const int mine = (n_ch - c_first + c_step - 1) / c_step;
        if (mine <= 2) ps_transpose_chunks<2>(src, (uint32_t)c_step * 4u * k_bytes, dst_row, swz, c_first, c_step, n_ch, k_bytes, atom_shift, atom_k, atom_bytes, in_tile);
        else if (mine <= 4) ps_transpose_chunks<4>(src, (uint32_t)c_step * 4u * k_bytes, dst_row, swz, c_first, c_step, n_ch, k_bytes, atom_shift, atom_k, atom_bytes, in_tile);
        else ps_transpose_chunks<8>(src, (uint32_t)c_step * 4u * k_bytes, dst_row, swz, c_first, c_step, n_ch, k_bytes, atom_shift, atom_k, atom_bytes, in_tile);
        if (shared_block) break;                                     // this warp has no other block
    }
}

template <int CG>
__global__ void __launch_bounds__(kGemmThreads, 1)
tt_gemm_ps_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                  const __grid_constant__ CUtensorMap tmap_x, const GemmArgs g) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t full_bar[kMaxStages];     // a stage's operands are in place (TMA bytes and/or the transposer warps)
    __shared__ uint64_t empty_bar[kMaxStages];    // every multiply-accumulate that reads the stage has completed
    __shared__ uint64_t stg_full[kMaxStages];     // a staging box has landed
    __shared__ uint64_t stg_empty[kMaxStages];    // the transposer warps are done with it
    __shared__ uint64_t pm_full[2];               // tap-major convolution: a pixel-major slab buffer has been written
    __shared__ uint64_t pm_empty[2];              // ... and every multiply-accumulate that reads it has completed
    __shared__ uint64_t acc_full[2];              // an accumulator holds a finished tile
    __shared__ uint64_t acc_empty[2];             // the read-out warps (of both CTAs) have drained it
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ __align__(16) float s_bias[2][256];

    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
    volatile int* abortp = &abort_flag;
    pdl_allow_next();
    const uint32_t rank = CG == 2 ? cluster_ctarank() : 0u;
    const int unit = (int)blockIdx.x / CG, n_units = (int)gridDim.x / CG;
    const int my_tiles = g.total_tiles > unit ? (g.total_tiles - unit + n_units - 1) / n_units : 0;
    const int tiles_per_batch = g.tiles_m * g.tiles_n;
    const int kt_n = g.k_tiles;

    const uint32_t tiles_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t stage_bytes = g.a_stage_bytes + g.b_stage_bytes;
    const bool a_mn = g.a_mn != 0, b_mn = g.b_mn != 0;
    // Tap-major convolution (see the one-tile kernel): operand A = re-packed filters by TMA; operand B = views of a
    // pixel-major slab that the transposer warps write once per 32-channel block from a staged NCHW box.  Here the
    // staging ring, the two slab buffers and the filter stages all run on across tile boundaries.
    const bool tapm = g.tap_major != 0;
    const bool any_mn = a_mn || b_mn, any_km = !a_mn || !b_mn;
    const bool any_stg = any_mn || tapm;
    const int b_rows = g.b_rows_cta;
    const int RS = g.R * g.S;
    const int blocks_per_tile = tapm ? kt_n * g.n_atoms / RS : 0;     // 32-channel blocks
    constexpr int tr_groups = 1;                                      // all transposer warps work on the same box
    constexpr int tr_warps = kPsTransposeWarps / tr_groups;

    if (threadIdx.x == 32) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_a) : "memory");
        if (!tapm) asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_b) : "memory");
        else asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_x) : "memory");
    }
    if (threadIdx.x == 0) {
        const uint32_t full_count = tapm ? 1u : (any_km ? 1u : 0u) + (any_mn ? (uint32_t)tr_warps : 0u);
        for (int s = 0; s < g.stages; ++s) {
            mbar_init(smem_u32(&full_bar[s]), full_count);
            mbar_init(smem_u32(&empty_bar[s]), 1u);
        }
        for (int s = 0; s < g.stg_depth; ++s) {
            mbar_init(smem_u32(&stg_full[s]), 1u);
            mbar_init(smem_u32(&stg_empty[s]), (uint32_t)(tapm ? kPsTransposeWarps : tr_warps));
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(smem_u32(&pm_full[a]), (uint32_t)kPsTransposeWarps);
            mbar_init(smem_u32(&pm_empty[a]), 1u);
            mbar_init(smem_u32(&acc_full[a]), 1u);
            mbar_init(smem_u32(&acc_empty[a]), (uint32_t)(kPsEpilogueWarps * CG));
        }
        abort_flag = 0;
        fence_mbar_init();
        fence_proxy_async_shared();
    }
    if (warp == 1) {
        if constexpr (CG == 1) {
            tmem_alloc(smem_u32(&tmem_slot), g.tmem_cols);
            tmem_relinquish();
        } else {
            // both CTAs of the pair allocate, with the same warp and the same destination offset
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(g.tmem_cols) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        }
    }
    tc_fence_before();
    __syncthreads();
    if constexpr (CG == 2) cluster_sync_all();           // the peer's barriers exist before anything arrives on them
    tc_fence_after();
    const uint32_t tmem_base = *(volatile uint32_t*)&tmem_slot;
    pdl_wait_prev();                                      // the set-up above touched no global memory

    auto decode = [&](int i, int& m0, int& n0, int& bz) {
        const int t = unit + i * n_units;
        bz = t / tiles_per_batch;
        const int r = t - bz * tiles_per_batch;
        int tm, tn;
        if (g.raster == 0) { tm = r % g.tiles_m; tn = r / g.tiles_m; }
        else               { tn = r % g.tiles_n; tm = r / g.tiles_n; }
        m0 = (tm * CG + (int)rank) * kHwTileM;
        n0 = tn * g.tile_n;
    };

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        // Two independent streams of requests, each with its own ring and cursor: boxes of a row-contiguous operand go
        // to the staging ring (g.stg_depth deep: what is in flight from DRAM), K-major tiles to the pipeline stages.
        // The warp polls both rings and serves whichever has a free slot, so the staging ring runs as far ahead as
        // its depth allows, whatever the multiply-accumulates are doing.
        const bool leader = elect_one();
        const uint32_t a_atom = (uint32_t)(kHwTileM * g.row_bytes), b_atom = (uint32_t)(b_rows * g.row_bytes);
        const uint32_t km_bytes = (a_mn ? 0u : g.a_stage_bytes) + ((b_mn || tapm) ? 0u : g.b_stage_bytes);
        const uint32_t mn_bytes = (a_mn ? g.stg_a_bytes : 0u) + (b_mn ? g.stg_b_bytes : 0u);
        struct Cursor { int i, kt, m0, n0, bz, slot; uint32_t ph; long long it; };
        const long long total_it = (long long)my_tiles * kt_n;
        const int inner_s = tapm ? blocks_per_tile : kt_n;            // staging boxes per tile
        const long long total_s = (long long)my_tiles * inner_s;
        auto cur_init = [&](Cursor& c) {
            c.i = 0; c.kt = 0; c.slot = 0; c.ph = 0; c.it = 0; c.m0 = c.n0 = c.bz = 0;
            if (my_tiles > 0) decode(0, c.m0, c.n0, c.bz);
        };
        auto cur_next = [&](Cursor& c, int depth, int inner) {
            ++c.it;
            if (++c.slot == depth) { c.slot = 0; c.ph ^= 1u; }
            if (++c.kt == inner) {
                c.kt = 0;
                if (++c.i < my_tiles) decode(c.i, c.m0, c.n0, c.bz);
            }
        };
        Cursor cs, ck;
        cur_init(cs); cur_init(ck);
        if (!any_stg) cs.it = total_s;
        if (!any_km) ck.it = total_it;
        bool ok = true;
        unsigned long long t_last = global_timer_ns();
        unsigned idle = 0;
        while (cs.it < total_s || ck.it < total_it) {
            bool progressed = false;
            if (cs.it < total_s && mbar_test_wait(smem_u32(&stg_empty[cs.slot]), cs.ph ^ 1u)) {
                if (leader && tapm) {
                    // the input rows of 32-channel block cs.kt behind this tile's pixels: one box that starts `gap` columns
                    // left of the image and at the tile's first input row (zero fill supplies padding and gaps)
                    const uint32_t bar = smem_u32(&stg_full[cs.slot]);
                    mbar_expect_tx(bar, g.slab_box_bytes);
                    tma_load_4d(tiles_base + g.slab_off + (uint32_t)cs.slot * g.slab_buf_bytes, &tmap_x, bar, -g.slab_gap,
                                cs.n0 / g.slab_wp - g.ph, cs.kt * 32, cs.bz);
                } else if (leader) {
                    const uint32_t bar = smem_u32(&stg_full[cs.slot]);
                    const int k0 = cs.kt * g.tile_k;
                    mbar_expect_tx(bar, mn_bytes);
                    if (a_mn) tma_load_3d(tiles_base + g.a_stg_off + (uint32_t)cs.slot * g.stg_a_bytes, &tmap_a, bar, cs.m0, k0, g.a_tma_batched ? cs.bz : 0);
                    if (b_mn) tma_load_3d(tiles_base + g.b_stg_off + (uint32_t)cs.slot * g.stg_b_bytes, &tmap_b, bar, cs.n0 + (int)rank * b_rows, k0,
                                          g.b_tma_batched ? cs.bz : 0);
                }
                __syncwarp();
                cur_next(cs, g.stg_depth, inner_s);
                progressed = true;
            }
            if (ck.it < total_it && mbar_test_wait(smem_u32(&empty_bar[ck.slot]), ck.ph ^ 1u)) {
                if (leader) {
                    uint32_t bar = smem_u32(&full_bar[ck.slot]);
                    const int k0 = ck.kt * g.tile_k;
                    const int nb0 = ck.n0 + (int)rank * b_rows;       // CG 2: this CTA's half of the B rows
                    const int a_bz = g.a_tma_batched ? ck.bz : 0, b_bz = g.b_tma_batched ? ck.bz : 0;
                    // (test facility: the first stage may be told to expect more than arrives, see tt_workload_test_stall)
                    if (rank == 0) mbar_expect_tx(bar, (uint32_t)CG * km_bytes + (ck.it == 0 ? g.extra_tx : 0u));
                    if constexpr (CG == 2) bar = map_to_peer(bar, 0u);       // the pair's loads all report to rank 0
                    const uint32_t a_dst = tiles_base + (uint32_t)ck.slot * stage_bytes;
                    if (!a_mn) {
                        uint32_t dst = a_dst;
                        int kc = k0;
#pragma unroll 1
                        for (int at = 0; at < g.n_atoms; ++at, dst += a_atom, kc += g.atom_k) {
                            if constexpr (CG == 2) tma_load_3d_pair(dst, &tmap_a, bar, kc, ck.m0, a_bz);
                            else tma_load_3d(dst, &tmap_a, bar, kc, ck.m0, a_bz);
                        }
                    }
                    if (!b_mn && !tapm) {
                        uint32_t dst = a_dst + g.a_stage_bytes;
                        int kc = k0;
#pragma unroll 1
                        for (int at = 0; at < g.n_atoms; ++at, dst += b_atom, kc += g.atom_k) {
                            if constexpr (CG == 2) tma_load_3d_pair(dst, &tmap_b, bar, kc, nb0, b_bz);
                            else tma_load_3d(dst, &tmap_b, bar, kc, nb0, b_bz);
                        }
                    }
                }
                __syncwarp();
                cur_next(ck, g.stages, kt_n);
                progressed = true;
            }
            if (progressed) { idle = 0; continue; }
            if ((++idle & 63u) == 0u) {
                // nothing to do for a while: the same bounded patience as every other wait of the kernel
                if (idle == 64u) t_last = global_timer_ns();
                bool give_up = *abortp != 0;
                if (!give_up && global_timer_ns() - t_last > g.wait_ns) {
                    *abortp = 1;
                    atomicCAS(g.status, 0u, (unsigned)TT_ERR_TIMEOUT | (1u << 8));
                    give_up = true;
                }
                if (__any_sync(0xffffffffu, give_up)) { ok = false; break; }
            }
        }
        if ((!ok || *abortp) && lane == 0) {
            // let copies in flight land before shared memory is given back (bounded)
            for (int pass = 0; pass < 2; ++pass) {
                const long long issued = pass == 0 ? ck.it : cs.it;
                const int depth = pass == 0 ? g.stages : g.stg_depth;
                if ((pass == 0 && (!any_km || rank != 0)) || (pass == 1 && !any_stg)) continue;
                const long long first = issued > depth ? issued - depth : 0;
                for (long long it = first; it < issued; ++it) {
                    const uint32_t bar = pass == 0 ? smem_u32(&full_bar[it % depth]) : smem_u32(&stg_full[it % depth]);
                    const uint32_t par = (uint32_t)(it / depth) & 1u;
                    const unsigned long long t0 = global_timer_ns();
                    while (!mbar_try_wait(bar, par)) { if (global_timer_ns() - t0 > 2000000ull) break; }
                }
            }
            if (rank != 0) {
                // this CTA's K-major loads report to rank 0's barriers: give them time to land instead (the pair leaves
                // together, after rank 0 has seen the pair's bytes or given up on them)
                const unsigned long long t0 = global_timer_ns();
                while (global_timer_ns() - t0 < 200000ull) { }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ---------------- MMA issuer (of a pair: rank 0's) ----------------
        const bool leader = elect_one();
        uint32_t st = 0, ph = 0;
        bool ok = true;
        if (CG == 2 && rank != 0) {
            // rank 0 issues for the pair
        } else {
            const uint64_t d0 = make_desc(0u, g.row_bytes);
            const uint32_t d_hi = (uint32_t)(d0 >> 32), d_lo = (uint32_t)d0;
            const uint32_t a_lo0 = d_lo + ((tiles_base & 0x3FFFFu) >> 4);
            const uint32_t stage_step = stage_bytes >> 4;
            const uint32_t a_atom = (uint32_t)(kHwTileM * g.row_bytes) >> 4, b_atom = (uint32_t)(b_rows * g.row_bytes) >> 4;
            const uint32_t b_off = g.a_stage_bytes >> 4;
            uint32_t gblock = 0;                         // tap-major: 32-channel blocks consumed so far, over all tiles
            for (int i = 0; i < my_tiles && ok; ++i) {
                const uint32_t acc = (uint32_t)i & 1u, aph = ((uint32_t)i >> 1) & 1u;
                // the read-out of the tile that used this accumulator two tiles ago has finished
                const bool freed = CG == 2 ? mbar_wait_cluster(smem_u32(&acc_empty[acc]), aph ^ 1u, abortp, g.status, 12u, g.wait_ns)
                                           : mbar_wait(smem_u32(&acc_empty[acc]), aph ^ 1u, abortp, g.status, 12u, g.wait_ns);
                if (!__all_sync(0xffffffffu, freed)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * (uint32_t)g.tile_n;
                if (tapm) {
                    // the B tile of reduction tile kt = (channel block, taps) is the block's pixel-major slab read from row
                    // lin0 + r * wp + s on: only the descriptor's start address changes from tap to tap
                    int m0t, n0t, bzt;
                    decode(i, m0t, n0t, bzt);
                    const uint32_t pm0 = tiles_base + g.pm_off;
                    const int lin0 = (n0t - (n0t / g.slab_wp) * g.slab_wp) + g.slab_gap - g.pw;
                    int tap = 0, fr = 0, fs = 0;
                    for (int kt = 0; kt < kt_n; ++kt) {
                        bool got = mbar_wait(smem_u32(&full_bar[st]), ph, abortp, g.status, 2u, g.wait_ns);        // the filter tile
                        if (tap == 0 && got) got = mbar_wait(smem_u32(&pm_full[gblock & 1u]), (gblock >> 1) & 1u, abortp, g.status, 7u, g.wait_ns);
                        if (!__all_sync(0xffffffffu, got)) { ok = false; break; }
                        tc_fence_after();
                        if (leader) {
                            uint32_t a_lo = a_lo0 + st * stage_step;
                            int r2 = fr, s2 = fs;
#pragma unroll 1
                            for (int t = 0; t < g.n_atoms; ++t, a_lo += a_atom) {
                                const uint32_t row = (uint32_t)(lin0 + r2 * g.slab_wp + s2);
                                const uint32_t b_lo = d_lo + (((pm0 + (gblock & 1u) * g.pm_buf_bytes + row * 128u) & 0x3FFFFu) >> 4);
#pragma unroll
                                for (int k8 = 0; k8 < 4; ++k8)
                                    mma_tf32_cg<CG>(d_tmem, ((uint64_t)d_hi << 32) | (uint64_t)(a_lo + 2u * (uint32_t)k8),
                                                    ((uint64_t)d_hi << 32) | (uint64_t)(b_lo + 2u * (uint32_t)k8), g.idesc,
                                                    (kt > 0 || t > 0 || k8 > 0) ? 1u : 0u);
                                if (++s2 == g.S) { s2 = 0; ++r2; }
                            }
                            mma_commit_cg<CG>(smem_u32(&empty_bar[st]));                           // filter stage reusable
                            if (tap + g.n_atoms == RS) mma_commit_cg<CG>(smem_u32(&pm_empty[gblock & 1u]));   // slab buffer reusable
                        }
                        __syncwarp();
                        for (int t = 0; t < g.n_atoms; ++t) if (++fs == g.S) { fs = 0; ++fr; }
                        tap += g.n_atoms;
                        if (tap == RS) { tap = 0; fr = 0; fs = 0; ++gblock; }
                        if (++st == (uint32_t)g.stages) { st = 0; ph ^= 1u; }
                    }
                } else
                for (int kt = 0; kt < kt_n; ++kt) {
                    const bool got = mbar_wait(smem_u32(&full_bar[st]), ph, abortp, g.status, 2u, g.wait_ns);
                    if (!__all_sync(0xffffffffu, got)) { ok = false; break; }
                    tc_fence_after();
                    if (leader) {
                        const uint32_t a_lo = a_lo0 + st * stage_step, b_lo = a_lo + b_off;
                        const uint32_t accumulate = kt > 0 ? 1u : 0u;
#pragma unroll 1
                        for (int at = 0; at < g.n_atoms; ++at) {
                            const int k8n = g.atom_k >> 3;
#pragma unroll 4
                            for (int k8 = 0; k8 < k8n; ++k8)
                                mma_tf32_cg<CG>(d_tmem, ((uint64_t)d_hi << 32) | (uint64_t)(a_lo + (uint32_t)at * a_atom + 2u * (uint32_t)k8),
                                                ((uint64_t)d_hi << 32) | (uint64_t)(b_lo + (uint32_t)at * b_atom + 2u * (uint32_t)k8), g.idesc,
                                                (at == 0 && k8 == 0) ? accumulate : 1u);
                        }
                        mma_commit_cg<CG>(smem_u32(&empty_bar[st]));          // stage reusable once these MMAs have read it
                    }
                    __syncwarp();
                    if (++st == (uint32_t)g.stages) { st = 0; ph ^= 1u; }
                }
                if (ok && leader) mma_commit_cg<CG>(smem_u32(&acc_full[acc]));   // the tile's accumulator is complete
                __syncwarp();
            }
        }
    } else if (warp < 2 + kPsTransposeWarps) {
        // ---------------- transposers ----------------
        if (tapm) {
            // staging box [32 channels][in_rows][wp] -> pixel-major slab: one 128-byte row per staged position (32
            // channels), 16-byte chunks swizzled by the row's absolute address like a TMA 128-byte tile.  Warp tw moves
            // the channel groups tw and tw + 4 of every position; lanes walk positions.
            const int tw = warp - 2;
            const int tt = (int)threadIdx.x - 64;
            const uint32_t st0 = tiles_base + g.slab_off, pm0 = tiles_base + g.pm_off;
            const int npix = g.slab_in_rows * g.slab_wp;
            // rows a view can touch beyond the transposed range must hold finite numbers: clear both buffers once
            for (uint32_t o = (uint32_t)tt * 16u; o < 2u * g.pm_buf_bytes; o += 32u * kPsTransposeWarps * 16u)
                st_shared_v4(pm0 + o, 0.f, 0.f, 0.f, 0.f);
            if (g.slab_box_ch < 32)                      // channels beyond the TMA box (which may already be landing) read as zero
                for (int sl = 0; sl < g.stg_depth; ++sl)
                    for (uint32_t o = g.slab_box_bytes + (uint32_t)tt * 16u; o < g.slab_buf_bytes; o += 32u * kPsTransposeWarps * 16u)
                        st_shared_v4(st0 + (uint32_t)sl * g.slab_buf_bytes + o, 0.f, 0.f, 0.f, 0.f);
            asm volatile("bar.sync 3, %0;" ::"n"(32 * kPsTransposeWarps) : "memory");
            const uint32_t ch_bytes = 4u * (uint32_t)g.slab_chpitch;
            uint32_t sst = 0, sph = 0, gb = 0;
            bool ok = true;
            const long long total_blocks = (long long)my_tiles * blocks_per_tile;
            for (long long j = 0; j < total_blocks && ok; ++j, ++gb) {
                const uint32_t b = gb & 1u;
                if (!mbar_wait(smem_u32(&stg_full[sst]), sph, abortp, g.status, 6u, g.wait_ns) ||
                    !mbar_wait(smem_u32(&pm_empty[b]), ((gb >> 1) & 1u) ^ 1u, abortp, g.status, 8u, g.wait_ns)) { ok = false; break; }
                const uint32_t dst = pm0 + b * g.pm_buf_bytes;
#pragma unroll 1
                for (int grp = tw; grp < 8; grp += kPsTransposeWarps) {
                    const uint32_t src = st0 + sst * g.slab_buf_bytes + (uint32_t)(4 * grp) * ch_bytes;
                    for (int p0 = lane; p0 < npix; p0 += 128) {
                        float v[4][4];
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const int pix = min(p0 + 32 * u, npix - 1);
                            const uint32_t a = src + 4u * (uint32_t)pix;
                            v[u][0] = ld_shared_f32(a);
                            v[u][1] = ld_shared_f32(a + ch_bytes);
                            v[u][2] = ld_shared_f32(a + 2u * ch_bytes);
                            v[u][3] = ld_shared_f32(a + 3u * ch_bytes);
                        }
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const int pix = p0 + 32 * u;
                            if (pix < npix) {
                                const uint32_t rowa = dst + 128u * (uint32_t)pix;
                                st_shared_v4(rowa + ((((uint32_t)grp) ^ ((rowa >> 7) & 7u)) << 4), v[u][0], v[u][1], v[u][2], v[u][3]);
                            }
                        }
                    }
                }
                fence_proxy_async_shared();              // generic-proxy stores -> visible to the tensor core's reads
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(smem_u32(&pm_full[b]));
                    mbar_arrive(smem_u32(&stg_empty[sst]));
                }
                if (++sst == (uint32_t)g.stg_depth) { sst = 0; sph ^= 1u; }
            }
        } else if (any_mn) {
            const int grp = (warp - 2) / tr_warps, tw = (warp - 2) - grp * tr_warps;
            int st = grp % g.stages, sst = grp % g.stg_depth;
            uint32_t ph = (uint32_t)(grp / g.stages) & 1u, sph = (uint32_t)(grp / g.stg_depth) & 1u;
            const long long total_it = (long long)my_tiles * kt_n;
            for (long long it = grp; it < total_it; it += tr_groups) {
                if (!mbar_wait(smem_u32(&stg_full[sst]), sph, abortp, g.status, 6u, g.wait_ns) ||
                    !mbar_wait(smem_u32(&empty_bar[st]), ph ^ 1u, abortp, g.status, 3u, g.wait_ns)) break;
                const uint32_t a_s = tiles_base + (uint32_t)st * stage_bytes, b_s = a_s + g.a_stage_bytes;
                if (a_mn) ps_transpose(tiles_base + g.a_stg_off + (uint32_t)sst * g.stg_a_bytes, a_s, kHwTileM, g.tile_k, g.atom_k, g.row_bytes, g.swz_mask, tw, tr_warps, lane);
                if (b_mn) ps_transpose(tiles_base + g.b_stg_off + (uint32_t)sst * g.stg_b_bytes, b_s, b_rows, g.tile_k, g.atom_k, g.row_bytes, g.swz_mask, tw, tr_warps, lane);
                fence_proxy_async_shared();              // generic-proxy stores -> visible to the tensor core's reads
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(smem_u32(&full_bar[st]));
                    mbar_arrive(smem_u32(&stg_empty[sst]));
                }
                st += tr_groups;
                while (st >= g.stages) { st -= g.stages; ph ^= 1u; }
                sst += tr_groups;
                while (sst >= g.stg_depth) { sst -= g.stg_depth; sph ^= 1u; }
            }
        }
    } else {
        // ---------------- read-out: tensor memory -> bias, residual, activation -> global memory ----------------
        const int ew = warp - (2 + kPsTransposeWarps);
        const int et = (int)threadIdx.x - 32 * (2 + kPsTransposeWarps);
        const int quad = warp & 3;                       // tensor-memory lane quadrant this warp may read
        EpiArgs e;
        e.y_ms = g.y_ms; e.y_ns = g.y_ns; e.M = g.M;
        e.lo = g.act == TT_ACT_NONE || g.act == TT_ACT_GELU_ERF ? -INFINITY : 0.f;
        e.hi = g.act == TT_ACT_RELU6 ? 6.f : INFINITY;
        e.gelu = g.act == TT_ACT_GELU_ERF;
        e.vec = (g.vec_store & 1) != 0;
        e.lin_wp = tapm ? g.slab_wp : 0; e.lin_q = g.Q; e.lin_p = g.Pout;
        const bool transposed = g.y_ns == 1 && g.y_ms != 1;
        const uint32_t stg = tiles_base + g.epi_off + (uint32_t)ew * (uint32_t)kStageBytesPerWarp;
        bool ok = true;
        for (int i = 0; i < my_tiles && ok; ++i) {
            int m0, n0, bz;
            decode(i, m0, n0, bz);
            const uint32_t acc = (uint32_t)i & 1u, aph = ((uint32_t)i >> 1) & 1u;
            const int m_first = m0 + quad * 32, m = m_first + lane;
            // this tile's bias values, staged while the tile is still being accumulated (the buffer's previous readers
            // finished two tiles ago: they passed the barrier below for tile i - 1 since)
            if (g.bias_mode == 2) for (int c = et; c < g.tile_n; c += 32 * kPsEpilogueWarps) s_bias[acc][c] = (n0 + c < g.N) ? __ldg(g.bias + n0 + c) : 0.f;
            const float bias_row = (g.bias_mode == 1 && m < g.M) ? __ldg(g.bias + m) : 0.f;
            const bool have = mbar_wait(smem_u32(&acc_full[acc]), aph, abortp, g.status, 4u, g.wait_ns);
            uint32_t all_acc;
            asm volatile(
                "{\n\t.reg .pred p, q;\n\t"
                "setp.ne.u32 q, %1, 0;\n\t"
                "bar.red.and.pred p, 2, %2, q;\n\t"
                "selp.u32 %0, 1, 0, p;\n\t}"
                : "=r"(all_acc) : "r"((uint32_t)have), "n"(32 * kPsEpilogueWarps) : "memory");
            if (!all_acc) { ok = false; break; }
            tc_fence_after();
            e.ybase = g.y + (long long)bz * g.y_bs;
            e.rbase = g.residual ? g.residual + (long long)bz * g.y_bs : nullptr;
            const uint32_t t_row = tmem_base + ((uint32_t)(quad * 32) << 16) + acc * (uint32_t)g.tile_n;
            uint32_t r[32];
            tmem_ld32(t_row, r);
#pragma unroll 1
            for (int c0 = 0; c0 < g.tile_n; c0 += 32) {
                float v[32];
                const int nb = n0 + c0;
                const int cnt = min(g.N - nb, g.tile_n - c0);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]);
                if (c0 + 32 < g.tile_n) tmem_ld32(t_row + (uint32_t)(c0 + 32), r);
                else {
                    // every value of this accumulator is in registers: hand it back to the MMA warp
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) {
                        if (CG == 2) mbar_arrive_remote(smem_u32(&acc_empty[acc]), 0u);
                        else mbar_arrive(smem_u32(&acc_empty[acc]));
                    }
                }
                if (cnt <= 0) continue;                  // warp-uniform
                if (g.bias_mode == 1) {
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] += bias_row;
                } else if (g.bias_mode == 2) {
#pragma unroll
                    for (int j = 0; j < 32; j += 4) {
                        const float4 b = *reinterpret_cast<const float4*>(&s_bias[acc][c0 + j]);
                        v[j] += b.x; v[j + 1] += b.y; v[j + 2] += b.z; v[j + 3] += b.w;
                    }
                }
                const bool full = !tapm && cnt >= 32 && m_first + 32 <= g.M && (e.vec || !transposed);
                if (e.rbase == nullptr) {
                    if (e.gelu) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) v[j] = gelu_erf(v[j]);
                    } else if (g.act != TT_ACT_NONE) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) v[j] = fminf(fmaxf(v[j], e.lo), e.hi);
                    }
                    if (full) epilogue_block<true, false>(v, e, m_first, nb, cnt, stg, lane, transposed);
                    else epilogue_block<false, false>(v, e, m_first, nb, cnt, stg, lane, transposed);
                } else {
                    if (full) epilogue_block<true, true>(v, e, m_first, nb, cnt, stg, lane, transposed);
                    else epilogue_block<false, true>(v, e, m_first, nb, cnt, stg, lane, transposed);
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    // a pair stays together until neither CTA touches the other's shared memory, barriers or tensor memory any more
    if constexpr (CG == 2) cluster_sync_all();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        if constexpr (CG == 1) tmem_dealloc(tmem_base, g.tmem_cols);
        else asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(g.tmem_cols) : "memory");
    }
}

// ------------------------------------------------------------------------------------------------------------
// DW_SIMT: depthwise conv + bias + activation.  One CTA = tile_c channels x tile_h x tile_w outputs of one image.
// The input halo tile is staged in shared memory with coalesced row reads; each thread then produces `items`
// consecutive outputs along the width and stores them with vec-wide stores.
// ------------------------------------------------------------------------------------------------------------
__global__ void tt_dwconv_kernel(const DwArgs d) {
    pdl_allow_next();
    pdl_wait_prev();
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
// DW_SIMT, register-window form (3x3 and 5x5 filters, stride 1 or 2).  A thread owns a strip of ROWS output rows
// x 4 or 8 consecutive output columns of one channel.  It walks the (ROWS-1)*STRIDE + R input rows the strip needs
// once: of each row it fetches 3*STRIDE + R values (aligned 16-byte loads for the columns under the strip when the
// image rows allow it, 4-byte loads for the ragged edges; neighbouring strips' loads meet in L1) and feeds every
// output row whose window contains that input row, so an input value is read once per strip and no shared
// memory or barrier is involved.  Bound by HBM: the only DRAM traffic is x once, y once.
// ------------------------------------------------------------------------------------------------------------
template <int R, int STRIDE, int ROWS, int WIDTH>
__global__ void __launch_bounds__(256, WIDTH == 4 ? 6 : 4) tt_dwconv_window_kernel(const DwArgs d) {
    constexpr int NCOL = (WIDTH - 1) * STRIDE + R;        // input columns under a WIDTH-wide strip
    constexpr int IN_ROWS = (ROWS - 1) * STRIDE + R;
    constexpr int PAD = R / 2;                            // "same" padding: the launcher checks it
    constexpr int NV = (NCOL - PAD) / 4;                  // aligned 16-byte groups per window row
    pdl_allow_next();
    pdl_wait_prev();
    const int n = blockIdx.y;
    int t = blockIdx.x;
    const int tw = t % d.tiles_w; t /= d.tiles_w;
    const int th = t % d.tiles_h; t /= d.tiles_h;
    const int c0 = t * d.tile_c, p0 = th * d.tile_h, q0 = tw * d.tile_w;
    const int nc = min(d.tile_c, d.C - c0);
    const int groups_w = d.tile_w / WIDTH;
    const int groups_h = (d.tile_h + ROWS - 1) / ROWS;
    const int work = nc * groups_h * groups_w;
    for (int i = threadIdx.x; i < work; i += blockDim.x) {
        const int gwi = i % groups_w;
        const int rest = i / groups_w;
        const int gh = rest % groups_h, cl = rest / groups_h;
        const int p = p0 + gh * ROWS, q = q0 + gwi * WIDTH;
        if (p >= d.P || q >= d.Q || gh * ROWS >= d.tile_h) continue;
        const int c = c0 + cl;
        const float* __restrict__ xc = d.x + ((long long)n * d.C + c) * d.H * (long long)d.W;
        const float* __restrict__ wc = d.w + (long long)c * (R * R);
        float wv[R * R];
#pragma unroll
        for (int k = 0; k < R * R; ++k) wv[k] = __ldg(wc + k);
        const float b = d.bias ? __ldg(d.bias + c) : 0.f;
        float acc[ROWS][WIDTH];
#pragma unroll
        for (int ro = 0; ro < ROWS; ++ro)
#pragma unroll
            for (int j = 0; j < WIDTH; ++j) acc[ro][j] = b;
        const int ih0 = p * STRIDE - PAD, iw0 = q * STRIDE - PAD;
#pragma unroll
        for (int ri = 0; ri < IN_ROWS; ++ri) {
            const int ih = ih0 + ri;
            float v[NCOL];
#pragma unroll
            for (int j = 0; j < NCOL; ++j) v[j] = 0.f;
            if ((unsigned)ih < (unsigned)d.H) {
                const float* __restrict__ xr = xc + (long long)ih * d.W;
                if (d.vec_in) {
                    // window slots [PAD, PAD + 4*NV) lie under the strip and start on a 16-byte boundary; a group
                    // of four columns is inside the row or outside it as a whole (W % 4 == 0)
#pragma unroll
                    for (int k = 0; k < NV; ++k) {
                        const int col = iw0 + PAD + 4 * k;
                        if (col < d.W) {
                            const float4 f = __ldg(reinterpret_cast<const float4*>(xr + col));
                            v[PAD + 4 * k] = f.x; v[PAD + 4 * k + 1] = f.y; v[PAD + 4 * k + 2] = f.z; v[PAD + 4 * k + 3] = f.w;
                        }
                    }
#pragma unroll
                    for (int j = 0; j < NCOL; ++j) {
                        if (j >= PAD && j < PAD + 4 * NV) continue;
                        const int col = iw0 + j;
                        if ((unsigned)col < (unsigned)d.W) v[j] = __ldg(xr + col);
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < NCOL; ++j) {
                        const int col = iw0 + j;
                        if ((unsigned)col < (unsigned)d.W) v[j] = __ldg(xr + col);
                    }
                }
            }
#pragma unroll
            for (int ro = 0; ro < ROWS; ++ro) {
                const int fr = ri - ro * STRIDE;              // compile-time after unrolling
                if (fr >= 0 && fr < R) {
#pragma unroll
                    for (int fs = 0; fs < R; ++fs)
#pragma unroll
                        for (int j = 0; j < WIDTH; ++j) acc[ro][j] = fmaf(v[j * STRIDE + fs], wv[fr * R + fs], acc[ro][j]);
                }
            }
        }
        float* __restrict__ yc = d.y + (((long long)n * d.C + c) * d.P + p) * (long long)d.Q + q;
#pragma unroll
        for (int ro = 0; ro < ROWS; ++ro) {
            if (p + ro >= d.P || gh * ROWS + ro >= d.tile_h) break;
            float* yo = yc + (long long)ro * d.Q;
#pragma unroll
            for (int j0 = 0; j0 < WIDTH; j0 += 4) {
                float o[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) o[j] = apply_act(acc[ro][j0 + j], d.act);
                if (d.vec == 4 && q + j0 + 4 <= d.Q) {
                    *reinterpret_cast<float4*>(yo + j0) = make_float4(o[0], o[1], o[2], o[3]);
                } else if (d.vec == 2 && q + j0 + 4 <= d.Q) {
                    *reinterpret_cast<float2*>(yo + j0) = make_float2(o[0], o[1]);
                    *reinterpret_cast<float2*>(yo + j0 + 2) = make_float2(o[2], o[3]);
                } else {
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        if (q + j0 + j < d.Q) yo[j0 + j] = o[j];
                }
            }
        }
    }
}

// ------------------------------------------------------------------------------------------------------------
// DW_SIMT, TMA-staged persistent form (3x3 and 5x5 "same" filters, stride 1 or 2, image rows of 16-byte multiples).
// The image is one 3-D tensor (W, H, planes = N * C).  A tile is tile_c consecutive planes x tile_h x tile_w
// outputs; its input box [tile_c][in_h][box_w] starts 4 columns left of the tile (a 16-byte aligned coordinate) and
// PAD rows above it, and the TMA zero fill supplies the padding, so the compute loop has no bounds test on inputs.
// CTAs walk the tiles persistently with `stages` boxes in flight: no thread waits on a global load, which is what
// limits the register-window kernel.  Threads work on ROWS x WIDTH strips exactly as there, reading the window rows
// with aligned 16-byte shared-memory loads.  Same FMAs in the same order: bit-identical outputs.
// The instruction stream per output is what bounds this kernel next to the memory system, so everything that does
// not depend on the plane is hoisted: a thread keeps its strip position for the whole kernel, tile coordinates
// advance by additions, and the filters and biases of a tile's planes are staged in shared memory (one buffer per
// box buffer, [tile_c][WP] floats: filter, bias, padding) when the tile's box is requested.
// ------------------------------------------------------------------------------------------------------------
template <int R, int STRIDE, int ROWS, int WIDTH>
__global__ void __launch_bounds__(256) tt_dwconv_tma_kernel(const __grid_constant__ CUtensorMap tmap_x, const DwArgs d) {
    constexpr int NCOL = (WIDTH - 1) * STRIDE + R;
    constexpr int IN_ROWS = (ROWS - 1) * STRIDE + R;
    constexpr int PAD = R / 2;
    constexpr int FIRST = 4 - PAD;                        // window slot 0 sits this many floats right of the strip's aligned base
    constexpr int NLD = (FIRST + NCOL + 3) / 4;           // aligned 16-byte loads per window row
    constexpr int WP = (R * R + 1 + 3) / 4 * 4;           // floats per plane in a weight buffer
    extern __shared__ uint8_t dw_raw[];
    __shared__ uint64_t full_bar[4];
    __shared__ int abort_flag;
    const uint32_t base = (smem_u32(dw_raw) + 127u) & ~127u;
    const uint32_t wbase = base + (uint32_t)d.tma_stages * (uint32_t)d.stage_bytes;
    volatile int* abortp = &abort_flag;
    pdl_allow_next();
    if (threadIdx.x == 0) {
        for (int s = 0; s < d.tma_stages; ++s) mbar_init(smem_u32(&full_bar[s]), 1u);
        abort_flag = 0;
        fence_mbar_init();
        fence_proxy_async_shared();
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_x) : "memory");
    }
    __syncthreads();
    pdl_wait_prev();                                      // the set-up above touched no global memory
    const int planes = d.N * d.C;
    const int per_plane_tiles = d.tiles_h * d.tiles_w;
    const int my_tiles = d.total_tiles > (int)blockIdx.x ? (d.total_tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
    // Tile t = blockIdx.x + i * gridDim.x as (plane tile, row tile, column tile, first channel): decomposed once, then
    // advanced by the decomposition of gridDim.x with carries -- no division per tile.
    struct TilePos { int tp, th, tw, c0; };
    int step_tp, step_th, step_tw, step_c;
    {
        const int gsz = (int)gridDim.x;
        step_tp = gsz / per_plane_tiles;
        const int rem = gsz - step_tp * per_plane_tiles;
        step_th = rem / d.tiles_w; step_tw = rem - step_th * d.tiles_w;
        step_c = (int)(((long long)step_tp * d.tile_c) % d.C);
    }
    const int tile_c_mod = d.tile_c % d.C;
    auto first_pos = [&]() {
        TilePos t;
        const int b = (int)blockIdx.x;
        t.tp = b / per_plane_tiles;
        const int rem = b - t.tp * per_plane_tiles;
        t.th = rem / d.tiles_w; t.tw = rem - t.th * d.tiles_w;
        t.c0 = (int)(((long long)t.tp * d.tile_c) % d.C);
        return t;
    };
    auto advance = [&](TilePos& t) {
        t.tw += step_tw; t.th += step_th; t.tp += step_tp; t.c0 += step_c;
        if (t.tw >= d.tiles_w) { t.tw -= d.tiles_w; ++t.th; }
        if (t.th >= d.tiles_h) { t.th -= d.tiles_h; ++t.tp; t.c0 += tile_c_mod; }
        while (t.c0 >= d.C) t.c0 -= d.C;
    };
    auto issue = [&](const TilePos& t, int s) {           // thread 0: request the input box of a tile into buffer s
        const uint32_t bar = smem_u32(&full_bar[s]);
        mbar_expect_tx(bar, (uint32_t)(d.tile_c * d.in_h * d.box_w * 4));
        tma_load_3d(base + (uint32_t)s * (uint32_t)d.stage_bytes, &tmap_x, bar, t.tw * d.tile_w * STRIDE - 4,
                    t.th * d.tile_h * STRIDE - PAD, t.tp * d.tile_c);
    };
    auto stage_weights = [&](const TilePos& t, int s) {   // all threads: the filters and biases of the tile's planes
        const uint32_t dst = wbase + (uint32_t)s * (uint32_t)d.wstage_bytes;
        const int pl0 = t.tp * d.tile_c;
        for (int idx = (int)threadIdx.x; idx < d.tile_c * WP; idx += (int)blockDim.x) {
            const int cl = idx / WP, k = idx - cl * WP;
            int c = t.c0 + cl;                            // tile_c <= C: one subtraction wraps it
            if (c >= d.C) c -= d.C;
            float v = 0.f;
            if (pl0 + cl < planes) {
                if (k < R * R) v = __ldg(d.w + c * (R * R) + k);
                else if (k == R * R && d.bias) v = __ldg(d.bias + c);
            }
            st_shared_f32(dst + 4u * (uint32_t)idx, v);
        }
    };
    TilePos cur = first_pos(), nxt = cur;
    {
        const int pre = min(my_tiles, d.tma_stages);
        for (int i = 0; i < pre; ++i) {
            if (threadIdx.x == 0) issue(nxt, i);
            stage_weights(nxt, i);
            advance(nxt);
        }
    }
    __syncthreads();                                      // the first weight buffers are in place
    // a thread's strip position inside a plane is fixed for the whole kernel when a plane has at most blockDim strips
    // (the thread then walks planes cl_f, cl_f + cpp, ...); otherwise it also walks strips
    const int groups_w = d.tile_w / WIDTH;
    const int groups_h = (d.tile_h + ROWS - 1) / ROWS;
    const int spp = groups_h * groups_w;                  // strips per plane
    const bool fixed_pos = spp <= (int)blockDim.x;
    const int cpp = fixed_pos ? (int)blockDim.x / spp : 1;                  // planes per pass
    const int cl_f = fixed_pos ? (int)threadIdx.x / spp : 0;
    const int s_f = (int)threadIdx.x - cl_f * spp;
    const int s_step = fixed_pos ? spp : (int)blockDim.x;                    // fixed: the strip loop runs once
    const bool active = cl_f < cpp;
    const int gh_f = s_f / groups_w, gwi_f = s_f - gh_f * groups_w;
    const uint32_t plane_bytes = 4u * (uint32_t)(d.in_h * d.box_w);
    const long long plane_out = (long long)d.P * d.Q;
    const bool clamp = d.act == TT_ACT_RELU || d.act == TT_ACT_RELU6, gelu = d.act == TT_ACT_GELU_ERF;
    const float hi = d.act == TT_ACT_RELU6 ? 6.f : INFINITY;
    int s = 0;
    uint32_t ph = 0;
    for (int i = 0; i < my_tiles; ++i) {
        // every thread waits for the box itself (all take the same decision: the same barrier and phase)
        if (!mbar_wait(smem_u32(&full_bar[s]), ph, abortp, d.status, 9u, d.wait_ns)) break;
        const int pl0 = cur.tp * d.tile_c, p0 = cur.th * d.tile_h, q0 = cur.tw * d.tile_w;
        const int ncl = min(d.tile_c, planes - pl0);
        const uint32_t stage = base + (uint32_t)s * (uint32_t)d.stage_bytes;
        const uint32_t wst = wbase + (uint32_t)s * (uint32_t)d.wstage_bytes;
        for (int sidx = s_f; active && sidx < spp; sidx += s_step) {
            int gh = gh_f, gwi = gwi_f;
            if (sidx != s_f) { gh = sidx / groups_w; gwi = sidx - gh * groups_w; }
            const int p = p0 + gh * ROWS, q = q0 + gwi * WIDTH;
            if (p >= d.P || q >= d.Q || gh * ROWS >= d.tile_h) continue;
            const int nrows = min(ROWS, min(d.P - p, d.tile_h - gh * ROWS));
            const bool whole = q + WIDTH <= d.Q;
            // the strip's window rows: box row gh*ROWS*STRIDE + ri, from the aligned float WIDTH*gwi*STRIDE on
            const uint32_t soff = stage + 4u * (uint32_t)((gh * ROWS * STRIDE) * d.box_w + WIDTH * gwi * STRIDE);
            float* __restrict__ y0 = d.y + ((long long)pl0 * d.P + p) * (long long)d.Q + q;
#pragma unroll 1
            for (int cl = cl_f; cl < ncl; cl += cpp) {
                float wv[WP];
#pragma unroll
                for (int k = 0; k < WP / 4; ++k) {
                    const float4 f = ld_shared_v4f(wst + 4u * (uint32_t)(cl * WP + 4 * k));
                    wv[4 * k] = f.x; wv[4 * k + 1] = f.y; wv[4 * k + 2] = f.z; wv[4 * k + 3] = f.w;
                }
                float acc[ROWS][WIDTH];
#pragma unroll
                for (int ro = 0; ro < ROWS; ++ro)
#pragma unroll
                    for (int j = 0; j < WIDTH; ++j) acc[ro][j] = wv[R * R];
                const uint32_t row0 = soff + (uint32_t)cl * plane_bytes;
#pragma unroll
                for (int ri = 0; ri < IN_ROWS; ++ri) {
                    float u[4 * NLD];
#pragma unroll
                    for (int k = 0; k < NLD; ++k) {
                        const float4 f = ld_shared_v4f(row0 + 4u * (uint32_t)(ri * d.box_w + 4 * k));
                        u[4 * k] = f.x; u[4 * k + 1] = f.y; u[4 * k + 2] = f.z; u[4 * k + 3] = f.w;
                    }
#pragma unroll
                    for (int ro = 0; ro < ROWS; ++ro) {
                        const int fr = ri - ro * STRIDE;          // compile-time after unrolling
                        if (fr >= 0 && fr < R) {
#pragma unroll
                            for (int fs = 0; fs < R; ++fs)
#pragma unroll
                                for (int j = 0; j < WIDTH; ++j) acc[ro][j] = fmaf(u[FIRST + j * STRIDE + fs], wv[fr * R + fs], acc[ro][j]);
                        }
                    }
                }
                float* __restrict__ yc = y0 + (long long)cl * plane_out;
#pragma unroll
                for (int ro = 0; ro < ROWS; ++ro) {
                    if (ro >= nrows) break;
                    if (clamp) {
#pragma unroll
                        for (int j = 0; j < WIDTH; ++j) acc[ro][j] = fminf(fmaxf(acc[ro][j], 0.f), hi);
                    } else if (gelu) {
#pragma unroll
                        for (int j = 0; j < WIDTH; ++j) acc[ro][j] = gelu_erf(acc[ro][j]);
                    }
                    float* yo = yc + (long long)ro * d.Q;
                    if (whole && d.vec == 4) {
#pragma unroll
                        for (int j = 0; j < WIDTH; j += 4)
                            *reinterpret_cast<float4*>(yo + j) = make_float4(acc[ro][j], acc[ro][j + 1], acc[ro][j + 2], acc[ro][j + 3]);
                    } else if (whole && d.vec == 2) {
#pragma unroll
                        for (int j = 0; j < WIDTH; j += 2) *reinterpret_cast<float2*>(yo + j) = make_float2(acc[ro][j], acc[ro][j + 1]);
                    } else {
#pragma unroll
                        for (int j = 0; j < WIDTH; ++j)
                            if (q + j < d.Q) yo[j] = acc[ro][j];
                    }
                }
            }
        }
        __syncthreads();                                  // everyone is done with this box and its weight buffer
        if (i + d.tma_stages < my_tiles) {
            if (threadIdx.x == 0) issue(nxt, s);
            stage_weights(nxt, s);                        // read again only after a later barrier (stages >= 2)
            advance(nxt);
        }
        advance(cur);
        if (++s == d.tma_stages) { s = 0; ph ^= 1u; }
    }
    // after a tripped wait: let the boxes still in flight land before the shared memory is given back (bounded)
    if (threadIdx.x == 0 && *abortp) {
        for (int b = 0; b < d.tma_stages; ++b) {
            const unsigned long long t0 = global_timer_ns();
            while (!mbar_try_wait(smem_u32(&full_bar[b]), 0u) && !mbar_try_wait(smem_u32(&full_bar[b]), 1u)) {
                if (global_timer_ns() - t0 > 2000000ull) break;
            }
        }
    }
}

// ------------------------------------------------------------------------------------------------------------
// ROW_SIMT: softmax(scale * x) per row; `lanes_per_row` threads of one warp share a row.
// ------------------------------------------------------------------------------------------------------------
__global__ void tt_softmax_kernel(const RowArgs a) {
    pdl_allow_next();
    pdl_wait_prev();
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

// ROW_SIMT, register-resident form: every lane keeps its share of the row (up to NV 16-byte groups) in registers,
// so x is read from memory once and each exponential is computed once.  Rows of up to lanes_per_row * 4 * NV columns
// whose length is a multiple of 4 and whose pointers are 16-byte aligned; everything else takes the kernel above.
template <int NV>
__global__ void tt_softmax_cached_kernel(const RowArgs a) {
    pdl_allow_next();
    pdl_wait_prev();
    const int lpr = a.lanes_per_row;
    const int sub = threadIdx.x % lpr;
    const long long row = (long long)blockIdx.x * a.rows_per_cta + threadIdx.x / lpr;
    const bool live = row < a.rows;
    const float4* xr = reinterpret_cast<const float4*>(a.x + (live ? row : 0) * (long long)a.cols);
    float4* yr = reinterpret_cast<float4*>(a.y + (live ? row : 0) * (long long)a.cols);
    const int groups = a.cols >> 2;
    float4 v[NV];
    float mx = -INFINITY;
#pragma unroll
    for (int i = 0; i < NV; ++i) {
        const int gidx = sub + i * lpr;
        if (live && gidx < groups) {
            v[i] = __ldg(xr + gidx);
            v[i].x *= a.scale; v[i].y *= a.scale; v[i].z *= a.scale; v[i].w *= a.scale;
            mx = fmaxf(mx, fmaxf(fmaxf(v[i].x, v[i].y), fmaxf(v[i].z, v[i].w)));
        }
    }
    for (int o = lpr >> 1; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    float sum = 0.f;
#pragma unroll
    for (int i = 0; i < NV; ++i) {
        const int gidx = sub + i * lpr;
        if (live && gidx < groups) {
            v[i].x = expf(v[i].x - mx); v[i].y = expf(v[i].y - mx); v[i].z = expf(v[i].z - mx); v[i].w = expf(v[i].w - mx);
            sum += (v[i].x + v[i].y) + (v[i].z + v[i].w);
        }
    }
    for (int o = lpr >> 1; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    const float inv = 1.f / sum;
#pragma unroll
    for (int i = 0; i < NV; ++i) {
        const int gidx = sub + i * lpr;
        if (live && gidx < groups) yr[gidx] = make_float4(v[i].x * inv, v[i].y * inv, v[i].z * inv, v[i].w * inv);
    }
}

// Filters [kout][C][RS] -> [kout][block of 32 channels][tap][channel in block], zero beyond C: the reduction order of the
// tap-major convolution.  One thread per output element; reads walk the channels of a tap (stride RS), writes are
// contiguous.
__global__ void tt_repack_filters_kernel(const float* __restrict__ w, float* __restrict__ out, int kout, int C, int RS, int CB) {
    const long long per_filter = (long long)CB * RS * 32;
    const long long total = (long long)kout * per_filter;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        const long long f = i / per_filter;
        const int rem = (int)(i - f * per_filter);
        const int ci = rem & 31, t2 = rem >> 5;
        const int cb = t2 / RS, tap = t2 - cb * RS;
        const int c = cb * 32 + ci;
        out[i] = c < C ? __ldg(w + (f * C + c) * RS + tap) : 0.f;
    }
}

// A kernel that does nothing, for the launch floor: launched with a record's grid, block size, shared memory,
// cluster shape and dependent-launch attribute, its time is what a launch of that record costs before any work.
__global__ void tt_floor_kernel() {
    pdl_allow_next();
    pdl_wait_prev();
}

// ------------------------------------------------------------------------------------------------------------
// Launchers (called from tt_device.cu)
// ------------------------------------------------------------------------------------------------------------
// Two CTAs fit one SM when each takes at most half of its shared memory (228 KB, of which 1 KB per CTA is the
// system's, plus the kernel's static part) and half of its 512 tensor-memory columns.
static bool gemm_two_per_sm(int smem_bytes, int tmem_cols) { return smem_bytes <= 112 * 1024 && tmem_cols <= 256; }

cudaError_t launch_gemm(const tt_apply_info& I, const GemmArgs& g, const void* tmap_a, const void* tmap_b, const void* tmap_x,
                        cudaStream_t st) {
    static int attr_set_for = -1;
    int dev = 0;
    cudaGetDevice(&dev);
    if (attr_set_for != dev) {
        cudaError_t e = cudaFuncSetAttribute(tt_gemm_tc_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kDynSmemLimit);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(tt_gemm_tc_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, kDynSmemLimit);
        if (e != cudaSuccess) return e;
        attr_set_for = dev;
    }
    CUtensorMap ta, tb, tx;
    memcpy(&ta, tmap_a, sizeof ta);
    memcpy(&tb, tmap_b, sizeof tb);
    memcpy(&tx, tmap_x, sizeof tx);
    dim3 grid(I.grid_x, I.grid_y, I.grid_z);
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid; cfg.blockDim = dim3(kGemmThreads, 1, 1); cfg.dynamicSmemBytes = (size_t)I.smem_bytes; cfg.stream = st;
    cudaLaunchAttribute attr[2];
    int n_attr = 0;
    // the kernel's set-up may overlap the tail of the kernel before it in the stream (it waits before its first
    // global access); captured into a graph this becomes a programmatic dependency edge
    attr[n_attr].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n_attr].val.programmaticStreamSerializationAllowed = 1;
    ++n_attr;
    if (g.cluster) {
        // the splits of one output tile (grid.y) form a thread-block cluster
        attr[n_attr].id = cudaLaunchAttributeClusterDimension;
        attr[n_attr].val.clusterDim.x = 1; attr[n_attr].val.clusterDim.y = (unsigned)g.cluster; attr[n_attr].val.clusterDim.z = 1;
        ++n_attr;
    }
    cfg.attrs = attr; cfg.numAttrs = (unsigned)n_attr;
    // which build runs is the record's choice (ctas_per_sm), resolved by the legaliser
    if (g.two_per_sm && gemm_two_per_sm(I.smem_bytes, g.tmem_cols)) return cudaLaunchKernelEx(&cfg, tt_gemm_tc_kernel<2>, ta, tb, tx, g);
    return cudaLaunchKernelEx(&cfg, tt_gemm_tc_kernel<1>, ta, tb, tx, g);
}

// The persistent form: one CTA (or one pair of CTAs, as a cluster of two) per SM.
cudaError_t launch_gemm_ps(const tt_apply_info& I, const GemmArgs& g, const void* tmap_a, const void* tmap_b, const void* tmap_x,
                           cudaStream_t st) {
    static int attr_set_for = -1, sm_count = 148;
    int dev = 0;
    cudaGetDevice(&dev);
    if (attr_set_for != dev) {
        cudaError_t e = cudaFuncSetAttribute(tt_gemm_ps_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kDynSmemLimit);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(tt_gemm_ps_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, kDynSmemLimit);
        if (e != cudaSuccess) return e;
        cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev);
        attr_set_for = dev;
    }
    CUtensorMap ta, tb, tx;
    memcpy(&ta, tmap_a, sizeof ta);
    memcpy(&tb, tmap_b, sizeof tb);
    memcpy(&tx, tmap_x, sizeof tx);
    const int cg = g.cta_group == 2 ? 2 : 1;
    const long long units = std::min<long long>(g.total_tiles, sm_count / cg);
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)(units * cg), 1, 1); cfg.blockDim = dim3(kGemmThreads, 1, 1);
    cfg.dynamicSmemBytes = (size_t)I.smem_bytes; cfg.stream = st;
    cudaLaunchAttribute attr[2];
    int n_attr = 0;
    attr[n_attr].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n_attr].val.programmaticStreamSerializationAllowed = 1;
    ++n_attr;
    if (cg == 2) {
        attr[n_attr].id = cudaLaunchAttributeClusterDimension;
        attr[n_attr].val.clusterDim.x = 2; attr[n_attr].val.clusterDim.y = 1; attr[n_attr].val.clusterDim.z = 1;
        ++n_attr;
    }
    cfg.attrs = attr; cfg.numAttrs = (unsigned)n_attr;
    if (cg == 2) return cudaLaunchKernelEx(&cfg, tt_gemm_ps_kernel<2>, ta, tb, tx, g);
    return cudaLaunchKernelEx(&cfg, tt_gemm_ps_kernel<1>, ta, tb, tx, g);
}

// Can a cluster of `cluster` CTAs with this much shared memory each be resident at all?
cudaError_t gemm_cluster_fits(int smem_bytes, int cluster, int* fits) {
    cudaError_t e = cudaFuncSetAttribute(tt_gemm_tc_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kDynSmemLimit);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(1, (unsigned)cluster, 1); cfg.blockDim = dim3(kGemmThreads, 1, 1); cfg.dynamicSmemBytes = (size_t)smem_bytes;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 1; attr[0].val.clusterDim.y = (unsigned)cluster; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    int n = 0;
    e = cudaOccupancyMaxActiveClusters(&n, tt_gemm_tc_kernel<1>, &cfg);   // the other build needs no more of anything
    if (e != cudaSuccess) return e;
    *fits = n > 0;
    return cudaSuccess;
}

cudaError_t launch_floor(const tt_apply_info& I, int cluster, cudaStream_t st) {
    static int attr_set_for = -1;
    int dev = 0;
    cudaGetDevice(&dev);
    if (attr_set_for != dev) {
        cudaError_t e = cudaFuncSetAttribute(tt_floor_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kDynSmemLimit);
        if (e != cudaSuccess) return e;
        attr_set_for = dev;
    }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(I.grid_x, I.grid_y, I.grid_z); cfg.blockDim = dim3(I.threads, 1, 1);
    cfg.dynamicSmemBytes = (size_t)I.smem_bytes; cfg.stream = st;
    cudaLaunchAttribute attr[2];
    int n_attr = 0;
    attr[n_attr].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n_attr].val.programmaticStreamSerializationAllowed = 1;
    ++n_attr;
    if (cluster) {
        attr[n_attr].id = cudaLaunchAttributeClusterDimension;
        attr[n_attr].val.clusterDim.x = 1; attr[n_attr].val.clusterDim.y = (unsigned)cluster; attr[n_attr].val.clusterDim.z = 1;
        ++n_attr;
    }
    cfg.attrs = attr; cfg.numAttrs = (unsigned)n_attr;
    return cudaLaunchKernelEx(&cfg, tt_floor_kernel);
}

cudaError_t launch_repack(const float* w, float* out, int kout, int C, int RS, int CB, cudaStream_t st) {
    const long long total = (long long)kout * CB * RS * 32;
    const int blocks = (int)std::min<long long>((total + 255) / 256, 148 * 8);
    tt_repack_filters_kernel<<<blocks, 256, 0, st>>>(w, out, kout, C, RS, CB);
    return cudaGetLastError();
}

// Launch with programmatic stream serialization (the kernels wait before their first global access): in a stream or
// a captured graph the kernel's launch latency and set-up hide behind its predecessor's tail.
template <typename... KArgs, typename... Args>
static cudaError_t launch_serialized(void (*kern)(KArgs...), dim3 grid, unsigned threads, size_t smem, cudaStream_t st, Args&&... args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid; cfg.blockDim = dim3(threads, 1, 1); cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, std::forward<Args>(args)...);
}

cudaError_t launch_dw_tma(const tt_apply_info& I, const DwArgs& dw, const void* tmap_x, cudaStream_t st) {
    CUtensorMap tx;
    memcpy(&tx, tmap_x, sizeof tx);
    dim3 grid(I.grid_x, 1, 1);
    int sm_count = 148, dev_now = 0;
    cudaGetDevice(&dev_now);
    cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev_now);
#define TT_DWT_CASE(RR, SS, RO, WI) \
    if (dw.R == RR && dw.sh == SS && dw.window_rows == RO && dw.items == WI) { \
        static int attr_dev = -1; int dev = 0; cudaGetDevice(&dev); \
        if (attr_dev != dev) { \
            cudaError_t e = cudaFuncSetAttribute(tt_dwconv_tma_kernel<RR, SS, RO, WI>, cudaFuncAttributeMaxDynamicSharedMemorySize, kDynSmemLimit); \
            if (e != cudaSuccess) return e; attr_dev = dev; } \
        int occ = 0; \
        cudaError_t eo = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, tt_dwconv_tma_kernel<RR, SS, RO, WI>, I.threads, (size_t)I.smem_bytes); \
        if (eo != cudaSuccess) return eo; \
        if (occ < 1) return cudaErrorLaunchOutOfResources; \
        /* persistent CTAs: never more than are resident at once (registers may allow fewer than shared memory does) */ \
        grid.x = (unsigned)std::min<long long>(grid.x, (long long)sm_count * occ); \
        return launch_serialized(tt_dwconv_tma_kernel<RR, SS, RO, WI>, grid, (unsigned)I.threads, (size_t)I.smem_bytes, st, tx, dw); }
    TT_DWT_CASE(3, 1, 1, 4) TT_DWT_CASE(3, 1, 2, 4) TT_DWT_CASE(3, 1, 4, 4) TT_DWT_CASE(3, 1, 1, 8) TT_DWT_CASE(3, 1, 2, 8)
    TT_DWT_CASE(3, 2, 1, 4) TT_DWT_CASE(3, 2, 2, 4) TT_DWT_CASE(3, 2, 4, 4) TT_DWT_CASE(3, 2, 1, 8) TT_DWT_CASE(3, 2, 2, 8)
    TT_DWT_CASE(5, 1, 1, 4) TT_DWT_CASE(5, 1, 2, 4) TT_DWT_CASE(5, 1, 4, 4) TT_DWT_CASE(5, 1, 1, 8) TT_DWT_CASE(5, 1, 2, 8)
    TT_DWT_CASE(5, 2, 1, 4) TT_DWT_CASE(5, 2, 2, 4) TT_DWT_CASE(5, 2, 4, 4) TT_DWT_CASE(5, 2, 1, 8) TT_DWT_CASE(5, 2, 2, 8)
#undef TT_DWT_CASE
    return cudaErrorInvalidValue;
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
    if (dw.window_rows > 0) {
        // register-window kernels: one instantiation per (filter size, stride, output rows per thread)
#define TT_DW_CASE(RR, SS, RO, WD) \
        if (dw.R == RR && dw.sh == SS && dw.window_rows == RO && dw.items == WD) return launch_serialized(tt_dwconv_window_kernel<RR, SS, RO, WD>, grid, (unsigned)I.threads, 0, st, dw);
        TT_DW_CASE(3, 1, 1, 4) TT_DW_CASE(3, 1, 2, 4) TT_DW_CASE(3, 1, 4, 4)
        TT_DW_CASE(3, 2, 1, 4) TT_DW_CASE(3, 2, 2, 4) TT_DW_CASE(3, 2, 4, 4)
        TT_DW_CASE(5, 1, 1, 4) TT_DW_CASE(5, 1, 2, 4) TT_DW_CASE(5, 1, 4, 4)
        TT_DW_CASE(5, 2, 1, 4) TT_DW_CASE(5, 2, 2, 4) TT_DW_CASE(5, 2, 4, 4)
        TT_DW_CASE(3, 1, 1, 8) TT_DW_CASE(3, 1, 2, 8) TT_DW_CASE(3, 2, 1, 8) TT_DW_CASE(3, 2, 2, 8)
        TT_DW_CASE(5, 1, 1, 8) TT_DW_CASE(5, 1, 2, 8) TT_DW_CASE(5, 2, 1, 8) TT_DW_CASE(5, 2, 2, 8)
#undef TT_DW_CASE
        return cudaErrorInvalidValue;
    }
    return launch_serialized(tt_dwconv_kernel, grid, (unsigned)I.threads, (size_t)I.smem_bytes, st, dw);
}

cudaError_t launch_row(const tt_apply_info& I, const RowArgs& row, cudaStream_t st) {
    // rows that fit the lanes' registers (and allow 16-byte accesses) are read once
    const int per_lane = row.vec == 4 ? ((row.cols >> 2) + row.lanes_per_row - 1) / row.lanes_per_row : 0;
    if (per_lane >= 1 && per_lane <= 8) {
        const dim3 grid(I.grid_x, 1, 1);
        if (per_lane == 1) return launch_serialized(tt_softmax_cached_kernel<1>, grid, (unsigned)I.threads, 0, st, row);
        if (per_lane == 2) return launch_serialized(tt_softmax_cached_kernel<2>, grid, (unsigned)I.threads, 0, st, row);
        if (per_lane <= 4) return launch_serialized(tt_softmax_cached_kernel<4>, grid, (unsigned)I.threads, 0, st, row);
        return launch_serialized(tt_softmax_cached_kernel<8>, grid, (unsigned)I.threads, 0, st, row);
    }
    return launch_serialized(tt_softmax_kernel, dim3(I.grid_x, 1, 1), (unsigned)I.threads, 0, st, row);
}

}  // namespace tt
