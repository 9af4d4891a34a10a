// Host logic of libtt: workloads, kernel classes, schedule records, the transfer /
// legalisation / validity layer, the selector.  Nothing here touches the device.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <string>
#include <vector>
#include <new>
#include "tt_internal.h"

using namespace tt;

namespace {

uint64_t fnv1a(const void* data, size_t n, uint64_t h = 1469598103934665603ull) {
    const unsigned char* p = static_cast<const unsigned char*>(data);
    for (size_t i = 0; i < n; ++i) { h ^= p[i]; h *= 1099511628211ull; }
    return h;
}

int round_up(int v, int m) { return (v + m - 1) / m * m; }
int pow2_ceil(int v) { int p = 1; while (p < v) p <<= 1; return p; }
int pow2_floor(int v) { int p = 1; while (p * 2 <= v) p <<= 1; return p; }

int family_of(tt_op op) {
    switch (op) {
        case TT_OP_CONV2D: case TT_OP_DENSE: case TT_OP_BATCH_MATMUL: return TT_FAMILY_GEMM_TC;
        case TT_OP_DWCONV2D: return TT_FAMILY_DW_SIMT;
        case TT_OP_SOFTMAX: return TT_FAMILY_ROW_SIMT;
    }
    return -1;
}

bool conv_like(tt_op op) { return op == TT_OP_CONV2D || op == TT_OP_DWCONV2D; }

}  // namespace

namespace tt {

uint64_t class_hash(int op, const tt_shapes& s) {
    // A kernel class is the sequence of operators, regardless of data sizes (Section 4.2).
    int32_t v[5] = {op, s.has_bias != 0, s.act, s.has_residual != 0, op == TT_OP_BATCH_MATMUL ? (s.trans_b != 0) : 0};
    return fnv1a(v, sizeof v);
}

size_t tensor_elems(const tt_workload* w, int which) {
    const tt_shapes& s = w->sh;
    switch (w->op) {
        case TT_OP_CONV2D:
            switch (which) {
                case 0: return (size_t)s.n * s.c * s.h * s.w;
                case 1: return (size_t)s.k * s.c * s.r * s.s;
                case 2: return s.has_bias ? (size_t)s.k : 0;
                case 3: return s.has_residual ? (size_t)s.n * s.k * w->P * w->Q : 0;
                default: return (size_t)s.n * s.k * w->P * w->Q;
            }
        case TT_OP_DWCONV2D:
            switch (which) {
                case 0: return (size_t)s.n * s.c * s.h * s.w;
                case 1: return (size_t)s.c * s.r * s.s;
                case 2: return s.has_bias ? (size_t)s.c : 0;
                case 3: return 0;
                default: return (size_t)s.n * s.c * w->P * w->Q;
            }
        case TT_OP_DENSE:
        case TT_OP_BATCH_MATMUL:
            switch (which) {
                case 0: return (size_t)s.batch * s.m * s.kk;
                case 1: return (size_t)s.batch * s.nn * s.kk;
                case 2: return s.has_bias ? (size_t)s.nn : 0;
                case 3: return s.has_residual ? (size_t)s.batch * s.m * s.nn : 0;
                default: return (size_t)s.batch * s.m * s.nn;
            }
        case TT_OP_SOFTMAX:
            return (which == 0 || which == 4) ? (size_t)s.batch * s.m * s.nn : 0;
    }
    return 0;
}

// ---- legalisation -------------------------------------------------------------------------------------------

// conv2d with k_order = 1: the reduction walks blocks of 32 channels and, inside a block, tap by tap.  Filters are
// re-packed into that order ([filter][block][tap][32 channels], zero-padded) before each run and arrive by TMA;
// the output columns are padded-linear pixels n = p * (W + gap) + q', so that the operand tile of tap (r, s) is the
// pixel-major slab read (r * (W + gap) + s) rows further down -- a view, no expansion.  Columns with q' >= Q are
// computed and dropped.
static bool tap_major_possible(const tt_workload* w) {
    const tt_shapes& s = w->sh;
    const int gap = round_up(std::max(1, std::max(s.pad_w, s.s - 1 - s.pad_w)), 4);
    // (an output row must fit a padded image row: the columns are numbered p * (W + gap) + q')
    return w->op == TT_OP_CONV2D && s.stride_h == 1 && s.stride_w == 1 && (s.w % 4) == 0 && !s.has_residual &&
           s.r * s.s <= 64 && (long long)w->P * w->Q > 1 && w->Q <= s.w + gap;
}

static tt_status legalise_conv_tapmajor(const tt_workload* w, const tt_schedule_record* rec, int mode, Plan* plan) {
    tt_apply_info& I = plan->info;
    const tt_shapes& s = w->sh;
    const bool strict = mode == TT_MODE_STRICT;
    tt_schedule_record L = *rec;
    int changed = 0;
    const int RS = s.r * s.s, CB = (s.c + 31) / 32;
    const int gap = round_up(std::max(1, std::max(s.pad_w, s.s - 1 - s.pad_w)), 4), wp = s.w + gap;
    if (wp > 256) return TT_ERR_RESOURCE;
    const int M = s.k, B = s.n;
    const long long Nl = (long long)w->P * wp;            // padded-linear output pixels
    if (Nl > 0x7fffffffLL) return TT_ERR_RESOURCE;
    const int N = (int)Nl, K = CB * RS * 32;
    // fixed by the mode: filters on the 128 rows, no split-K, one accumulator; a reduction tile is `tps` taps of one
    // 32-channel block (tile_k = 32 * tps, tps a divisor of the tap count, tile_k <= 128)
    int tps = 1;
    for (int d = 1; d <= 4; ++d) if (RS % d == 0 && 32 * d <= rec->tile_k) tps = d;
    const int tk = 32 * tps;
    if (strict && (rec->mma_m_axis == 2 || rec->tile_k != tk || rec->split_k != 1)) return TT_ERR_INVALID_SCHEDULE;
    L.mma_m_axis = 1; L.tile_m = kHwTileM; L.tile_k = tk; L.split_k = 1; L.acc_split = 1; L.slab_tiles = 0; L.k_order = 1;
    if (rec->persistent < 0 || rec->persistent > 1 || rec->cta_group < 0 || rec->cta_group > 2 || rec->ctas_per_sm < 0 ||
        rec->ctas_per_sm > 2 || rec->warp_layout != 0 || rec->precision < 0 || rec->precision > 1)
        return TT_ERR_INVALID_SCHEDULE;
    // both kernel forms walk this reduction order; CTA pairs do not
    const bool persistent = rec->persistent == 1;
    L.persistent = persistent ? 1 : 0; L.cta_group = 1;
    if (rec->cta_group == 2) { if (strict) return TT_ERR_INVALID_SCHEDULE; changed |= TT_CHG_FORM; }
    L.precision = 0;                                      // (no error-compensated products for convolutions)
    if (rec->precision != 0) { if (strict) return TT_ERR_INVALID_SCHEDULE; changed |= TT_CHG_FORM; }
    if (rec->tile_m != kHwTileM) changed |= TT_CHG_TILE_M;
    if (rec->tile_k != tk) changed |= TT_CHG_TILE_K;
    if (rec->split_k != 1) changed |= TT_CHG_SPLIT_K;
    int tn = std::min(256, std::max(16, round_up(rec->tile_n, 16)));
    tn = std::min(tn, round_up(N, 16));
    if (tn != rec->tile_n) changed |= TT_CHG_TILE_N;
    L.tile_n = tn;
    const int k_tiles = CB * RS / tps;
    // (the persistent form's filter pipeline runs on across tiles: no point in clamping it to one tile's reduction)
    int st = persistent ? std::min(kMaxStages, rec->stages) : std::min(std::min(kMaxStages, rec->stages), k_tiles);
    if (st != rec->stages) changed |= TT_CHG_STAGES;
    if (strict && (changed & ~TT_CHG_TILE_M)) return TT_ERR_INVALID_SCHEDULE;
    // shared memory: filter stages | NCHW staging of a block (TMA box [32][in_rows][wp], one buffer) | pixel-major slab
    // (two buffers of (in_rows * wp + reach) rows of 128 bytes)
    const int out_rows = std::min(w->P, (tn + wp - 2) / wp + 1);
    const int in_rows = out_rows - 1 + s.r;
    if (in_rows > 256) return TT_ERR_RESOURCE;
    const unsigned a_stage = (unsigned)tps * kHwTileM * 128;
    const long long s_buf = (((long long)32 * in_rows * wp) * 4 + 127) / 128 * 128;
    // furthest row a tile's views can touch (all tile_n rows are read, also those of pixels past the image)
    const long long pm_rows = (long long)((tn + wp - 2) / wp + s.r) * wp + s.s + gap + 8;
    const long long pm_buf = pm_rows * 128;
    const int nbuf = (CB > 1 || persistent) ? 2 : 1;
    long long smem = 0;
    const long long min_pipe = (long long)kGatherWarps * 32 * 36 * 4;
    // persistent form: the read-out has its own staging area (the pipeline buffers are busy with the next tile), and
    // the NCHW staging ring is two boxes deep when that fits
    const long long epi = persistent ? 4ll * 32 * 36 * 4 : 0;
    int sd = persistent ? 2 : 1;
    for (;;) {
        const long long pipe = persistent ? (long long)st * a_stage : std::max<long long>((long long)st * a_stage, min_pipe);
        smem = pipe + sd * s_buf + nbuf * pm_buf + epi + 1024;
        if (smem <= kDynSmemLimit) break;
        if (sd > 1) { --sd; continue; }
        if (strict || st <= 1) break;
        --st; changed |= TT_CHG_STAGES;
    }
    L.stages = st;
    const long long pipe = persistent ? (long long)st * a_stage : std::max<long long>((long long)st * a_stage, min_pipe);
    const int tiles_m = (M + kHwTileM - 1) / kHwTileM, tiles_n = (N + tn - 1) / tn;
    const int tmem_cols_t = std::max(32, pow2_ceil(persistent ? 2 * tn : tn));
    if (persistent) {
        L.ctas_per_sm = 1;
        if (rec->ctas_per_sm == 2) { if (strict) return TT_ERR_INVALID_SCHEDULE; changed |= TT_CHG_FORM; }
    } else {
        // which build: two CTAs per SM need half the shared memory and half the tensor memory each
        const bool fits2 = smem <= 112 * 1024 && tmem_cols_t <= 256;
        const long long ctas = (long long)tiles_m * tiles_n * B;
        int cps = rec->ctas_per_sm == 0 ? ((ctas > 2 * 148 && fits2) ? 2 : 1) : rec->ctas_per_sm;
        if (cps == 2 && !fits2) { if (strict) return TT_ERR_INVALID_SCHEDULE; cps = 1; changed |= TT_CHG_FORM; }
        L.ctas_per_sm = cps;
    }
    I = tt_apply_info{};
    I.legal = L; I.changed = changed;
    I.grid_x = tiles_m * tiles_n; I.grid_y = 1; I.grid_z = B;
    const long long units = (long long)tiles_m * tiles_n * B;
    if (persistent) {
        if (units > 0x7fffffffLL) return TT_ERR_RESOURCE;
        I.grid_x = (int)std::min<long long>(units, 148); I.grid_z = 1;      // the launcher clamps to the device's SM count
    }
    I.threads = kGemmThreads;
    I.smem_bytes = (int)std::min<long long>(persistent ? std::max<long long>(smem, 116 * 1024) : smem, 0x7fffffff);
    I.tmem_cols = tmem_cols_t;
    I.workspace_bytes = (int64_t)M * K * 4;              // the re-packed filters
    I.launches = 2;
    if (smem > kDynSmemLimit || (long long)tiles_m * tiles_n > 0x7fffffffLL || B > 65535) return TT_ERR_RESOURCE;
    plan->swap_ab = false;
    plan->gm = M; plan->gn = N; plan->gk = K; plan->gbatch = B;
    plan->partial_bytes = 0;
    plan->repack = true; plan->repack_cb = CB;
    plan->a_tensor = 1; plan->b_tensor = 0;               // A: filters (re-packed), B: the image
    GemmArgs& g = plan->g;
    g = GemmArgs{};
    g.M = M; g.N = N; g.K = K; g.batch = B;
    g.tile_n = tn; g.tile_k = tk; g.stages = st;
    g.k_tiles = k_tiles; g.k_tiles_per_split = k_tiles; g.split_k = 1;
    g.tiles_m = tiles_m; g.tiles_n = tiles_n; g.raster = L.raster;
    g.atom_k = 32; g.n_atoms = tps; g.row_bytes = 128; g.swz_mask = 7;
    g.a_stage_bytes = a_stage; g.b_stage_bytes = 0; g.tx_bytes = a_stage;
    g.tmem_cols = (unsigned)I.tmem_cols; g.n_acc = 1; g.cluster = 0;
    g.idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((unsigned)(tn >> 3) << 17) | ((unsigned)(kHwTileM >> 4) << 24);
    g.a_mode = OPM_TMA; g.a_rs = K; g.a_ks = 1; g.a_bs = 0; g.a_tma_batched = 0;
    g.b_mode = OPM_IM2COL_T; g.b_rs = 0; g.b_ks = 0; g.b_bs = (long long)s.c * s.h * s.w; g.b_tma_batched = 1;
    g.y_ms = (long long)w->P * w->Q; g.y_ns = 1; g.y_bs = (long long)s.k * w->P * w->Q;
    g.bias_mode = s.has_bias ? 1 : 0;
    g.act = s.act;
    g.C = s.c; g.H = s.h; g.W = s.w; g.R = s.r; g.S = s.s; g.Q = w->Q; g.Pout = w->P;
    g.sh = 1; g.sw = 1; g.ph = s.pad_h; g.pw = s.pad_w;
    g.vec_store = (w->Q % 4 == 0 && ((long long)w->P * w->Q) % 4 == 0) ? 1 : 0;   // a lane's four columns: one aligned 16-byte store
    g.tap_major = 1;
    g.two_per_sm = L.ctas_per_sm == 2;
    g.b_rows_cta = tn; g.cta_group = 1;
    g.persistent = persistent ? 1 : 0; g.total_tiles = (int)units; g.stg_depth = sd;
    g.epi_off = (unsigned)(pipe + (long long)sd * s_buf + (long long)nbuf * pm_buf);
    g.slab_tma = 1; g.slab_tiles = RS / tps; g.slab_nbuf = 1; g.pm_nbuf = nbuf;
    g.slab_off = (unsigned)pipe; g.slab_buf_bytes = (unsigned)s_buf;
    g.slab_wp = wp; g.slab_gap = gap; g.slab_chpitch = in_rows * wp; g.slab_in_rows = in_rows; g.slab_rstep = 1;
    g.slab_box_ch = std::min(32, s.c);                   // (fewer than 32 channels: the rest of the staging buffer stays zero)
    g.slab_box_bytes = (unsigned)((long long)g.slab_box_ch * in_rows * wp * 4);
    g.slab_vec16 = 1;
    g.pm_off = (unsigned)(pipe + (long long)sd * s_buf); g.pm_buf_bytes = (unsigned)pm_buf;
    return TT_OK;
}

static tt_status legalise_gemm(const tt_workload* w, const tt_schedule_record* rec, int mode, Plan* plan) {
    if (rec->k_order < 0 || rec->k_order > 1) return TT_ERR_INVALID_SCHEDULE;
    if (rec->k_order == 1) {
        if (tap_major_possible(w)) return legalise_conv_tapmajor(w, rec, mode, plan);
        if (mode == TT_MODE_STRICT) return TT_ERR_INVALID_SCHEDULE;       // no such reduction order on this kernel
    }
    tt_apply_info& I = plan->info;
    tt_schedule_record L = *rec;
    int changed = 0;
    const bool strict = mode == TT_MODE_STRICT;
    if (rec->tile_m <= 0 || rec->tile_n <= 0 || rec->tile_k <= 0 || rec->stages <= 0 || rec->split_k <= 0 ||
        rec->raster < 0 || rec->raster > 1 || rec->mma_m_axis < 0 || rec->mma_m_axis > 2 || rec->persistent < 0 ||
        rec->persistent > 1 || rec->cta_group < 0 || rec->cta_group > 2 || rec->ctas_per_sm < 0 || rec->ctas_per_sm > 2 ||
        rec->warp_layout != 0 || rec->precision < 0 || rec->precision > 1)
        return TT_ERR_INVALID_SCHEDULE;
    // Which output axis becomes the accumulator's 128 rows.  Left to the library (0), the shorter-than-a-tile
    // axis goes to the MMA's N side, where 16..256 columns are legal.
    tt_shapes s = w->sh;                                  // a copy: a pointwise convolution is re-viewed below
    int P = w->P, Q = w->Q;
    bool swap = rec->mma_m_axis == 2;
    if (rec->mma_m_axis == 0) swap = w->view.gm <= 64 && w->view.gn > w->view.gm;
    L.mma_m_axis = swap ? 2 : 1;
    L.k_order = 0;
    if (rec->k_order != 0) changed |= TT_CHG_KORDER;    // reformulated: the stored channel-major order
    plan->repack = false;
    plan->swap_ab = swap;
    plan->gm = swap ? w->view.gn : w->view.gm;
    plan->gn = swap ? w->view.gm : w->view.gn;
    const int M = plan->gm, N = plan->gn, K = plan->gk, B = plan->gbatch;
    // A split factor larger than the loop itself is invalid code when nothing may be reformulated (Section 4.2).
    if (strict && (rec->tile_m > round_up(M, 32) || rec->tile_n > round_up(N, 16) || rec->tile_k > round_up(K, 8)))
        return TT_ERR_INVALID_SCHEDULE;
    // tile_m: the accumulator always spans 128 tensor-memory lanes; smaller logical tiles leave rows idle.
    L.tile_m = kHwTileM;
    if (L.tile_m != rec->tile_m) changed |= TT_CHG_TILE_M;
    // tile_n: legal MMA N for M = 128 is a multiple of 16 in [16, 256]; no wider than the padded extent.
    int tn = std::min(256, std::max(16, round_up(rec->tile_n, 16)));
    tn = std::min(tn, round_up(N, 16));
    if (tn != rec->tile_n) changed |= TT_CHG_TILE_N;
    L.tile_n = tn;
    // tile_k: power of two in [8, 128] (one to four 128-byte swizzle atoms, or one 32/64-byte atom).
    int tk = std::min(128, std::max(8, pow2_floor(rec->tile_k)));
    tk = std::min(tk, std::max(8, pow2_ceil(K)));
    if (tk != rec->tile_k) changed |= TT_CHG_TILE_K;
    L.tile_k = tk;
    int st = std::min(kMaxStages, rec->stages);
    if (st != rec->stages) changed |= TT_CHG_STAGES;
    L.stages = st;
    const int k_tiles = (K + tk - 1) / tk;
    // The persistent form: both operands must be reachable by TMA -- K-major with 16-byte rows, or row-contiguous (the
    // image of a pointwise convolution, the second operand of an NN batch_matmul) with 16-byte row pitch.
    // Error-compensated products need both operands as K-major TMA tiles (their remainders are worked out in place, tile by
    // tile) and exist in the one-tile form only: dense and batch_matmul NT with 16-byte rows.
    bool x3 = rec->precision == 1;
    if (x3 && !((w->op == TT_OP_DENSE || (w->op == TT_OP_BATCH_MATMUL && w->sh.trans_b)) && (K % 4) == 0)) {
        if (strict) return TT_ERR_INVALID_SCHEDULE;
        x3 = false; changed |= TT_CHG_FORM;
    }
    L.precision = x3 ? 1 : 0;
    bool persistent = rec->persistent == 1;
    if (persistent && x3) { if (strict) return TT_ERR_INVALID_SCHEDULE; persistent = false; changed |= TT_CHG_FORM; }
    {
        const tt_shapes& o = w->sh;
        bool can = (K % 4) == 0;
        if (w->op == TT_OP_CONV2D)
            can = can && o.r == 1 && o.s == 1 && o.stride_h == 1 && o.stride_w == 1 && o.pad_h == 0 && o.pad_w == 0 &&
                  ((long long)o.h * o.w) % 4 == 0;
        else if (w->op == TT_OP_BATCH_MATMUL && !o.trans_b)
            can = can && (o.nn % 4) == 0;
        if (persistent && !can) { if (strict) return TT_ERR_INVALID_SCHEDULE; persistent = false; changed |= TT_CHG_FORM; }
    }
    const bool mn_operand = persistent && (w->op == TT_OP_CONV2D || (w->op == TT_OP_BATCH_MATMUL && !w->sh.trans_b));
    int cg = rec->cta_group == 2 ? 2 : 1;
    if (cg == 2 && (!persistent || mn_operand || tn < 32)) { if (strict) return TT_ERR_INVALID_SCHEDULE; cg = 1; changed |= TT_CHG_FORM; }
    L.persistent = persistent ? 1 : 0;
    L.cta_group = cg;
    int sk = persistent ? 1 : rec->split_k;
    if (sk > k_tiles) {
        if (strict) return TT_ERR_INVALID_SCHEDULE;
        sk = k_tiles;
    }
    const int per_split = (k_tiles + sk - 1) / sk;
    sk = (k_tiles + per_split - 1) / per_split;          // every split owns at least one reduction tile
    if (sk != rec->split_k) changed |= TT_CHG_SPLIT_K;
    L.split_k = sk;
    // accumulators: a power of two, all of them inside the 512 columns of tensor memory, none left without a step
    if (rec->acc_split < 0) return TT_ERR_INVALID_SCHEDULE;
    int nacc = (persistent || x3) ? 1 : std::min(8, pow2_floor(std::max(1, rec->acc_split)));
    while (nacc > 1 && (nacc * tn > 512 || (long long)nacc > (long long)per_split * (tk / 8))) nacc >>= 1;
    if (nacc != std::max(1, rec->acc_split)) { if (strict) return TT_ERR_INVALID_SCHEDULE; changed |= TT_CHG_ACC; }
    L.acc_split = nacc;
    // buffers beyond the reduction tiles of one CTA would never be filled
    // (the persistent form's pipeline runs on across tiles: there the depth is bounded by shared memory alone)
    if (!persistent && st > per_split) { st = per_split; changed |= TT_CHG_STAGES; L.stages = st; }
    if (strict && (changed & ~TT_CHG_TILE_M)) return TT_ERR_INVALID_SCHEDULE;

    const int atom_k = std::min(tk, 32), n_atoms = tk / atom_k, row_bytes = atom_k * 4;
    const unsigned a_stage = (unsigned)n_atoms * kHwTileM * row_bytes;
    const unsigned b_stage = (unsigned)n_atoms * (tn / cg) * row_bytes;
    if (persistent) {
        // ---- the persistent form: its own shared-memory plan, grid and arguments ----
        const tt_shapes& o = w->sh;
        const bool conv1 = w->op == TT_OP_CONV2D, nn = w->op == TT_OP_BATCH_MATMUL && !o.trans_b;
        // logical operands U (rows i of the output) and V (columns j): which of them is row-contiguous
        const bool u_mn = false, v_mn = conv1 || nn;
        const bool a_mn = swap ? v_mn : u_mn, b_mn = swap ? u_mn : v_mn;
        const unsigned stg_a = a_mn ? (unsigned)(tk * kHwTileM * 4) : 0u, stg_b = b_mn ? (unsigned)(tk * tn * 4) : 0u;
        const long long epi = 4ll * 32 * 36 * 4;
        // the staging ring of a row-contiguous operand has its own depth (record field slab_tiles; 0 = as deep as fits,
        // at most 8): it is what is in flight from DRAM, while the K-major stages only decouple transposing from multiplying
        if (rec->slab_tiles < 0) return TT_ERR_INVALID_SCHEDULE;
        const bool any_stg = stg_a + stg_b > 0;
        int sd = any_stg ? (rec->slab_tiles == 0 ? kMaxStages : std::min(kMaxStages, rec->slab_tiles)) : 0;
        long long smem_p = 0;
        for (;;) {
            smem_p = (long long)st * (a_stage + b_stage) + (long long)sd * (stg_a + stg_b) + epi + 1024;
            if (smem_p <= kDynSmemLimit) break;
            if (any_stg && sd > 1 && (rec->slab_tiles == 0 || !strict) && (rec->slab_tiles == 0 || sd >= st)) { --sd; continue; }
            if (strict || st <= 1) break;
            --st; changed |= TT_CHG_STAGES;
        }
        if (any_stg && rec->slab_tiles != 0 && sd != rec->slab_tiles) { if (strict) return TT_ERR_INVALID_SCHEDULE; changed |= TT_CHG_SLAB; }
        if (!any_stg && rec->slab_tiles != 0) changed |= TT_CHG_SLAB;
        L.stages = st; L.split_k = 1; L.acc_split = 1; L.slab_tiles = (any_stg && rec->slab_tiles != 0) ? sd : 0; L.ctas_per_sm = 1;
        if (rec->ctas_per_sm == 2) { if (strict) return TT_ERR_INVALID_SCHEDULE; changed |= TT_CHG_FORM; }
        if (strict && (changed & ~TT_CHG_TILE_M)) return TT_ERR_INVALID_SCHEDULE;
        const int rows_m = kHwTileM * cg;
        const int tiles_m = (M + rows_m - 1) / rows_m, tiles_n = (N + tn - 1) / tn;
        const long long units = (long long)tiles_m * tiles_n * B;
        if (units > 0x7fffffffLL) return TT_ERR_RESOURCE;
        I = tt_apply_info{};
        I.legal = L; I.changed = changed;
        I.grid_x = (int)std::min<long long>(units, 148 / cg) * cg; I.grid_y = 1; I.grid_z = 1;   // the launcher clamps to the device's SM count
        I.threads = kGemmThreads;
        // one CTA per SM: ask for more than half of an SM's shared memory
        I.smem_bytes = (int)std::max<long long>(smem_p, 116 * 1024);
        I.tmem_cols = std::max(32, pow2_ceil(2 * tn));
        I.workspace_bytes = 0; I.launches = 1;
        plan->partial_bytes = 0;
        if (smem_p > kDynSmemLimit) return TT_ERR_RESOURCE;
        GemmArgs& g = plan->g;
        g = GemmArgs{};
        g.M = M; g.N = N; g.K = K; g.batch = B;
        g.tile_n = tn; g.tile_k = tk; g.stages = st;
        g.k_tiles = k_tiles; g.k_tiles_per_split = k_tiles; g.split_k = 1;
        g.tiles_m = tiles_m; g.tiles_n = tiles_n; g.raster = L.raster;
        g.atom_k = atom_k; g.n_atoms = n_atoms; g.row_bytes = row_bytes;
        g.swz_mask = row_bytes == 128 ? 7 : (row_bytes == 64 ? 3 : 1);
        g.a_stage_bytes = a_stage; g.b_stage_bytes = b_stage;
        g.tmem_cols = (unsigned)I.tmem_cols; g.n_acc = 1; g.cluster = 0;
        g.idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((unsigned)(tn >> 3) << 17) | ((unsigned)(rows_m >> 4) << 24);
        g.persistent = 1; g.cta_group = cg; g.total_tiles = (int)units;
        g.a_mn = a_mn; g.b_mn = b_mn; g.b_rows_cta = tn / cg;
        g.stg_depth = std::max(sd, 1);
        g.a_stg_off = (unsigned)((long long)st * (a_stage + b_stage));
        g.b_stg_off = g.a_stg_off + (unsigned)sd * stg_a;
        g.stg_a_bytes = stg_a; g.stg_b_bytes = stg_b;
        g.epi_off = g.b_stg_off + (unsigned)sd * stg_b;
        struct Opnd { int mode; long long rs, ks, bs; int batched; } U{}, V{};
        long long y_is, y_js, y_bs;
        int bias_on;
        if (conv1) {
            const long long hw = (long long)o.h * o.w;
            U = {OPM_TMA, K, 1, 0, 0};                              // filters [k][c]
            V = {OPM_TMA_MN, 1, hw, (long long)o.c * hw, 1};        // image: pixel index contiguous, channels hw apart
            y_is = hw; y_js = 1; y_bs = (long long)o.k * hw; bias_on = 1;
        } else if (w->op == TT_OP_DENSE) {
            U = {OPM_TMA, K, 1, 0, 0};
            V = {OPM_TMA, K, 1, 0, 0};
            y_is = o.nn; y_js = 1; y_bs = 0; bias_on = 2;
        } else {
            U = {OPM_TMA, K, 1, (long long)o.m * K, 1};
            if (o.trans_b) V = {OPM_TMA, K, 1, (long long)o.nn * K, 1};
            else V = {OPM_TMA_MN, 1, o.nn, (long long)o.nn * K, 1};
            y_is = o.nn; y_js = 1; y_bs = (long long)o.m * o.nn; bias_on = 2;
        }
        const int u_tensor = conv1 ? 1 : 0;
        plan->a_tensor = swap ? 1 - u_tensor : u_tensor;
        plan->b_tensor = 1 - plan->a_tensor;
        const Opnd& A = swap ? V : U;
        const Opnd& Bo = swap ? U : V;
        g.a_mode = A.mode; g.a_rs = A.rs; g.a_ks = A.ks; g.a_bs = A.bs; g.a_tma_batched = A.batched;
        g.b_mode = Bo.mode; g.b_rs = Bo.rs; g.b_ks = Bo.ks; g.b_bs = Bo.bs; g.b_tma_batched = Bo.batched;
        g.y_ms = swap ? y_js : y_is; g.y_ns = swap ? y_is : y_js; g.y_bs = y_bs;
        g.bias_mode = o.has_bias ? (swap ? 3 - bias_on : bias_on) : 0;
        g.act = o.act;
        g.tx_bytes = (a_mn ? 0 : a_stage) + (b_mn ? 0 : b_stage);
        g.vec_store = (g.y_ns == 1 && g.y_ms % 4 == 0 && g.y_bs % 4 == 0) ? 1 : 0;
        return TT_OK;
    }
    // Shared memory: pipeline buffers (reused by the epilogue as a 32 x 36-float staging area per warp), then for
    // conv2d the k-table (one word per reduction index of a CTA's K range) and the slab of input rows from which
    // the im2col operand is expanded; 1 KB of alignment slack.
    // A slab row is an image row followed by `gap` zeros (the left/right padding of neighbouring rows share them).
    // Per channel the slab holds, for each of the output rows a tile can span, the input rows its filter rows
    // touch: consecutive rows when stride <= filter height, else `r` rows per output row.  A chunk holds the
    // channels that `slab_tiles` consecutive reduction tiles touch; two buffers when there are several chunks.
    // split_k of 2..8: the splits of a tile form a thread-block cluster and reduce through distributed shared memory
    // (each sends the bands of its partial tile to the CTAs that finish them); beyond 8 the partial tiles go through
    // a global workspace and the split that arrives last adds them up
    const int cluster = (sk >= 2 && sk <= 8) ? sk : 0;
    // the read-out stages through the pipeline buffers (idle by then): a 32 x 36 float block per warp, or, for the
    // cluster reduction, this split's whole partial tile in the layout of the reduction area
    const long long min_pipe = std::max<long long>((long long)kGatherWarps * 32 * 36 * 4, cluster ? 4LL * kHwTileM * (tn + 4) : 0);
    // cluster reduction area, apart from the pipeline buffers (peers write into it while this CTA may still be in its
    // main loop): per OTHER split, this CTA's band of the tile -- rows x (tile_n + 4) or columns x 128 floats
    const long long red_bytes = cluster ? (4 * std::max<long long>((long long)(sk - 1) * ((kHwTileM + sk - 1) / sk) * (tn + 4),
                                                                    (long long)(sk - 1) * ((tn + sk - 1) / sk) * kHwTileM) + 127) / 128 * 128 : 0;
    const bool conv = w->op == TT_OP_CONV2D;
    const long long ktab = conv ? (((long long)per_split * tk * 4 + 127) / 128) * 128 : 0;
    int sl_tiles = 0, sl_nbuf = 0, sl_wp = 0, sl_gap = 0, sl_chpitch = 0, sl_in_rows = 0, sl_rstep = 1;
    long long sl_buf_bytes = 0, chp = 0;
    const int RS = conv ? s.r * s.s : 1;
    if (conv) {
        if (rec->slab_tiles < 0) return TT_ERR_INVALID_SCHEDULE;
        if (strict && rec->slab_tiles > per_split) return TT_ERR_INVALID_SCHEDULE;
        const int pix_rows = swap ? kHwTileM : tn;       // output pixels per tile of the im2col operand
        // A pointwise convolution (1x1, stride 1, no padding) sees no neighbourhood: its H x W pixels are one run of
        // H*W values per channel, and any H' x W' with the same product is the same kernel.  Rows of W' pixels with
        // W' the largest multiple of 4 that divides both H*W and the tile's pixel count make every tile a whole
        // number of rows, so a slab chunk holds exactly the tile's pixels (the image's own rows would add up to a
        // row on either side: 224 staged pixels for 128 at 56 x 56).
        bool whole_rows = false;
        if (s.r == 1 && s.s == 1 && s.stride_h == 1 && s.stride_w == 1 && s.pad_h == 0 && s.pad_w == 0) {
            const long long hw = (long long)s.h * s.w;
            int best = 0;
            for (int d = 16; d <= 248 && d <= pix_rows; d += 4)
                if (hw % d == 0 && pix_rows % d == 0) best = d;
            if (best > 0) { s.w = best; s.h = (int)(hw / best); P = s.h; Q = s.w; whole_rows = true; }
        }
        const int out_rows = whole_rows ? std::min(P, pix_rows / Q) : std::min(P, (pix_rows + 2 * Q - 2) / Q);
        sl_rstep = std::min(s.stride_h, s.r);
        sl_in_rows = s.stride_h <= s.r ? (out_rows - 1) * s.stride_h + s.r : out_rows * s.r;
        sl_gap = round_up(std::max(1, std::max(s.pad_w, s.s - 1 - s.pad_w)), 4);
        sl_wp = s.w + sl_gap;
        chp = round_up(sl_in_rows * sl_wp, 4);
        if (chp * (long long)s.c >= (1ll << 28) || s.w > 4095 || sl_in_rows > 4095) return TT_ERR_RESOURCE;
        sl_chpitch = (int)chp;
    }
    // TMA can stage the slab when image rows are 16-byte multiples and consecutive slab rows are consecutive image
    // rows; a chunk is then one box of at most 256 channels
    const bool slab_tma = conv && (s.w % 4) == 0 && s.stride_h <= s.r && sl_wp <= 256 && sl_in_rows <= 256;
    auto chunk_channels = [&](long long tiles) { return std::min<long long>(s.c, (tiles * tk + RS - 2) / RS + 1); };
    auto chunk_bytes = [&](long long tiles) {
        // a tail of gap + 4 zeros follows the last row of the last channel
        return ((chunk_channels(tiles) * chp + sl_gap + 4) * 4 + 127) / 128 * 128;
    };
    long long smem = 0;
    for (;;) {
        const long long pipe_try = std::max<long long>((long long)st * (a_stage + b_stage) * (x3 ? 2 : 1), min_pipe);
        long long slab_total = 0;
        bool fits = true;
        if (conv) {
            const long long budget = kDynSmemLimit - 1024 - pipe_try - ktab - red_bytes;
            // largest chunk not above the request that fits (one buffer if it covers the CTA's whole K range)
            int t = rec->slab_tiles == 0 ? per_split : std::min(rec->slab_tiles, per_split);
            while (t >= 1 && ((t >= per_split ? 1 : 2) * chunk_bytes(t) > budget || (slab_tma && chunk_channels(t) > 256))) --t;
            fits = t >= 1;
            sl_tiles = std::max(t, 1);
            sl_nbuf = sl_tiles >= per_split ? 1 : 2;
            sl_buf_bytes = chunk_bytes(sl_tiles);
            slab_total = sl_nbuf * sl_buf_bytes;
        }
        smem = pipe_try + ktab + slab_total + red_bytes + 1024;
        if (fits && smem <= kDynSmemLimit) break;
        // reformulate: a shallower pipeline leaves room (never in strict mode, never below one buffer)
        if (strict || st <= 1) break;
        --st;
        changed |= TT_CHG_STAGES;
    }
    L.stages = st;
    const long long pipe = std::max<long long>((long long)st * (a_stage + b_stage) * (x3 ? 2 : 1), min_pipe);
    if (conv) {
        if (rec->slab_tiles != 0 && sl_tiles != rec->slab_tiles) {
            if (strict) return TT_ERR_INVALID_SCHEDULE;
            changed |= TT_CHG_SLAB;
        }
        L.slab_tiles = rec->slab_tiles == 0 ? 0 : sl_tiles;
    } else {
        L.slab_tiles = 0;
    }
    int tmem_cols = std::max(32, pow2_ceil(nacc * tn));
    const int tiles_m = (M + kHwTileM - 1) / kHwTileM, tiles_n = (N + tn - 1) / tn;
    if ((long long)tiles_m * tiles_n > 0x7fffffffLL || sk > 65535 || B > 65535) return TT_ERR_RESOURCE;

    {
        // which build: two CTAs per SM need half the shared memory and half the tensor memory each
        const bool fits2 = smem <= 112 * 1024 && tmem_cols <= 256;
        const long long ctas = (long long)tiles_m * tiles_n * sk * B;
        int cps = rec->ctas_per_sm == 0 ? ((ctas > 2 * 148 && fits2) ? 2 : 1) : rec->ctas_per_sm;
        if (cps == 2 && !fits2) { if (strict) return TT_ERR_INVALID_SCHEDULE; cps = 1; changed |= TT_CHG_FORM; }
        L.ctas_per_sm = cps;
    }
    I = tt_apply_info{};
    I.legal = L;
    I.changed = changed;
    I.grid_x = tiles_m * tiles_n; I.grid_y = sk; I.grid_z = B;
    I.threads = kGemmThreads;
    I.smem_bytes = (int)std::min<long long>(smem, 0x7fffffff);
    I.tmem_cols = tmem_cols;
    // split-K workspace: partial tiles, then one arrival counter per (batch, tile)
    const bool ws = sk > 1 && cluster == 0;
    plan->partial_bytes = ws ? (((long long)sk * B * M * N * 4 + 255) / 256) * 256 : 0;
    I.workspace_bytes = ws ? plan->partial_bytes + (int64_t)B * tiles_m * tiles_n * 4 : 0;
    I.launches = 1;
    if (smem > kDynSmemLimit) return TT_ERR_RESOURCE;

    GemmArgs& g = plan->g;
    g = GemmArgs{};
    g.M = M; g.N = N; g.K = K; g.batch = B;
    g.tile_n = tn; g.tile_k = tk; g.stages = st;
    g.k_tiles = k_tiles; g.k_tiles_per_split = per_split; g.split_k = sk;
    g.tiles_m = tiles_m; g.tiles_n = tiles_n; g.raster = L.raster;
    g.atom_k = atom_k; g.n_atoms = n_atoms; g.row_bytes = row_bytes;
    g.swz_mask = row_bytes == 128 ? 7 : (row_bytes == 64 ? 3 : 1);
    g.a_stage_bytes = a_stage; g.b_stage_bytes = b_stage;
    g.ktab_off = (unsigned)pipe;
    g.slab_off = (unsigned)(pipe + ktab);
    g.red_off = (unsigned)(pipe + ktab + (long long)sl_nbuf * sl_buf_bytes);
    g.slab_buf_bytes = (unsigned)sl_buf_bytes; g.slab_nbuf = sl_nbuf; g.slab_tiles = sl_tiles;
    g.slab_wp = sl_wp; g.slab_gap = sl_gap; g.slab_chpitch = sl_chpitch; g.slab_in_rows = sl_in_rows;
    g.slab_rstep = sl_rstep;
    g.slab_tma = slab_tma ? 1 : 0;
    if (slab_tma) {
        g.slab_box_ch = (int)chunk_channels(sl_tiles);
        g.slab_box_bytes = (unsigned)((long long)g.slab_box_ch * chp * 4);
    }
    g.magic_rstep = sl_rstep > 1 ? (unsigned)((0x100000000ull + sl_rstep - 1) / sl_rstep) : 0u;
    g.slab_vec16 = (s.w % 4) == 0;
    {
        const unsigned wpieces = (unsigned)(g.slab_vec16 ? s.w / 4 : s.w);
        g.magic_wpieces = wpieces > 1 ? (unsigned)((0x100000000ull + wpieces - 1) / wpieces) : 0u;
        g.magic_in_rows = sl_in_rows > 1 ? (unsigned)((0x100000000ull + sl_in_rows - 1) / sl_in_rows) : 0u;
    }
    g.tmem_cols = (unsigned)tmem_cols;
    g.n_acc = nacc;
    g.cluster = cluster;
    g.two_per_sm = L.ctas_per_sm == 2;
    g.x3 = x3 ? 1 : 0;
    g.b_rows_cta = tn; g.cta_group = 1;
    // Instruction descriptor, kind::tf32: D = F32 (bits 4-5 = 1), A and B = TF32 (bits 7-9, 10-12 = 2), both
    // K-major (bits 15, 16 = 0), N >> 3 at bits 17-22, M >> 4 at bits 24-28.
    g.idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((unsigned)(tn >> 3) << 17) | ((unsigned)(kHwTileM >> 4) << 24);
    // Operands of the logical contraction Y[b][i][j] = sum_k U[b][i][k] V[b][j][k], then the optional swap.
    struct Opnd { int mode; long long rs, ks, bs; int batched; } U{}, V{};
    long long y_is, y_js, y_bs;
    int bias_on;   // 1: bias indexed by i, 2: by j
    const bool k4 = (K % 4) == 0;
    if (w->op == TT_OP_CONV2D) {
        U = {k4 ? OPM_TMA : OPM_GATHER_K, K, 1, 0, 0};                         // filters [k][c*r*s], shared by images
        V = {OPM_IM2COL, 0, 0, (long long)s.c * s.h * s.w, 1};                 // pixels x (c,r,s) gathered from NCHW
        y_is = (long long)P * Q; y_js = 1; y_bs = (long long)s.k * P * Q; bias_on = 1;
    } else if (w->op == TT_OP_DENSE) {
        U = {k4 ? OPM_TMA : OPM_GATHER_K, K, 1, 0, 0};
        V = {k4 ? OPM_TMA : OPM_GATHER_K, K, 1, 0, 0};
        y_is = s.nn; y_js = 1; y_bs = 0; bias_on = 2;
    } else {
        U = {k4 ? OPM_TMA : OPM_GATHER_K, K, 1, (long long)s.m * K, 1};
        if (s.trans_b) V = {k4 ? OPM_TMA : OPM_GATHER_K, K, 1, (long long)s.nn * K, 1};
        else V = {OPM_GATHER_ROWS, 1, s.nn, (long long)s.nn * K, 1};           // w[b][k][j]: rows j are contiguous
        y_is = s.nn; y_js = 1; y_bs = (long long)s.m * s.nn; bias_on = 2;
    }
    const int u_tensor = w->op == TT_OP_CONV2D ? 1 : 0;       // conv: U is the filter tensor; dense/bmm: U is x
    plan->a_tensor = swap ? 1 - u_tensor : u_tensor;
    plan->b_tensor = 1 - plan->a_tensor;
    const Opnd& A = swap ? V : U;
    const Opnd& Bo = swap ? U : V;
    g.a_mode = A.mode; g.a_rs = A.rs; g.a_ks = A.ks; g.a_bs = A.bs; g.a_tma_batched = A.batched;
    g.b_mode = Bo.mode; g.b_rs = Bo.rs; g.b_ks = Bo.ks; g.b_bs = Bo.bs; g.b_tma_batched = Bo.batched;
    g.y_ms = swap ? y_js : y_is; g.y_ns = swap ? y_is : y_js; g.y_bs = y_bs;
    g.bias_mode = s.has_bias ? (swap ? 3 - bias_on : bias_on) : 0;
    g.act = s.act;
    g.C = s.c; g.H = s.h; g.W = s.w; g.R = s.r; g.S = s.s; g.Q = Q;
    g.sh = s.stride_h; g.sw = s.stride_w; g.ph = s.pad_h; g.pw = s.pad_w;
    g.tx_bytes = (A.mode == OPM_TMA ? a_stage : 0) + (Bo.mode == OPM_TMA ? b_stage : 0);
    g.vec_store = (g.y_ns == 1 && g.y_ms % 4 == 0 && g.y_bs % 4 == 0) ? 1 : 0;
    return TT_OK;
}

static tt_status legalise_dw(const tt_workload* w, const tt_schedule_record* rec, int mode, Plan* plan) {
    const tt_shapes& s = w->sh;
    const bool strict = mode == TT_MODE_STRICT;
    tt_schedule_record L = *rec;
    int changed = 0;
    if (rec->tile_m <= 0 || rec->block_x <= 0 || rec->block_y <= 0 || rec->items_per_thread <= 0 ||
        rec->vec_width <= 0 || rec->threads <= 0)
        return TT_ERR_INVALID_SCHEDULE;
    if (strict && (rec->tile_m > s.c || rec->block_y > w->P || rec->block_x > round_up(w->Q, 4)))
        return TT_ERR_INVALID_SCHEDULE;
    L.tile_m = std::min(rec->tile_m, s.c);
    if (L.tile_m != rec->tile_m) changed |= TT_CHG_TILE_M;
    L.block_y = std::min(rec->block_y, w->P);
    int vec = rec->vec_width >= 4 ? 4 : (rec->vec_width >= 2 ? 2 : 1);
    while (vec > 1 && (w->Q % vec) != 0) vec >>= 1;        // rows of y must stay vector-aligned
    int items = std::min(8, pow2_floor(rec->items_per_thread));
    items = std::max(items, vec);
    // unroll >= 1 asks for the register-window kernel (that many output rows per thread: 1, 2 or 4), which exists
    // for square 3x3 / 5x5 filters with "same" padding and stride 1 or 2 and works on strips of 4 columns;
    // unroll == 0, or any other filter, takes the shared-memory staged kernel
    const bool window_ok = s.r == s.s && (s.r == 3 || s.r == 5) && s.stride_h == s.stride_w &&
                           (s.stride_h == 1 || s.stride_h == 2) && s.pad_h == s.r / 2 && s.pad_w == s.r / 2;
    int window_rows = 0;
    if (rec->unroll < 0) return TT_ERR_INVALID_SCHEDULE;
    if (rec->unroll >= 1 && window_ok) {
        window_rows = rec->unroll >= 4 ? 4 : (rec->unroll >= 2 ? 2 : 1);
        items = rec->items_per_thread >= 8 ? 8 : 4;      // strips of 4 or 8 columns; 8-wide strips are at most 2 rows tall
        if (items == 8 && window_rows > 2) window_rows = 2;
    }
    L.unroll = window_rows;
    // a record that names the register-window form (or a strip height it does not have) on a filter without one runs
    // another kernel form than it was written for: a reformulation, invalid when nothing may be reformulated
    if (window_rows != rec->unroll) changed |= TT_CHG_FORM;
    int bx = std::min(rec->block_x, round_up(w->Q, items));
    bx = round_up(bx, items);
    if (bx != rec->block_x || L.block_y != rec->block_y) changed |= TT_CHG_BLOCK;
    L.block_x = bx;
    if (items != rec->items_per_thread) changed |= TT_CHG_ITEMS;
    L.items_per_thread = items;
    if (vec != rec->vec_width) changed |= TT_CHG_VEC;
    L.vec_width = vec;
    int th = std::min(window_rows ? 256 : 1024, std::max(32, round_up(rec->threads, 32)));
    if (th != rec->threads) changed |= TT_CHG_BLOCK;
    L.threads = th;
    if (strict && changed) return TT_ERR_INVALID_SCHEDULE;

    DwArgs& d = plan->dw;
    d = DwArgs{};
    d.N = s.n; d.C = s.c; d.H = s.h; d.W = s.w; d.R = s.r; d.S = s.s; d.P = w->P; d.Q = w->Q;
    d.sh = s.stride_h; d.sw = s.stride_w; d.ph = s.pad_h; d.pw = s.pad_w; d.act = s.act;
    d.tile_c = L.tile_m; d.tile_h = L.block_y; d.tile_w = L.block_x;
    d.in_h = (d.tile_h - 1) * d.sh + d.R;
    d.in_w = (d.tile_w - 1) * d.sw + d.S;
    d.items = items; d.vec = vec;
    d.tiles_c = (s.c + d.tile_c - 1) / d.tile_c;
    d.tiles_h = (w->P + d.tile_h - 1) / d.tile_h;
    d.tiles_w = (w->Q + d.tile_w - 1) / d.tile_w;
    d.window_rows = window_rows;
    d.vec_in = (s.w % 4) == 0;
    long long smem = window_rows ? 0 : (long long)d.tile_c * ((long long)d.in_h * d.in_w + d.R * d.S + 1) * 4;
    tt_apply_info& I = plan->info;
    I = tt_apply_info{};
    I.legal = L; I.changed = changed;
    long long gx = (long long)d.tiles_w * d.tiles_h * d.tiles_c;
    // raster = 1 (with a window-kernel filter and 16-byte image rows): the tiles' input boxes are staged by TMA in
    // `stages` buffers, next to the filters and biases of their planes, and CTAs walk the tiles persistently
    L.raster = 0;
    if (rec->raster < 0 || rec->raster > 1) return TT_ERR_INVALID_SCHEDULE;
    if (rec->raster == 1 && window_rows > 0 && (s.w % 4) == 0) {
        const int st = d.sh, pad = d.pw;
        const int ncol = (items - 1) * st + d.R, nld = (4 - pad + ncol + 3) / 4;      // 16-byte loads per window row
        const int box_w = (d.tile_w - items) * st + 4 * nld;
        // strips are window_rows tall: the box covers the rows of the last, possibly partial, strip too
        const int in_h_box = (round_up(d.tile_h, window_rows) - 1) * d.sh + d.R;
        const long long planes = (long long)s.n * s.c;
        const long long box = (((long long)d.tile_c * in_h_box * box_w * 4) + 127) / 128 * 128;
        const long long wstage = (((long long)d.tile_c * round_up(d.R * d.S + 1, 4) * 4) + 127) / 128 * 128;
        const long long stage = box + wstage;
        int stg = std::min(4, std::max(2, rec->stages));
        while (stg > 2 && stg * stage + 128 > kDynSmemLimit) --stg;
        if (box_w <= 256 && in_h_box <= 256 && d.tile_c <= 256 && stg * stage + 128 <= kDynSmemLimit && planes <= 0x7fffffffLL) {
            d.in_h = in_h_box;
            if (stg != rec->stages) { if (strict) return TT_ERR_INVALID_SCHEDULE; I.changed |= TT_CHG_STAGES; }
            L.raster = 1; L.stages = stg;
            d.tma_stages = stg; d.box_w = box_w; d.stage_bytes = (int)box; d.wstage_bytes = (int)wstage;
            d.tiles_p = (int)((planes + d.tile_c - 1) / d.tile_c);
            const long long total = (long long)d.tiles_p * d.tiles_h * d.tiles_w;
            if (total > 0x7fffffffLL) return TT_ERR_RESOURCE;
            d.total_tiles = (int)total;
            smem = stg * stage + 128;
            const long long per_sm = std::max<long long>(1, std::min<long long>(8, (228 * 1024) / (smem + 1024)));   // the launcher lowers it to what registers allow
            gx = std::min<long long>(total, 148 * per_sm);
            I.legal = L;
            I.grid_x = (int)gx; I.grid_y = 1; I.grid_z = 1;
            I.threads = th; I.smem_bytes = (int)smem; I.launches = 1;
            return TT_OK;
        }
    }
    if (rec->raster != 0) { if (strict) return TT_ERR_INVALID_SCHEDULE; I.changed |= TT_CHG_FORM; }
    I.legal = L;
    I.grid_x = (int)std::min<long long>(gx, 0x7fffffff); I.grid_y = s.n; I.grid_z = 1;
    I.threads = th; I.smem_bytes = (int)std::min<long long>(smem, 0x7fffffff);
    I.launches = 1;
    if (smem > kDynSmemLimit || gx > 0x7fffffffLL || s.n > 65535) return TT_ERR_RESOURCE;
    return TT_OK;
}

static tt_status legalise_row(const tt_workload* w, const tt_schedule_record* rec, int mode, Plan* plan) {
    const tt_shapes& s = w->sh;
    const bool strict = mode == TT_MODE_STRICT;
    tt_schedule_record L = *rec;
    int changed = 0;
    if (rec->block_x <= 0 || rec->block_y <= 0 || rec->vec_width <= 0) return TT_ERR_INVALID_SCHEDULE;
    const long long rows = (long long)s.batch * s.m;
    int lanes = std::min(32, pow2_floor(rec->block_x));
    int vec = rec->vec_width >= 4 ? 4 : (rec->vec_width >= 2 ? 2 : 1);
    while (vec > 1 && (s.nn % vec) != 0) vec >>= 1;
    if (strict && (long long)rec->block_x * rec->vec_width > round_up(s.nn, 4)) return TT_ERR_INVALID_SCHEDULE;
    int rpc = rec->block_y;
    while ((rpc * lanes) % 32 != 0) ++rpc;                 // whole warps
    if ((long long)rpc * lanes > 1024) rpc = 1024 / lanes;
    if (lanes != rec->block_x || rpc != rec->block_y) changed |= TT_CHG_BLOCK;
    if (vec != rec->vec_width) changed |= TT_CHG_VEC;
    L.block_x = lanes; L.block_y = rpc; L.vec_width = vec;
    if (strict && changed) return TT_ERR_INVALID_SCHEDULE;
    RowArgs& r = plan->row;
    r = RowArgs{};
    r.rows = rows; r.cols = s.nn; r.scale = s.scale; r.lanes_per_row = lanes; r.rows_per_cta = rpc; r.vec = vec;
    tt_apply_info& I = plan->info;
    I = tt_apply_info{};
    I.legal = L; I.changed = changed;
    const long long gx = (rows + rpc - 1) / rpc;
    I.grid_x = (int)std::min<long long>(gx, 0x7fffffff); I.grid_y = 1; I.grid_z = 1;
    I.threads = rpc * lanes; I.launches = 1;
    if (gx > 0x7fffffffLL) return TT_ERR_RESOURCE;
    return TT_OK;
}

tt_status legalise(const tt_workload* w, const tt_schedule_record* rec, int mode, int strict_class, Plan* plan) {
    if (!w || !rec || !plan) return TT_ERR_INVALID_ARG;
    if (rec->version != TT_RECORD_VERSION) return TT_ERR_INVALID_SCHEDULE;
    // A schedule written for another loop structure tries to transform loops that do not exist (Section 4.2).
    if ((int)rec->family != w->family) return TT_ERR_CLASS_MISMATCH;
    if (strict_class && class_hash(rec->origin_op, rec->origin) != class_hash(w->op, w->sh)) return TT_ERR_CLASS_MISMATCH;
    plan->gm = w->view.gm; plan->gn = w->view.gn; plan->gk = w->view.gk; plan->gbatch = w->view.batch;
    switch (w->family) {
        case TT_FAMILY_GEMM_TC: return legalise_gemm(w, rec, mode, plan);
        case TT_FAMILY_DW_SIMT: return legalise_dw(w, rec, mode, plan);
        case TT_FAMILY_ROW_SIMT: return legalise_row(w, rec, mode, plan);
    }
    return TT_ERR_INVALID_ARG;
}

}  // namespace tt

// ---- C ABI (host-only entry points) -------------------------------------------------------------------------

extern "C" {

const char* tt_status_string(tt_status s) {
    switch (s) {
        case TT_OK: return "ok";
        case TT_ERR_INVALID_ARG: return "invalid argument";
        case TT_ERR_INVALID_SCHEDULE: return "schedule invalid for this workload";
        case TT_ERR_CLASS_MISMATCH: return "schedule belongs to another kernel class";
        case TT_ERR_RESOURCE: return "schedule exceeds hardware resources";
        case TT_ERR_NOT_APPLIED: return "no schedule applied";
        case TT_ERR_CUDA: return "CUDA error";
        case TT_ERR_TIMEOUT: return "device wait timed out";
        case TT_ERR_OOM: return "out of device memory";
        case TT_ERR_NOT_IMPLEMENTED: return "not implemented";
        case TT_SKIPPED: return "pair left out by pool sub-sampling";
    }
    return "unknown status";
}

tt_status tt_workload_create(tt_op op, const tt_shapes* sp, tt_workload** out) {
    if (!sp || !out) return TT_ERR_INVALID_ARG;
    *out = nullptr;
    const int fam = family_of(op);
    if (fam < 0) return TT_ERR_INVALID_ARG;
    tt_shapes s = *sp;
    if (s.act < TT_ACT_NONE || s.act > TT_ACT_GELU_ERF) return TT_ERR_INVALID_ARG;
    int P = 0, Q = 0;
    tt_gemm_view v{};
    if (conv_like(op)) {
        if (s.n <= 0 || s.c <= 0 || s.h <= 0 || s.w <= 0 || s.r <= 0 || s.s <= 0 || s.stride_h <= 0 || s.stride_w <= 0 ||
            s.pad_h < 0 || s.pad_w < 0)
            return TT_ERR_INVALID_ARG;
        if (op == TT_OP_CONV2D && s.k <= 0) return TT_ERR_INVALID_ARG;
        if (s.h + 2 * s.pad_h < s.r || s.w + 2 * s.pad_w < s.s) return TT_ERR_INVALID_ARG;
        if (op == TT_OP_DWCONV2D) { s.k = s.c; if (s.has_residual) return TT_ERR_INVALID_ARG; }
        P = (s.h + 2 * s.pad_h - s.r) / s.stride_h + 1;
        Q = (s.w + 2 * s.pad_w - s.s) / s.stride_w + 1;
        s.batch = s.m = s.nn = s.kk = s.trans_b = 0;
        if (op == TT_OP_CONV2D) {
            // implicit GEMM: rows = filters, columns = output pixels, reduction = (c, r, s), one GEMM per image
            v.batch = s.n; v.gm = s.k; v.gn = P * Q; v.gk = s.c * s.r * s.s;
            v.flops = 2.0 * v.batch * v.gm * (double)v.gn * v.gk;
            v.bytes = 4.0 * ((double)s.n * s.c * s.h * s.w + (double)s.k * v.gk + (s.has_bias ? s.k : 0) +
                             (double)s.n * s.k * P * Q * (s.has_residual ? 2 : 1));
        } else {
            v.batch = s.n; v.gm = s.c; v.gn = P * Q; v.gk = s.r * s.s;
            v.flops = 2.0 * s.n * s.c * (double)P * Q * s.r * s.s;
            v.bytes = 4.0 * ((double)s.n * s.c * s.h * s.w + (double)s.c * s.r * s.s + (s.has_bias ? s.c : 0) +
                             (double)s.n * s.c * P * Q);
        }
    } else {
        if (op == TT_OP_DENSE) { s.batch = 1; s.trans_b = 1; }
        if (s.batch <= 0 || s.m <= 0 || s.nn <= 0) return TT_ERR_INVALID_ARG;
        if (op != TT_OP_SOFTMAX && s.kk <= 0) return TT_ERR_INVALID_ARG;
        if (op == TT_OP_SOFTMAX) { s.kk = 0; s.has_bias = 0; s.has_residual = 0; s.act = TT_ACT_NONE; s.trans_b = 0; }
        s.n = s.c = s.h = s.w = s.k = s.r = s.s = s.stride_h = s.stride_w = s.pad_h = s.pad_w = 0;
        v.batch = s.batch; v.gm = s.m; v.gn = s.nn; v.gk = s.kk;
        if (op == TT_OP_SOFTMAX) {
            v.flops = 5.0 * s.batch * (double)s.m * s.nn;
            v.bytes = 8.0 * s.batch * (double)s.m * s.nn;
        } else {
            v.flops = 2.0 * s.batch * (double)s.m * s.nn * s.kk;
            v.bytes = 4.0 * ((double)s.batch * s.m * s.kk + (double)s.batch * s.nn * s.kk + (s.has_bias ? s.nn : 0) +
                             (double)s.batch * s.m * s.nn * (s.has_residual ? 2 : 1));
        }
    }
    if (op != TT_OP_SOFTMAX) s.scale = 0.f;
    s.has_bias = s.has_bias != 0; s.has_residual = s.has_residual != 0;
    tt_workload* w = new (std::nothrow) tt_workload();
    if (!w) return TT_ERR_OOM;
    w->op = op; w->sh = s; w->family = fam; w->P = P; w->Q = Q; w->view = v;
    *out = w;
    return TT_OK;
}

tt_status tt_workload_destroy(tt_workload* w) {
    if (!w) return TT_ERR_INVALID_ARG;
    tt::release_device(w);
    delete w;
    return TT_OK;
}

tt_status tt_workload_key(const tt_workload* w, uint64_t* key) {
    if (!w || !key) return TT_ERR_INVALID_ARG;
    int32_t op = w->op;
    uint64_t h = fnv1a(&op, sizeof op);
    // field by field: padding bytes of the struct never enter the hash
    const tt_shapes& s = w->sh;
    const int32_t f[] = {s.n, s.c, s.h, s.w, s.k, s.r, s.s, s.stride_h, s.stride_w, s.pad_h, s.pad_w,
                         s.batch, s.m, s.nn, s.kk, s.trans_b, s.has_bias, s.has_residual, s.act};
    h = fnv1a(f, sizeof f, h);
    h = fnv1a(&s.scale, sizeof s.scale, h);
    *key = h;
    return TT_OK;
}

tt_status tt_workload_class(const tt_workload* w, uint64_t* cls) {
    if (!w || !cls) return TT_ERR_INVALID_ARG;
    *cls = tt::class_hash(w->op, w->sh);
    return TT_OK;
}

tt_status tt_workload_family(const tt_workload* w, int32_t* family) {
    if (!w || !family) return TT_ERR_INVALID_ARG;
    *family = w->family;
    return TT_OK;
}

tt_status tt_workload_gemm_view(const tt_workload* w, tt_gemm_view* out) {
    if (!w || !out) return TT_ERR_INVALID_ARG;
    *out = w->view;
    return TT_OK;
}

tt_status tt_default_schedule(const tt_workload* w, tt_schedule_record* out) {
    if (!w || !out) return TT_ERR_INVALID_ARG;
    tt_schedule_record r;
    std::memset(&r, 0, sizeof r);
    r.version = TT_RECORD_VERSION;
    r.family = (uint32_t)w->family;
    r.origin_op = w->op;
    r.origin = w->sh;
    // One generic, shape-blind record per family: the counterpart of a compiler's default schedule.
    r.tile_m = 128; r.tile_n = 128; r.tile_k = 32; r.stages = 4; r.split_k = 1; r.raster = 0; r.acc_split = 1;
    r.cta_group = 1;
    r.block_x = 32; r.block_y = 4; r.items_per_thread = 1; r.vec_width = 1; r.unroll = 1; r.threads = 128;
    if (w->family == TT_FAMILY_DW_SIMT) { r.tile_m = 1; r.block_x = 32; r.block_y = 8; r.items_per_thread = 4; r.unroll = 2; }
    if (w->family == TT_FAMILY_ROW_SIMT) { r.block_x = 8; r.block_y = 16; r.vec_width = 4; }
    *out = r;
    return TT_OK;
}

tt_status tt_schedule_check(const tt_workload* w, const tt_schedule_record* rec, int32_t mode, int32_t strict_class,
                            tt_apply_info* info_out) {
    if (!w || !rec) return TT_ERR_INVALID_ARG;
    tt::Plan* p = new (std::nothrow) tt::Plan();
    if (!p) return TT_ERR_OOM;
    tt_status st = tt::legalise(w, rec, mode, strict_class, p);
    if (info_out && (st == TT_OK || st == TT_ERR_RESOURCE)) *info_out = p->info;
    delete p;
    return st;
}

// ---- refinement of a transferred record (named as future work in Section 7): a local search over the fields of a
// record that another model's tuning produced ----
namespace {
struct FieldLadder { int32_t tt_schedule_record::*field; std::vector<int> steps; };   // two steps = a toggle when both differ

const std::vector<FieldLadder>& ladders_of(uint32_t family) {
    static const std::vector<FieldLadder> gemm = {
        {&tt_schedule_record::tile_n, {16, 32, 48, 64, 96, 128, 160, 192, 224, 256}},
        {&tt_schedule_record::tile_k, {8, 16, 32, 64, 96, 128}},
        {&tt_schedule_record::stages, {1, 2, 3, 4, 5, 6, 7, 8}},
        {&tt_schedule_record::split_k, {1, 2, 3, 4, 5, 6, 7, 8, 12, 16, 24, 32}},
        {&tt_schedule_record::raster, {0, 1}},
        {&tt_schedule_record::mma_m_axis, {1, 2}},
        {&tt_schedule_record::slab_tiles, {0, 1, 2, 4, 8}},
        {&tt_schedule_record::acc_split, {1, 2, 4, 8}},
        {&tt_schedule_record::k_order, {0, 1}},
        {&tt_schedule_record::persistent, {0, 1}},
        {&tt_schedule_record::cta_group, {1, 2}},
        {&tt_schedule_record::ctas_per_sm, {1, 2}},
    };
    static const std::vector<FieldLadder> dw = {
        {&tt_schedule_record::tile_m, {1, 2, 4, 8, 16, 32}},
        {&tt_schedule_record::block_y, {1, 2, 4, 7, 8, 14, 16, 28, 56}},
        {&tt_schedule_record::block_x, {8, 16, 28, 32, 56, 64, 112}},
        {&tt_schedule_record::items_per_thread, {1, 2, 4, 8}},
        {&tt_schedule_record::vec_width, {1, 2, 4}},
        {&tt_schedule_record::threads, {32, 64, 128, 256, 512}},
        {&tt_schedule_record::unroll, {0, 1, 2, 4}},
        {&tt_schedule_record::raster, {0, 1}},
        {&tt_schedule_record::stages, {2, 3, 4}},
    };
    static const std::vector<FieldLadder> row = {
        {&tt_schedule_record::block_x, {1, 2, 4, 8, 16, 32}},
        {&tt_schedule_record::block_y, {1, 2, 4, 8, 16}},
        {&tt_schedule_record::vec_width, {1, 2, 4}},
    };
    return family == TT_FAMILY_GEMM_TC ? gemm : (family == TT_FAMILY_DW_SIMT ? dw : row);
}
}  // namespace

tt_status tt_record_neighbours(const tt_workload* w, const tt_schedule_record* rec, tt_schedule_record* out, size_t cap,
                               size_t* n_out) {
    if (!w || !rec || !n_out || (cap > 0 && !out)) return TT_ERR_INVALID_ARG;
    if (rec->version != TT_RECORD_VERSION || (int)rec->family != (int)w->family) return TT_ERR_INVALID_SCHEDULE;
    // the start in its legalised form: a neighbour that legalises back to it is no neighbour
    tt_apply_info start;
    const tt_status s0 = tt_schedule_check(w, rec, TT_MODE_LEGALISE, 0, &start);
    if (s0 != TT_OK) return s0;
    std::vector<tt_schedule_record> found;
    auto consider = [&](tt_schedule_record r) {
        tt_apply_info info;
        if (tt_schedule_check(w, &r, TT_MODE_LEGALISE, 0, &info) != TT_OK) return;
        tt_schedule_record l = info.legal;
        l.origin_op = rec->origin_op; l.origin = rec->origin;
        tt_schedule_record s = start.legal;
        s.origin_op = rec->origin_op; s.origin = rec->origin;
        if (std::memcmp(&l, &s, sizeof l) == 0) return;
        for (const auto& f : found) if (std::memcmp(&f, &l, sizeof l) == 0) return;
        found.push_back(l);
    };
    for (const FieldLadder& fl : ladders_of(w->family)) {
        const int v = start.legal.*(fl.field);
        int below = INT32_MIN, above = INT32_MAX;       // nearest rungs on either side of v (v need not be a rung)
        for (int step : fl.steps) {
            if (step < v && step > below) below = step;
            if (step > v && step < above) above = step;
        }
        if (below != INT32_MIN) { tt_schedule_record r = start.legal; r.*(fl.field) = below; consider(r); }
        if (above != INT32_MAX) { tt_schedule_record r = start.legal; r.*(fl.field) = above; consider(r); }
    }
    *n_out = found.size();
    if (found.size() > cap) return cap == 0 ? TT_OK : TT_ERR_RESOURCE;     // cap == 0: count only
    for (size_t i = 0; i < found.size(); ++i) out[i] = found[i];
    return TT_OK;
}

tt_status tt_refine_with(const tt_workload* w, const tt_schedule_record* start, tt_time_fn time_us, void* user,
                         int32_t max_rounds, float min_gain, tt_schedule_record* best, float* best_us, float* start_us,
                         int32_t* n_timed) {
    if (!w || !start || !time_us || !best || !best_us || max_rounds < 0 || !(min_gain >= 0.f)) return TT_ERR_INVALID_ARG;
    tt_apply_info info;
    const tt_status s0 = tt_schedule_check(w, start, TT_MODE_LEGALISE, 0, &info);
    if (s0 != TT_OK) return s0;
    tt_schedule_record cur = info.legal;
    cur.origin_op = start->origin_op; cur.origin = start->origin;
    float cur_us = time_us(user, &cur);
    int timed = 1;
    if (start_us) *start_us = cur_us;
    if (!(cur_us >= 0.f)) { if (n_timed) *n_timed = timed; return TT_ERR_INVALID_SCHEDULE; }
    std::vector<tt_schedule_record> seen{cur};           // never time a record twice
    for (int round = 0; round < max_rounds; ++round) {
        size_t n = 0;
        std::vector<tt_schedule_record> nb(32);
        const tt_status sn = tt_record_neighbours(w, &cur, nb.data(), nb.size(), &n);
        if (sn != TT_OK) return sn;
        int pick = -1;
        float pick_us = cur_us;
        for (size_t i = 0; i < n; ++i) {
            bool dup = false;
            for (const auto& r : seen) if (std::memcmp(&r, &nb[i], sizeof r) == 0) { dup = true; break; }
            if (dup) continue;
            seen.push_back(nb[i]);
            const float us = time_us(user, &nb[i]);
            ++timed;
            if (us >= 0.f && us < pick_us) { pick = (int)i; pick_us = us; }    // ties keep the earlier neighbour
        }
        // move only for a gain of more than min_gain (a fraction of the current time): noise does not walk the record
        if (pick < 0 || !(pick_us < cur_us * (1.f - min_gain))) break;
        cur = nb[(size_t)pick]; cur_us = pick_us;
    }
    *best = cur; *best_us = cur_us;
    if (n_timed) *n_timed = timed;
    return TT_OK;
}

// ---- pool files ---------------------------------------------------------------------------------------------------
namespace {
struct RecField { const char* name; int32_t tt_schedule_record::*field; };
const RecField kRecFields[] = {
    {"tile_m", &tt_schedule_record::tile_m}, {"tile_n", &tt_schedule_record::tile_n}, {"tile_k", &tt_schedule_record::tile_k},
    {"stages", &tt_schedule_record::stages}, {"split_k", &tt_schedule_record::split_k}, {"raster", &tt_schedule_record::raster},
    {"block_x", &tt_schedule_record::block_x}, {"block_y", &tt_schedule_record::block_y},
    {"items_per_thread", &tt_schedule_record::items_per_thread}, {"vec_width", &tt_schedule_record::vec_width},
    {"unroll", &tt_schedule_record::unroll}, {"threads", &tt_schedule_record::threads},
    {"mma_m_axis", &tt_schedule_record::mma_m_axis}, {"slab_tiles", &tt_schedule_record::slab_tiles},
    {"acc_split", &tt_schedule_record::acc_split}, {"k_order", &tt_schedule_record::k_order},
    {"persistent", &tt_schedule_record::persistent}, {"cta_group", &tt_schedule_record::cta_group},
    {"ctas_per_sm", &tt_schedule_record::ctas_per_sm}, {"warp_layout", &tt_schedule_record::warp_layout},
    {"precision", &tt_schedule_record::precision},
};
int32_t* shape_ints(tt_shapes& s, int i) {
    int32_t* f[] = {&s.n, &s.c, &s.h, &s.w, &s.k, &s.r, &s.s, &s.stride_h, &s.stride_w, &s.pad_h, &s.pad_w,
                    &s.batch, &s.m, &s.nn, &s.kk, &s.trans_b, &s.has_bias, &s.has_residual, &s.act};
    return f[i];
}
constexpr int kShapeInts = 19;
}  // namespace

tt_status tt_pool_save(const char* path, const tt_schedule_record* records, const float* us, size_t n) {
    if (!path || (n && !records)) return TT_ERR_INVALID_ARG;
    FILE* f = std::fopen(path, "w");
    if (!f) return TT_ERR_INVALID_ARG;
    std::fprintf(f, "# schedule pool: one record per line, field=value\n");
    for (size_t i = 0; i < n; ++i) {
        tt_schedule_record r = records[i];
        std::fprintf(f, "version=%u family=%u origin_op=%d origin=", r.version, r.family, r.origin_op);
        for (int j = 0; j < kShapeInts; ++j) std::fprintf(f, "%d,", *shape_ints(r.origin, j));
        std::fprintf(f, "%.9g", (double)r.origin.scale);
        for (const RecField& rf : kRecFields) std::fprintf(f, " %s=%d", rf.name, r.*(rf.field));
        std::fprintf(f, " us=%.6g\n", us ? (double)us[i] : -1.0);
    }
    const bool ok = std::fclose(f) == 0;
    return ok ? TT_OK : TT_ERR_INVALID_ARG;
}

tt_status tt_pool_load(const char* path, tt_schedule_record* out, float* us, size_t cap, size_t* n_out) {
    if (!path || !n_out || (cap && !out)) return TT_ERR_INVALID_ARG;
    FILE* f = std::fopen(path, "r");
    if (!f) return TT_ERR_INVALID_ARG;
    size_t n = 0;
    tt_status rc = TT_OK;
    char line[2048];
    while (rc == TT_OK && std::fgets(line, sizeof line, f)) {
        char* p = line;
        while (*p == ' ' || *p == '\t') ++p;
        if (*p == '#' || *p == '\n' || *p == '\r' || *p == 0) continue;
        tt_schedule_record r;
        std::memset(&r, 0, sizeof r);
        float t = -1.f;
        bool have_version = false;
        for (char* tok = std::strtok(p, " \t\r\n"); tok && rc == TT_OK; tok = std::strtok(nullptr, " \t\r\n")) {
            char* eq = std::strchr(tok, '=');
            if (!eq) { rc = TT_ERR_INVALID_ARG; break; }
            *eq = 0;
            const std::string key(tok);
            const char* val = eq + 1;
            char* end = nullptr;
            if (key == "version") { r.version = (uint32_t)std::strtoul(val, &end, 10); have_version = true; }
            else if (key == "family") r.family = (uint32_t)std::strtoul(val, &end, 10);
            else if (key == "origin_op") r.origin_op = (int32_t)std::strtol(val, &end, 10);
            else if (key == "us") t = std::strtof(val, &end);
            else if (key == "origin") {
                const char* q = val;
                for (int j = 0; j < kShapeInts && rc == TT_OK; ++j) {
                    *shape_ints(r.origin, j) = (int32_t)std::strtol(q, &end, 10);
                    if (end == q || *end != ',') rc = TT_ERR_INVALID_ARG;
                    q = end + 1;
                }
                if (rc == TT_OK) { r.origin.scale = std::strtof(q, &end); if (end == q) rc = TT_ERR_INVALID_ARG; }
            } else {
                bool found = false;
                for (const RecField& rf : kRecFields)
                    if (key == rf.name) { r.*(rf.field) = (int32_t)std::strtol(val, &end, 10); found = true; break; }
                if (!found) rc = TT_ERR_INVALID_ARG;
            }
            if (rc == TT_OK && (end == val || (end && *end != 0))) rc = TT_ERR_INVALID_ARG;
        }
        if (rc != TT_OK) break;
        if (!have_version || r.version != TT_RECORD_VERSION) { rc = TT_ERR_INVALID_ARG; break; }
        if (n < cap) { out[n] = r; if (us) us[n] = t; }
        ++n;
    }
    std::fclose(f);
    *n_out = n;
    if (rc != TT_OK) return rc;
    return (cap && n > cap) ? TT_ERR_RESOURCE : TT_OK;
}

tt_status tt_pool_subsample(size_t n_pool, size_t count, uint64_t seed, int32_t* idx_out) {
    if (count > n_pool || (count && !idx_out) || n_pool > 0x7fffffffu) return TT_ERR_INVALID_ARG;
    std::vector<int32_t> perm(n_pool);
    for (size_t i = 0; i < n_pool; ++i) perm[i] = (int32_t)i;
    uint64_t state = seed;
    for (size_t i = 0; i < count; ++i) {
        // splitmix64: advance the state by the golden-ratio increment, then mix
        state += 0x9E3779B97F4A7C15ull;
        uint64_t z = state;
        z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
        z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
        z ^= z >> 31;
        const size_t j = i + (size_t)(z % (uint64_t)(n_pool - i));
        std::swap(perm[i], perm[j]);
        idx_out[i] = perm[i];
    }
    return TT_OK;
}

tt_status tt_split_check(int64_t extent, const int64_t* factors, size_t n, int32_t reformulate, int32_t* valid) {
    if (!factors || !valid || n == 0 || extent <= 0) return TT_ERR_INVALID_ARG;
    if (reformulate) {
        // Split(N, N/f, f): the outer range adapts to the extent, so only divisibility remains.
        *valid = factors[0] > 0 && extent % factors[0] == 0;
        return TT_OK;
    }
    // Split(N, f0, f1, ...): fixed ranges must traverse the loop exactly.
    __int128 prod = 1;
    for (size_t i = 0; i < n; ++i) {
        if (factors[i] <= 0) { *valid = 0; return TT_OK; }
        prod *= factors[i];
        if (prod > (__int128)extent) { *valid = 0; return TT_OK; }
    }
    *valid = prod == (__int128)extent;
    return TT_OK;
}

tt_status tt_select(const float* times_us, size_t n_wl, size_t n_cols, int32_t* chosen) {
    if (!times_us || !chosen || n_cols == 0) return TT_ERR_INVALID_ARG;
    for (size_t i = 0; i < n_wl; ++i) {
        int best = -1;
        float bt = 0.f;
        for (size_t j = 0; j < n_cols; ++j) {
            const float t = times_us[i * n_cols + j];
            if (!(t >= 0.f) || !std::isfinite(t)) continue;     // negative = invalid pair, NaN never wins
            if (best < 0 || t < bt) { best = (int)j; bt = t; }
        }
        chosen[i] = best;
    }
    return TT_OK;
}

tt_status tt_rank_pools(const double* class_share, size_t n_classes, const int32_t* class_kernels, size_t n_models,
                        double* scores, int32_t* order) {
    if (!class_share || !class_kernels || !order || n_classes == 0) return TT_ERR_INVALID_ARG;
    std::vector<double> sc(n_models, 0.0);
    for (size_t t = 0; t < n_models; ++t) {
        double s = 0.0;
        for (size_t c = 0; c < n_classes; ++c) {
            const int32_t n = class_kernels[t * n_classes + c];
            if (n < 0 || !(class_share[c] >= 0.0)) return TT_ERR_INVALID_ARG;
            s += class_share[c] * class_share[c] * std::sqrt((double)n);
        }
        sc[t] = s;
    }
    for (size_t t = 0; t < n_models; ++t) order[t] = (int32_t)t;
    std::stable_sort(order, order + n_models, [&](int32_t a, int32_t b) { return sc[a] > sc[b]; });
    if (scores) for (size_t t = 0; t < n_models; ++t) scores[t] = sc[t];
    return TT_OK;
}

tt_status tt_model_latency(const float* times_us, size_t n_wl, size_t n_cols, const int32_t* chosen,
                           const int32_t* use_count, double* latency_us) {
    if (!times_us || !chosen || !use_count || !latency_us) return TT_ERR_INVALID_ARG;
    double sum = 0.0;
    for (size_t i = 0; i < n_wl; ++i) {
        if (chosen[i] < 0 || (size_t)chosen[i] >= n_cols) continue;
        sum += (double)use_count[i] * (double)times_us[i * n_cols + chosen[i]];
    }
    *latency_us = sum;
    return TT_OK;
}

}  // extern "C"
