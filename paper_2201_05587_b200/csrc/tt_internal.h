// Internal declarations shared by the host logic and the CUDA launchers of libtt.
#pragma once
#include <cstdint>
#include <cstddef>
#include <vector>
#include "tt.h"

namespace tt {

constexpr int kHwTileM = 128;           // tcgen05 accumulator rows per CTA (cta_group::1, M = 128)
constexpr int kMaxStages = 8;
constexpr int kSmemLimit = 232448;      // 227 KB opt-in shared memory per CTA on sm_100
constexpr int kDynSmemLimit = kSmemLimit - 6144;  // what is left for dynamic shared memory beside barriers
constexpr int kGatherWarps = 8;
constexpr int kGatherThreads = kGatherWarps * 32;
constexpr int kGemmThreads = 64 + kGatherThreads;   // warp 0 TMA, warp 1 MMA + TMEM, warps 2-9 gather + epilogue

// How one operand of the contraction reaches shared memory.
enum OperandMode : int {
    OPM_TMA = 0,          // K-major 2-D/3-D tensor map, hardware swizzle
    OPM_GATHER_ROWS = 1,  // strided view, lanes walk rows (row stride 1): 16-byte swizzled stores
    OPM_GATHER_K = 2,     // strided view, lanes walk k (k stride 1): 4-byte swizzled stores
    OPM_IM2COL = 3,       // rows are output pixels, k = (c, r, s): expanded from a slab of NCHW input rows
    OPM_IM2COL_T = 4,     // rows are padded-linear output pixels, k = (32-channel block, tap, channel): every tap's tile
                          // is a shifted view of a pixel-major slab in shared memory (nothing is staged per tile)
    OPM_TMA_MN = 5        // persistent kernel: the row index is the contiguous one in memory; [tile_k][rows] boxes arrive by
                          // TMA in a staging ring and are transposed into the K-major stage by four warps
};

// Device-side arguments of the GEMM_TC kernel (plain data, passed by value).
struct GemmArgs {
    int M, N, K, batch;
    int tile_n, tile_k, stages;
    int k_tiles, k_tiles_per_split, split_k;
    int tiles_m, tiles_n, raster;
    int atom_k, n_atoms, swz_mask, row_bytes;
    int a_mode, b_mode;
    const float* a; long long a_rs, a_ks, a_bs; int a_tma_batched;
    const float* b; long long b_rs, b_ks, b_bs; int b_tma_batched;
    int C, H, W, R, S, Q, sh, sw, ph, pw;       // im2col geometry of operand B
    float* y; long long y_ms, y_ns, y_bs;
    const float* bias; int bias_mode;           // 0 none, 1 per row (m), 2 per column (n)
    int act;
    const float* residual;
    float* partial;                             // split-K partial sums [split][batch][M][N]
    unsigned* counters;                         // split-K arrival counters [batch][tiles], zero between launches
    unsigned* status;
    unsigned idesc, tmem_cols;
    unsigned red_off;                           // cluster reduction area: byte offset from the aligned tile base
    int cluster;                                // > 0: split-K over a thread-block cluster of this many CTAs (= split_k)
    int n_acc;                                  // accumulators of tile_n columns each, reduction steps dealt round-robin
    unsigned a_stage_bytes, b_stage_bytes, tx_bytes;
    unsigned ktab_off;                          // im2col k-table: byte offset from the aligned tile base
    int vec_store;                              // bit 0: y rows allow aligned float4 stores; bit 1: so does bias
    // im2col slab: the input rows a CTA's pixels need, staged once in shared memory per chunk of reduction tiles
    unsigned slab_off;                          // byte offset of the first slab buffer from the aligned tile base
    unsigned slab_buf_bytes;                    // bytes per slab buffer (multiple of 16)
    int slab_nbuf;                              // 1: the CTA's whole K range in one chunk; 2: double-buffered chunks
    int slab_tiles;                             // reduction tiles per chunk
    int slab_wp, slab_gap, slab_chpitch;        // row pitch (W + gap), zero gap, channel pitch, in elements
    int slab_in_rows;                           // slab rows per channel (the most a tile can need)
    int slab_rstep;                             // slab rows per output row: min(stride_h, r)
    int slab_vec16;                             // rows copied 16 bytes at a time (W % 4 == 0 and x aligned)
    unsigned magic_wpieces, magic_in_rows, magic_rstep;
    // slab by TMA (rows 16-byte aligned, stride <= filter height): a chunk is one box [box_ch channels][in_rows][W + gap]
    // starting `gap` columns left of the image, so the hardware's zero fill writes the gaps and the rows outside
    int slab_tma;                               // 1: chunks arrive by TMA; 0: by cp.async from the gather warps
    int slab_box_ch;                            // channels per box
    unsigned slab_box_bytes;
    unsigned pm_off, pm_buf_bytes; int pm_nbuf; // tap-major convolutions: the pixel-major slab buffers (one or two)
    int tap_major;                              // 1: OPM_IM2COL_T on operand B
    int Pout;                                   // output rows (padded-linear pixel -> (p, q'))
    const int* ktab_dev;                        // per reduction index: byte offset of (c, r, s) inside the slab (absolute channel)
    unsigned long long wait_ns;                 // limit of every bounded wait inside the kernel
    unsigned extra_tx;                          // test facility: bytes added to what the first stage's barrier expects
    int w_operand;                              // 1 / 2: operand A / B is constant (weights the caller promised nobody is
                                                // writing): its first stages are requested before the wait on the kernel in front
    int two_per_sm;                             // the register-capped build, so that two CTAs share an SM
    int x3;                                     // error-compensated products: a stage holds [A][B][A lo][B lo]
    // persistent kernel (record field persistent = 1)
    int persistent, cta_group;
    int total_tiles;                            // tiles_m * tiles_n * batch; tiles_m counts 128 * cta_group rows
    int a_mn, b_mn;                             // operand arrives as [tile_k][rows] boxes and is transposed in shared memory
    int b_rows_cta;                             // rows of operand B one CTA loads: tile_n / cta_group
    unsigned a_stg_off, b_stg_off;              // staging rings: byte offsets from the aligned tile base
    unsigned stg_a_bytes, stg_b_bytes;          // ... and bytes per box
    int stg_depth;                              // boxes per staging ring (what is in flight from DRAM)
    unsigned epi_off;                           // read-out staging area (one 32 x 36-float block per read-out warp)
};

struct DwArgs {
    const float* x; const float* w; const float* bias; float* y;
    int N, C, H, W, R, S, P, Q, sh, sw, ph, pw, act;
    int tile_c, tile_h, tile_w, in_h, in_w, items, vec;
    int tiles_c, tiles_h, tiles_w;
    int window_rows;   // > 0: register-window kernel with this many output rows per thread; 0: staged kernel
    int vec_in;        // input rows start on 16-byte boundaries (W % 4 == 0 and x aligned)
    // TMA-staged persistent kernel (record raster = 1): tiles of tile_c planes x tile_h x tile_w outputs, their input
    // boxes [tile_c][in_h][box_w] land in `stages` shared-memory buffers by TMA (zero fill = padding)
    int tma_stages;    // > 0 selects it
    int box_w, stage_bytes, tiles_p, total_tiles;   // box width in floats (multiple of 4), bytes per buffer (multiple of 128)
    int wstage_bytes;  // bytes per filter-and-bias buffer (one per box buffer, multiple of 128)
    unsigned* status;  // the workload's status word (bounded waits)
    unsigned long long wait_ns;   // limit of every bounded wait inside the kernel
};

struct RowArgs {
    const float* x; float* y; long long rows; int cols; float scale;
    int lanes_per_row, rows_per_cta, vec;
};

// Host-side plan of an applied record.
struct Plan {
    bool applied = false;
    tt_apply_info info{};
    // GEMM lowering
    int gm = 0, gn = 0, gk = 0, gbatch = 1;
    bool swap_ab = false;
    int a_tensor = 0, b_tensor = 1;   // which caller tensor feeds operand A / B: 0 = x, 1 = w
    GemmArgs g{};
    long long partial_bytes = 0;      // counters start here inside the workspace
    bool repack = false;              // tap-major convolution: filters are re-packed into the workspace before each run
    int repack_cb = 0;                // 32-channel blocks
    DwArgs dw{};
    RowArgs row{};
};

struct TmapPair {
    const void* a_ptr; const void* b_ptr;
    alignas(64) unsigned char a[128];
    alignas(64) unsigned char b[128];
    alignas(64) unsigned char x[128];   // conv2d: the image as a (W, H, C, N) tensor, for the slab
};

}  // namespace tt

struct tt_workload {
    tt_op op;
    tt_shapes sh;
    int family;
    int P, Q;                    // conv output size
    tt_gemm_view view;
    tt::Plan plan;
    void* workspace = nullptr;   // device: split-K partials
    int* ktab_dev = nullptr;     // device: conv2d reduction-index table of the applied record
    size_t ktab_bytes = 0;
    size_t workspace_bytes = 0;
    unsigned* status_word = nullptr;  // device
    unsigned long long wait_ns = 1000000000ull;   // one second per wait inside a kernel, then the kernel gives up
    unsigned extra_tx = 0;            // test facility (tt_workload_test_stall)
    bool constant_weights = false;    // the caller's promise of tt_workload_set_constant_weights
    const void* repacked_for = nullptr;   // tap-major convolution: the weight pointer whose re-packed copy the workspace holds
    // device staging buffers of tt_run_host
    void* hbuf[5] = {nullptr, nullptr, nullptr, nullptr, nullptr};
    size_t hbytes[5] = {0, 0, 0, 0, 0};
    std::vector<tt::TmapPair> tmaps;  // tensor maps encoded so far for the applied record, by operand pointers
};

namespace tt {
// host logic (tt_host.cpp)
tt_status legalise(const tt_workload* w, const tt_schedule_record* rec, int mode, int strict_class, Plan* plan);
uint64_t class_hash(int op, const tt_shapes& s);
size_t tensor_elems(const tt_workload* w, int which);   // 0 x, 1 w, 2 bias, 3 residual, 4 y
// device side (launch.cu)
tt_status bind_device(tt_workload* w);                          // workspace + status word
tt_status launch(tt_workload* w, const tt_tensors* t, void* stream);
void release_device(tt_workload* w);
}  // namespace tt
