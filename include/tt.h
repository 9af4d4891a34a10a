/*
 * tt.h — C ABI of the transfer-tuning hot path on B200 (sm_100a).
 *
 * Transfer-tuning (Gibson & Cano, PACT '22) reuses schedules tuned for the kernels
 * of one model on the kernels of another: every kernel of the target model is run
 * standalone under every compatible schedule of a pool, timed, and the fastest
 * schedule that produced valid code is kept (Section 4.3).  A kernel is a fused
 * group of operators identified by its class (operator sequence) and its data
 * sizes (Section 4.2); a schedule is the list of transformations applied to the
 * kernel's loop nest (Section 2, Algorithm 1).
 *
 * Here a schedule is a fixed-size record of the choices those transformations make
 * on a GPU (tile sizes, pipeline depth, split-K, tile order, vector width ...), and
 * applying it to a kernel of another shape legalises it or declares it invalid.
 *
 * General conventions
 *   - Every function returns a tt_status; nothing throws or aborts across the ABI.
 *   - Handles (tt_workload*) are owned by the library and released by *_destroy.
 *   - Tensor pointers in tt_tensors are DEVICE pointers owned by the caller, fp32,
 *     dense row-major in the layouts stated at tt_op; they are borrowed for the
 *     call and never retained.  tt_run_host takes HOST pointers instead.
 *   - The only device memory the library owns is a per-workload workspace (split-K
 *     partial sums and a status word), allocated by tt_schedule_apply and released
 *     by tt_workload_destroy or the next apply.
 *   - Launches are asynchronous on the given CUDA stream (a cudaStream_t passed as
 *     void*; NULL is the default stream).  tt_time, tt_transfer_tune, tt_grid_tune
 *     and tt_run_host synchronise that stream before returning.
 *   - One handle must not be used from two threads at once.
 *   - A CUDA device must be present for everything except the pure host calls
 *     (tt_workload_create/key/class/gemm_view, tt_default_schedule, tt_schedule_check,
 *     tt_select, tt_model_latency, tt_rank_pools, tt_split_check, tt_status_string); there is no
 *     CPU fallback: without a device the others return TT_ERR_CUDA.
 */
#ifndef TT_H_
#define TT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    TT_OK = 0,
    TT_ERR_INVALID_ARG = 1,       /* null pointer, non-positive extent, unknown enum */
    TT_ERR_INVALID_SCHEDULE = 2,  /* the record cannot be applied to this shape ("invalid code", Section 4.2) */
    TT_ERR_CLASS_MISMATCH = 3,    /* record of another kernel family/class (always invalid, Section 4.2) */
    TT_ERR_RESOURCE = 4,          /* legal record, but exceeds shared memory / tensor memory / thread limits */
    TT_ERR_NOT_APPLIED = 5,       /* tt_run / tt_time before a successful tt_schedule_apply */
    TT_ERR_CUDA = 6,              /* a CUDA runtime or driver call failed (or no device) */
    TT_ERR_TIMEOUT = 7,           /* a bounded wait inside a kernel expired; the context stays usable */
    TT_ERR_OOM = 8,               /* workspace allocation failed */
    TT_ERR_NOT_IMPLEMENTED = 9,
    TT_SKIPPED = 10               /* evaluator only: the pair was left out by pool sub-sampling (neither valid nor invalid) */
} tt_status;

/* Operators (each is one fused kernel; bias and activation are applied as soon as an
 * output's partial sums are complete, Section 4.2).
 *   TT_OP_CONV2D        Algorithm 2: y = act(conv2d(pad(x), w) + bias [+ residual]).
 *                       x [n,c,h,w]  w [k,c,r,s]  bias [k]  residual,y [n,k,p,q]; cross-correlation,
 *                       zero padding pad_h/pad_w per side, p = (h + 2 pad_h - r)/stride_h + 1.
 *   TT_OP_DWCONV2D      the same with one r x s filter per channel: w [c,1,r,s], bias [c], y [n,c,p,q].
 *   TT_OP_DENSE         y[m,nn] = act(bias[nn] + sum_kk x[m,kk] w[nn,kk]); x [m,kk], w [nn,kk] (Algorithm 1 with
 *                       the second operand stored transposed), bias [nn].
 *   TT_OP_BATCH_MATMUL  y[b,m,nn] = sum_kk x[b,m,kk] * w[b,nn,kk] (trans_b = 1) or * w[b,kk,nn] (trans_b = 0);
 *                       Algorithm 1 per batch entry.
 *   TT_OP_SOFTMAX       y[row,:] = softmax(scale * x[row,:]) over nn columns, rows = batch*m.
 */
typedef enum { TT_OP_CONV2D = 0, TT_OP_DWCONV2D = 1, TT_OP_DENSE = 2, TT_OP_BATCH_MATMUL = 3, TT_OP_SOFTMAX = 4 } tt_op;
typedef enum { TT_ACT_NONE = 0, TT_ACT_RELU = 1, TT_ACT_RELU6 = 2, TT_ACT_GELU_ERF = 3 } tt_act;

/* Kernel families: the loop structure a record was written for.  A record only applies inside its family. */
typedef enum { TT_FAMILY_GEMM_TC = 0,   /* tcgen05 TF32 contraction: conv2d (implicit GEMM), dense, batch_matmul */
               TT_FAMILY_DW_SIMT = 1,   /* fp32 SIMT depthwise convolution */
               TT_FAMILY_ROW_SIMT = 2   /* fp32 SIMT row-wise kernels (softmax) */
} tt_family;

typedef struct tt_shapes {
    int32_t n, c, h, w, k, r, s, stride_h, stride_w, pad_h, pad_w; /* conv2d, dwconv2d (k ignored for depthwise) */
    int32_t batch, m, nn, kk, trans_b;                             /* dense (batch=1), batch_matmul, softmax */
    int32_t has_bias, has_residual;
    int32_t act;                                                   /* tt_act */
    float scale;                                                   /* softmax only */
} tt_shapes;

#define TT_RECORD_VERSION 3u

/* A schedule record.  Correspondence with the primitives listed under Algorithm 1:
 *   Split     -> tile_m, tile_n, tile_k (CTA tile of the output and of the reduction), split_k
 *   Reorder   -> raster (order in which output tiles are handed to CTAs), mma_m_axis (which output loop is the
 *                accumulator's row loop)
 *   Fuse+Parallel -> the (tile_m x tile_n x split_k x batch) grid
 *   cache buffer / ComputeAt -> the accumulator lives in tensor memory and the bias/activation run on read-out;
 *                               `stages` shared-memory buffers decouple loading from the multiply
 *   Vectorize -> vec_width;   Unroll -> unroll / items_per_thread
 * GEMM_TC uses tile_m, tile_n, tile_k, stages, split_k, raster, mma_m_axis, slab_tiles, acc_split, k_order, persistent,
 *         cta_group, ctas_per_sm, warp_layout, precision.
 * DW_SIMT uses tile_m (channels per CTA), block_y x block_x (output rows x columns per CTA tile),
 *         items_per_thread (consecutive outputs along the width per thread), vec_width, threads, and unroll:
 *         0 = shared-memory staged kernel; 1, 2, 4 = register-window kernel with that many output rows per thread
 *         (3x3 and 5x5 filters with "same" padding, stride 1 or 2; strips of 4 or 8 columns).  raster = 1 with
 *         unroll >= 1 and image rows of 16-byte multiples: the same strips, but CTAs walk the tiles persistently and
 *         a tile's input box and its planes' filters are staged in `stages` (2..4) shared-memory buffers by TMA.
 * ROW_SIMT uses block_x (threads cooperating on one row: 1..32, power of two), block_y (rows per CTA), vec_width.
 * origin_* say which kernel the record was tuned on (its "native" kernel, Section 3). */
typedef struct tt_schedule_record {
    uint32_t version;      /* TT_RECORD_VERSION */
    uint32_t family;       /* tt_family */
    int32_t origin_op;     /* tt_op */
    tt_shapes origin;
    int32_t tile_m, tile_n, tile_k;
    int32_t stages, split_k, raster;
    int32_t block_x, block_y, items_per_thread, vec_width, unroll, threads;
    int32_t mma_m_axis;    /* GEMM_TC: which output axis rides the 128 accumulator rows: 0 library's choice by shape,
                              1 output rows (conv filters, dense/bmm rows m), 2 output columns (conv pixels, nn) */
    int32_t slab_tiles;    /* GEMM_TC, conv2d: reduction tiles served by one staging of the input rows in shared
                              memory (the cache buffer of the im2col operand); 0 = as many as fit.  Persistent form with a
                              row-contiguous operand: boxes in that operand's staging ring, i.e. how much is in flight
                              from memory; 0 = as many as fit, at most 8 */
    int32_t acc_split;     /* GEMM_TC: independent accumulators in tensor memory (1, 2, 4 or 8; 0 = 1) to which the
                              8-wide reduction steps are dealt round-robin; they are added in fixed order on read-out.
                              Consecutive multiply-accumulates into one accumulator wait for each other; into several,
                              they overlap (the reduction-factoring of a schedule). */
    int32_t k_order;       /* GEMM_TC, conv2d: order in which the reduction (c, r, s) is walked.  0 = as the filters are
                              stored (channel-major; the im2col operand is expanded stage by stage).  1 = blocks of 32
                              channels, tap by tap inside a block: the filters are re-packed into that order by a small
                              kernel (once per weight pointer: again only when tt_run sees other weights), the input rows are transposed once per block into a pixel-major
                              slab, and every tap's operand tile is a shifted view of that slab -- no expansion.
                              Stride-1 convolutions with 16-byte image rows, filters on the 128 rows, split_k = 1;
                              tile_k = 32 * (taps per pipeline stage), the tap count a divisor of r*s, at most 128. */
    int32_t persistent;    /* GEMM_TC: 1 = the grid is one CTA (or CTA pair) per SM and every CTA walks output tiles; the
                              operand pipeline runs on across tiles and two accumulators in tensor memory alternate, so a
                              tile is read out (bias, activation, stores) while the next one is accumulated.  Needs
                              split_k = 1 and operands that TMA can fetch: dense and batch_matmul with 16-byte rows, 1x1
                              stride-1 unpadded convolutions with h*w and c multiples of 4 (an operand whose row index is
                              the contiguous one -- the image, the second operand of an NN batch_matmul -- is staged as
                              [tile_k][rows] boxes and transposed in shared memory).  Elsewhere legalised to 0. */
    int32_t cta_group;     /* GEMM_TC, persistent: 2 = two CTAs of a cluster share a 256-row tile; each loads its own rows of
                              the first operand and HALF of the second operand's rows, the multiply-accumulate runs across
                              both SMs (tcgen05 cta_group::2).  K-major operands only, tile_n >= 32.  0 or 1 = one CTA. */
    int32_t ctas_per_sm;   /* GEMM_TC, not persistent: 2 = the register-capped build of the kernel, so that two CTAs share an
                              SM when the record needs at most 112 KB of shared memory and 256 tensor-memory columns (one
                              CTA's set-up and read-out overlap the other's main loop); 1 = all registers, one CTA per SM;
                              0 = the library's choice by grid size (2 when the grid has more than two CTAs per SM). */
    int32_t warp_layout;   /* GEMM_TC: warps by role.  0 = the only layout of each kernel form: 1 TMA + 1 MMA + 8 operand
                              producers that then read out (320 threads), or, persistent, 1 TMA + 1 MMA + 4 transposers + 4
                              read-out warps.  Reserved for further layouts; any other value is invalid. */
    int32_t precision;     /* GEMM_TC: 0 = operands are read by the tensor core as TF32 (their fp32 values truncated to 10
                              mantissa bits).  1 = error-compensated ("3xTF32"): each operand tile is split in shared memory
                              into what the tensor core sees and the remainder, and every reduction step issues three
                              multiply-accumulates (a*b_lo, a_lo*b, a*b), which brings the result to within fp32
                              accumulation error of the exact product at three times the tensor work and twice the
                              shared memory per stage.  One-tile form, dense and batch_matmul NT with K a multiple of 4;
                              elsewhere legalised to 0 (TT_CHG_FORM). */
} tt_schedule_record;

typedef struct tt_tensors {
    const void* x;
    const void* w;
    const void* bias;      /* NULL when has_bias == 0 */
    const void* residual;  /* NULL when has_residual == 0 */
    void* y;
} tt_tensors;

/* The contraction a GEMM_TC workload is lowered to, and its algorithmic work:
 * flops = 2*batch*gm*gn*gk (depthwise: 2*outputs*r*s; softmax: 5 per element), bytes = 4 * (every tensor once). */
typedef struct tt_gemm_view {
    int32_t batch, gm, gn, gk;
    double flops, bytes;
} tt_gemm_view;

/* What tt_schedule_apply / tt_schedule_check decided. */
typedef struct tt_apply_info {
    tt_schedule_record legal;   /* the record after legalisation: what will actually run */
    int32_t changed;            /* bit mask of fields legalisation had to change (TT_CHG_*) */
    int32_t grid_x, grid_y, grid_z, threads;
    int32_t smem_bytes, tmem_cols;
    int64_t workspace_bytes;
    int32_t launches;           /* kernels per tt_run (2 with split-K) */
} tt_apply_info;

enum { TT_CHG_TILE_M = 1, TT_CHG_TILE_N = 2, TT_CHG_TILE_K = 4, TT_CHG_STAGES = 8, TT_CHG_SPLIT_K = 16,
       TT_CHG_VEC = 32, TT_CHG_BLOCK = 64, TT_CHG_ITEMS = 128, TT_CHG_SLAB = 256, TT_CHG_ACC = 512, TT_CHG_KORDER = 1024,
       TT_CHG_FORM = 2048   /* the record named a kernel form this shape does not have (DW_SIMT unroll / raster) */ };

/* Validity modes for mapping a record onto another shape (Section 4.1).
 *   TT_MODE_LEGALISE  reformulate: clamp/round tile sizes to the new extents and the hardware's legal set,
 *                     lower the vector width to what divides the row, clamp split_k to the reduction tiles;
 *                     invalid only when resources are exceeded or a field is nonsensical.
 *   TT_MODE_STRICT    no reformulation: a record whose tile factor exceeds the loop extent, whose split_k
 *                     exceeds the number of reduction tiles, or that needs any rounding is invalid. */
typedef enum { TT_MODE_LEGALISE = 0, TT_MODE_STRICT = 1 } tt_mode;

typedef struct tt_timing_opts {
    int32_t warmup_batches;   /* default 3 */
    int32_t batches;          /* default 10; the median over batches is reported (evaluation protocol, Section 5.1) */
    int32_t min_batch_us;     /* each batch repeats the launch until it lasts at least this long; default 200 */
    int32_t max_repeats;      /* cap on launches per batch; default 4096 */
    int32_t use_graph;        /* 1: replay each batch as a CUDA graph (no CPU launch gaps) */
    int32_t floor;            /* 1: time, instead of the kernel, an empty kernel launched the same way (same grid, block
                                 size, shared memory, cluster shape, dependent launch): what a launch of this record costs
                                 before it does any work */
    int32_t reserved[2];
} tt_timing_opts;

typedef struct tt_timing {
    float median_us, min_us, max_us, q1_us, q3_us;  /* per launch of the whole workload (all its kernels) */
    int32_t repeats, batches;
} tt_timing;

typedef struct tt_tune_opts {
    tt_timing_opts timing;
    int32_t mode;            /* tt_mode */
    int32_t strict_class;    /* 1: the record's origin kernel class (op, bias, activation, residual) must equal the
                                workload's (the paper's rule); 0: same family suffices */
    int32_t include_default; /* 1 (default): column 0 of the table is the workload's default ("untuned") record */
    int32_t subsample_percent; /* 0 or 100: every pool record is evaluated.  1..99: per workload, a seeded subset of that
                                share of the pool (tt_pool_subsample; at least one record) is evaluated first, and the
                                rest only if the subset's best time is not below the default record's by more than
                                subsample_gain_percent.  Records left out are marked TT_SKIPPED (time -1).  The paper
                                notes that a larger pool lengthens the search (Section 5.5); this bounds it. */
    int32_t subsample_gain_percent; /* the gain over the default record that ends a workload's search early */
    uint32_t subsample_seed;
    int32_t reserved[2];
} tt_tune_opts;

/* Result arrays are allocated by the caller.  n_cols = n_pool + 1; column 0 is the default record, column j+1 is
 * pool[j].  times_us < 0 marks an invalid pair (plotted as -1 in the paper's Figure 4). */
typedef struct tt_tune_result {
    int32_t* chosen;        /* [n_wl]        column index of the fastest valid record, -1 if none */
    float* best_us;         /* [n_wl]        */
    float* times_us;        /* [n_wl*n_cols] */
    int32_t* status;        /* [n_wl*n_cols] tt_status of apply/timing for the pair */
    double search_seconds;  /* wall time of the call: apply + warm-up + timing + selection */
    int32_t pairs_timed, pairs_invalid;
    int32_t pairs_skipped;  /* pairs left out by pool sub-sampling */
} tt_tune_result;

typedef struct tt_workload tt_workload;

const char* tt_status_string(tt_status s);

/* Create a kernel from its operator and data sizes (Section 4.2: a kernel is its class plus its sizes).
 * Validates the shape (positive extents, filter fits the padded input). */
tt_status tt_workload_create(tt_op op, const tt_shapes* shapes, tt_workload** out);
tt_status tt_workload_destroy(tt_workload* w);
/* Workload ID: hash of operator type and sizes; identical kernels share schedules and are tuned once (Section 2). */
tt_status tt_workload_key(const tt_workload* w, uint64_t* key);
/* Kernel class: hash of (operator, bias, activation, residual) only, regardless of sizes (Section 4.2). */
tt_status tt_workload_class(const tt_workload* w, uint64_t* cls);
tt_status tt_workload_family(const tt_workload* w, int32_t* family);
tt_status tt_workload_gemm_view(const tt_workload* w, tt_gemm_view* out);
/* The built-in "untuned" record of the workload's family: baseline of every speedup and fallback when no
 * pool record is valid (Section 4.3). */
tt_status tt_default_schedule(const tt_workload* w, tt_schedule_record* out);

/* Host-only: legalise and validate `rec` against `w` without touching the device. */
tt_status tt_schedule_check(const tt_workload* w, const tt_schedule_record* rec, int32_t mode, int32_t strict_class,
                            tt_apply_info* info_out);
/* Legalise, validate and bind `rec` to `w` (tensor maps, descriptors, grid, workspace).  info_out may be NULL.
 * Uses TT_MODE_LEGALISE and family matching; tt_schedule_apply_ex takes both options. */
tt_status tt_schedule_apply(tt_workload* w, const tt_schedule_record* rec, tt_apply_info* info_out);
tt_status tt_schedule_apply_ex(tt_workload* w, const tt_schedule_record* rec, int32_t mode, int32_t strict_class,
                               tt_apply_info* info_out);
/* Literal form of the split example of Section 4.1: does splitting a loop of `extent` iterations by the given
 * factors traverse it exactly?  reformulate != 0 tests Split(N, N/f, f) for the single factor f instead. */
tt_status tt_split_check(int64_t extent, const int64_t* factors, size_t n_factors, int32_t reformulate, int32_t* valid);

/* Run the workload once under the applied record (device pointers). */
tt_status tt_run(tt_workload* w, const tt_tensors* t, void* cuda_stream);
/* The same with HOST pointers: copies x, w, bias, residual to library-owned device buffers, runs, copies y back,
 * synchronises.  bytes_h2d/bytes_d2h (may be NULL) receive the bytes copied. */
tt_status tt_run_host(tt_workload* w, const tt_tensors* host, void* cuda_stream, int64_t* bytes_h2d, int64_t* bytes_d2h);
/* The same without the final synchronisation: the copies and the kernel are only enqueued on `cuda_stream`, so calls
 * for DIFFERENT workloads on different streams overlap their transfers (both directions) and kernels.  The host
 * buffers must be page-locked for the copies to be asynchronous and must stay untouched until the stream has been
 * synchronised; y and the device status are valid after tt_workload_status(w, cuda_stream) (or any synchronisation
 * of that stream).  A workload owns one set of device staging buffers: enqueue its calls on one stream at a time. */
tt_status tt_run_host_async(tt_workload* w, const tt_tensors* host, void* cuda_stream, int64_t* bytes_h2d,
                            int64_t* bytes_d2h);
/* A promise by the caller, off by default: the w and bias tensors passed to tt_run for this workload are constants
 * (the parameters of an inference pass) -- no kernel enqueued directly in front of the run on the same stream writes
 * them.  A dense or conv2d kernel then requests the first tiles of w BEFORE it waits for the kernel in front of it
 * (kernels are launched with programmatic stream serialization), so the weights stream in while that kernel is still
 * running.  Results are unchanged as long as the promise holds.  batch_matmul operands are never treated this way. */
tt_status tt_workload_set_constant_weights(tt_workload* w, int32_t on);
/* Read and clear the device status word of the last runs (TT_OK or TT_ERR_TIMEOUT); synchronises the stream.
 * After a TT_ERR_TIMEOUT the split-K arrival counters of the applied record are cleared too, so the next run starts
 * from a clean workspace (an invalid pair is a result of the search, which then goes on: Section 4.3). */
tt_status tt_workload_status(tt_workload* w, void* cuda_stream);
/* Every wait inside a kernel (on a copy, on a pipeline buffer, on the accumulator) gives up after this many
 * nanoseconds: the kernel then records TT_ERR_TIMEOUT in the status word, lets its copies land, releases its tensor
 * memory and returns, and the context stays usable.  Default: one second.  Takes effect with the next run. */
tt_status tt_workload_set_wait_limit(tt_workload* w, uint64_t nanoseconds);
/* Test facility for that path.  With extra_bytes > 0 (a multiple of 16) the barrier of the first pipeline stage of a
 * GEMM_TC kernel whose operands arrive by TMA is told to expect extra_bytes more than its copies deliver (in the CTAs
 * of the first reduction split only, so that a split-K record is left half finished): every copy still lands, only
 * the barrier never completes, so the wait on it runs into the limit above.  0 switches it off.
 * Nothing traps and nothing waits without a limit. */
tt_status tt_workload_test_stall(tt_workload* w, uint32_t extra_bytes);

/* Time the applied record: warm-up batches, then `batches` batches of back-to-back launches between two CUDA
 * events.  `sets` holds n_sets tensor sets used round-robin (n_sets > 1 with a footprint beyond L2 gives cold-cache
 * times). */
tt_status tt_time(tt_workload* w, const tt_tensors* sets, size_t n_sets, void* cuda_stream, const tt_timing_opts* o,
                  tt_timing* out);

/* Pure host: per row of times_us[n_wl x n_cols] the column of the smallest non-negative time, ties to the lowest
 * column, -1 when the row has none. */
tt_status tt_select(const float* times_us, size_t n_wl, size_t n_cols, int32_t* chosen);
/* Pure host: sum_w use_count[w] * times_us[w, chosen[w]] (kernels assumed independent, Section 2). */
tt_status tt_model_latency(const float* times_us, size_t n_wl, size_t n_cols, const int32_t* chosen,
                           const int32_t* use_count, double* latency_us);

/* Pure host: the model-selection heuristic, Equation 1 of Section 4.4.  For a target model whose kernel classes
 * take the shares class_share[c] (fractions of its untuned inference time) and n_models candidate models with
 * class_kernels[t * n_classes + c] unique kernels of class c, scores[t] = sum_c class_share[c]^2 * sqrt(kernels of
 * class c in t); order[] lists the candidates by decreasing score, ties keeping the lower index first.  scores may
 * be NULL.  Shares can come from the default-record times of the evaluator's table. */
tt_status tt_rank_pools(const double* class_share, size_t n_classes, const int32_t* class_kernels, size_t n_models,
                        double* scores, int32_t* order);

/* The evaluator of Section 4.3: every workload x every compatible pool record (plus the default), standalone, on
 * the workload's own tensors; invalid pairs are recorded, not fatal.  On return each workload is left with its
 * chosen record applied.  tensors[i] belongs to model_workloads[i]. */
tt_status tt_transfer_tune(tt_workload* const* model_workloads, const tt_tensors* tensors, size_t n_wl,
                           const tt_schedule_record* pool, size_t n_pool, const tt_tune_opts* o, void* cuda_stream,
                           tt_tune_result* out);

/* The same with several tensor sets per workload: workload i owns set_counts[i] consecutive entries of `tensors` and
 * every timed batch walks them round-robin.  Sets that differ only in w and bias, with a total footprint beyond the L2,
 * time a kernel the way it runs inside a model: weights from memory, activations from the cache. */
tt_status tt_transfer_tune_sets(tt_workload* const* model_workloads, const tt_tensors* tensors, const size_t* set_counts,
                                size_t n_wl, const tt_schedule_record* pool, size_t n_pool, const tt_tune_opts* o,
                                void* cuda_stream, tt_tune_result* out);

/* Native tuning of one workload (stands in for the auto-scheduler that fills a pool, Section 2): exhaustive walk
 * over a grid of records of the workload's family, each timed with `o`; writes the best `top_k` records (fastest
 * first) to out_records/out_us and their number to n_out.  level 0 = coarse grid, 1 = full grid. */
tt_status tt_grid_tune(tt_workload* w, const tt_tensors* t, void* cuda_stream, const tt_timing_opts* o, int32_t level,
                       size_t top_k, tt_schedule_record* out_records, float* out_us, size_t* n_out,
                       int32_t* n_tried);

/* Schedules persist as records keyed by the kernel they were tuned on (Section 2: tuned schedules are kept in a log and
 * looked up by workload ID).  A pool file is text, one record per line, "field=value" pairs separated by blanks
 * (version, family, origin_op, origin=<the nineteen integers of tt_shapes, comma-separated, then scale>, every
 * record field by name, us=<the time it was tuned to, microseconds>); lines that start with '#' are comments.
 * Pure host.  tt_pool_save overwrites `path`; us may be NULL (written as -1).  tt_pool_load reads at most `cap`
 * records into out/us (us may be NULL), sets *n_out to the number of records in the file (more than cap:
 * TT_ERR_RESOURCE, nothing beyond cap is written); cap == 0 counts only.  A line that cannot be parsed, names an
 * unknown field or carries another record version: TT_ERR_INVALID_ARG.  A missing file: TT_ERR_INVALID_ARG. */
tt_status tt_pool_save(const char* path, const tt_schedule_record* records, const float* us, size_t n);
tt_status tt_pool_load(const char* path, tt_schedule_record* out, float* us, size_t cap, size_t* n_out);

/* Pure host: the first `count` entries of a seeded shuffle of 0 .. n_pool-1 (Fisher-Yates from the front, position i
 * swapped with i + r mod (n_pool - i), r the next output of the splitmix64 generator started at `seed`).  The subset
 * of the pool that sub-sampling evaluates first; count > n_pool: TT_ERR_INVALID_ARG. */
tt_status tt_pool_subsample(size_t n_pool, size_t count, uint64_t seed, int32_t* idx_out);

/* Refining a transferred record (Section 7 names it as the next step: vary the parameters of schedules that were
 * transfer-tuned from another model).  The neighbourhood of a record: every field its family uses is moved one rung
 * down and one rung up its ladder of values (two-valued fields are toggled), one field at a time, in the order the
 * fields are listed below; each candidate is legalised for `w`, and candidates that are invalid, that legalise back
 * to the (legalised) start or that repeat an earlier neighbour are dropped.
 *   GEMM_TC  tile_n {16,32,48,64,96,128,160,192,224,256}  tile_k {8,16,32,64,96,128}  stages {1..8}
 *            split_k {1..8,12,16,24,32}  raster {0,1}  mma_m_axis {1,2}  slab_tiles {0,1,2,4,8}  acc_split {1,2,4,8}
 *            k_order {0,1}  persistent {0,1}  cta_group {1,2}  ctas_per_sm {1,2}
 *   DW_SIMT  tile_m {1,2,4,8,16,32}  block_y {1,2,4,7,8,14,16,28,56}  block_x {8,16,28,32,56,64,112}
 *            items_per_thread {1,2,4,8}  vec_width {1,2,4}  threads {32,...,512}  unroll {0,1,2,4}  raster {0,1}
 *            stages {2,3,4}
 *   ROW_SIMT block_x {1,...,32}  block_y {1,...,16}  vec_width {1,2,4}
 * Pure host.  out[cap] receives the neighbours, *n_out their number (cap == 0: count only; more than cap:
 * TT_ERR_RESOURCE).  At most two per field, so 24 entries always suffice. */
tt_status tt_record_neighbours(const tt_workload* w, const tt_schedule_record* rec, tt_schedule_record* out, size_t cap,
                               size_t* n_out);

/* Time of one record in microseconds, negative when the record cannot run. */
typedef float (*tt_time_fn)(void* user, const tt_schedule_record* rec);

/* Greedy descent over that neighbourhood, pure host given the timing function: the start (legalised) is timed, then,
 * up to max_rounds times, every neighbour of the current record that has not been timed before is timed and the
 * fastest becomes the current record if it beats it by more than the fraction min_gain (ties keep the earlier
 * neighbour); otherwise the search stops.  best/best_us receive the last current record and its time, start_us (may
 * be NULL) the start's time, n_timed (may be NULL) the number of calls of time_us.  TT_ERR_INVALID_SCHEDULE when the
 * start itself cannot run. */
tt_status tt_refine_with(const tt_workload* w, const tt_schedule_record* start, tt_time_fn time_us, void* user,
                         int32_t max_rounds, float min_gain, tt_schedule_record* best, float* best_us, float* start_us,
                         int32_t* n_timed);

/* The same on the device: a record's time is the median of tt_time under `o` on the tensors `t` (records that fail to
 * apply or trip a wait count as unable to run).  On return the best record is applied to `w`. */
tt_status tt_refine(tt_workload* w, const tt_tensors* t, void* cuda_stream, const tt_timing_opts* o,
                    const tt_schedule_record* start, int32_t max_rounds, float min_gain, tt_schedule_record* best,
                    float* best_us, float* start_us, int32_t* n_timed);

/* (No counterpart in the paper.)  dense+bias+activation under a split-K record for callers that cannot allocate
 * device memory when they need the kernel: hosts whose memory pool already owns the whole device, loops that may
 * not take the allocator's lock, plug-ins that are forbidden to allocate after start-up.  The partial sums of the
 * splits, their arrival counters and the status word live in ONE fixed device array of TT_STATIC_SCRATCH_BYTES
 * that belongs to the library image (each device that loads the library holds it until the process exits), so
 * this call makes no cudaMalloc/cudaFree and calls no allocating routine.
 *   x [m,kk], w [nn,kk], bias [nn] or NULL, y [m,nn]: DEVICE pointers, fp32, row-major, 16-byte aligned, owned by
 *   the caller; `rec` is a GEMM_TC record (legalised as in tt_schedule_apply); act is a tt_act.
 *   scratch_bytes_used (may be NULL) receives what the legalised record needs of the array.
 * Errors: TT_ERR_RESOURCE when that exceeds TT_STATIC_SCRATCH_BYTES (lower split_k, or use tt_run, which
 * allocates) or when the record's split-K cluster cannot be resident; the statuses of tt_schedule_apply for a bad
 * record; TT_ERR_CUDA; TT_ERR_TIMEOUT from the kernel.
 * The call launches on `cuda_stream`, synchronises it and reads the status word back before returning, so it cannot
 * be part of a stream capture.  The first call on a device loads the library's device image (which is when the
 * driver sets the array aside) and looks up the array's address, with that device current: make that first call at
 * start-up, before the application declares its allocation phase over.
 * All calls share the array: it keeps the previous call's contents (the words that must start at zero are cleared
 * on the stream before each launch), and two calls that overlap on the GPU race on it -- issue them one at a
 * time per device. */
#define TT_STATIC_SCRATCH_BYTES (8u << 20)
tt_status tt_dense_static_scratch(const void* x, const void* w, const void* bias, void* y, int32_t m, int32_t nn,
                                  int32_t kk, int32_t act, const tt_schedule_record* rec, void* cuda_stream,
                                  int64_t* scratch_bytes_used);

#ifdef __cplusplus
}
#endif
#endif /* TT_H_ */
