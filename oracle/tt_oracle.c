/*
 * CPU oracle for the fused DNN operators that transfer-tuning runs under schedules.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition of what each
 * kernel class computes.  It shares no code with the CUDA library, is never called
 * by the product path, and exists so that tests (and the CPU-baseline leg of the
 * benchmark) have something independent to compare against.
 *
 * A schedule changes how fast a kernel runs, never what it computes (Section 2:
 * the algorithm is described separately from its optimisation), so the oracle is
 * the unscheduled algorithm itself:
 *   - dense / batch_matmul : the unmodified row-major matrix multiply of Algorithm 1
 *   - conv2d(+bias+act)    : the kernel class of Algorithm 2 (pad, conv2d, +B, ReLU)
 *   - dwconv2d             : the same with one filter per channel
 *   - softmax              : the textbook row softmax
 *
 * Every reduction is accumulated in double and rounded to float once at the end;
 * bias, residual and activation are applied in double before that rounding.
 *
 * `mode` selects how the float inputs of a contraction are read:
 *   0 exact fp32 values
 *   1 mantissa truncated to 10 bits   (diagnostic: TF32 by truncation)
 *   2 mantissa rounded to 10 bits, ties away from zero (diagnostic: TF32 by rounding)
 * Modes 1 and 2 are never the pass/fail reference.
 *
 * Parallelism: OpenMP over independent output rows/channels only.  The order of
 * the additions inside one output element never depends on the thread count.
 */
#include <math.h>
#include <stdint.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ACT_NONE = 0, ACT_RELU = 1, ACT_RELU6 = 2, ACT_GELU_ERF = 3 };

static inline double rd(float v, int mode) {
    if (mode == 0) return (double)v;
    uint32_t u;
    memcpy(&u, &v, 4);
    if (mode == 2) u += 0x1000u;          /* half of the dropped 13 bits */
    u &= 0xFFFFE000u;
    float r;
    memcpy(&r, &u, 4);
    return (double)r;
}

static inline double activate(double v, int act) {
    switch (act) {
        case ACT_RELU:     return v > 0.0 ? v : 0.0;
        case ACT_RELU6:    return v < 0.0 ? 0.0 : (v > 6.0 ? 6.0 : v);
        case ACT_GELU_ERF: return 0.5 * v * (1.0 + erf(v * 0.70710678118654752440));
        default:           return v;
    }
}

int orc_max_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

static int pick_threads(int threads) {
#ifdef _OPENMP
    int mx = omp_get_max_threads();
    if (threads <= 0 || threads > mx) threads = mx;
    return threads;
#else
    (void)threads;
    return 1;
#endif
}

/* Algorithm 2: Y = act(Conv2d(Pad(X)) + B [+ residual]).  Cross-correlation, zero
 * padding of ph/pw on each side, dilation 1.  X[N,C,H,W], Wt[K,C,R,S], bias[K] or
 * NULL, residual[N,K,P,Q] or NULL, Y[N,K,P,Q], P = (H+2ph-R)/sh+1.
 * Returns the thread count used. */
int orc_conv2d(const float* x, const float* wt, const float* bias, const float* residual, float* y,
               int N, int C, int H, int W, int K, int R, int S, int sh, int sw, int ph, int pw,
               int act, int mode, int threads) {
    const int P = (H + 2 * ph - R) / sh + 1;
    const int Q = (W + 2 * pw - S) / sw + 1;
    threads = pick_threads(threads);
    const long NK = (long)N * K;
#pragma omp parallel for schedule(dynamic, 1) num_threads(threads)
    for (long nk = 0; nk < NK; ++nk) {
        const int n = (int)(nk / K), k = (int)(nk % K);
        for (int p = 0; p < P; ++p) {
            for (int q = 0; q < Q; ++q) {
                double acc = 0.0;
                for (int c = 0; c < C; ++c) {
                    for (int r = 0; r < R; ++r) {
                        const int ih = p * sh + r - ph;
                        if (ih < 0 || ih >= H) continue;      /* padded zero */
                        for (int s = 0; s < S; ++s) {
                            const int iw = q * sw + s - pw;
                            if (iw < 0 || iw >= W) continue;  /* padded zero */
                            acc += rd(x[(((long)n * C + c) * H + ih) * W + iw], mode) *
                                   rd(wt[(((long)k * C + c) * R + r) * S + s], mode);
                        }
                    }
                }
                const long o = (((long)n * K + k) * P + p) * Q + q;
                if (bias) acc += (double)bias[k];
                if (residual) acc += (double)residual[o];
                y[o] = (float)activate(acc, act);
            }
        }
    }
    return threads;
}

/* Depthwise variant of Algorithm 2: one R x S filter per channel, multiplier 1.
 * X[N,C,H,W], Wt[C,1,R,S], bias[C] or NULL, Y[N,C,P,Q]. */
int orc_dwconv2d(const float* x, const float* wt, const float* bias, float* y,
                 int N, int C, int H, int W, int R, int S, int sh, int sw, int ph, int pw,
                 int act, int threads) {
    const int P = (H + 2 * ph - R) / sh + 1;
    const int Q = (W + 2 * pw - S) / sw + 1;
    threads = pick_threads(threads);
    const long NC = (long)N * C;
#pragma omp parallel for schedule(dynamic, 1) num_threads(threads)
    for (long nc = 0; nc < NC; ++nc) {
        const int c = (int)(nc % C);
        const float* xc = x + nc * H * W;
        for (int p = 0; p < P; ++p) {
            for (int q = 0; q < Q; ++q) {
                double acc = 0.0;
                for (int r = 0; r < R; ++r) {
                    const int ih = p * sh + r - ph;
                    if (ih < 0 || ih >= H) continue;
                    for (int s = 0; s < S; ++s) {
                        const int iw = q * sw + s - pw;
                        if (iw < 0 || iw >= W) continue;
                        acc += (double)xc[(long)ih * W + iw] * (double)wt[((long)c * R + r) * S + s];
                    }
                }
                if (bias) acc += (double)bias[c];
                y[(nc * P + p) * Q + q] = (float)activate(acc, act);
            }
        }
    }
    return threads;
}

/* Algorithm 1, unmodified row-major matrix multiply, one per batch entry:
 *   C[b][n][m] = sum_k A[b][n][k] * Bm[b][k][m]            (trans_b = 0, Bm is [K,M])
 *   C[b][n][m] = sum_k A[b][n][k] * Bm[b][m][k]            (trans_b = 1, Bm is [M,K])
 * followed by + bias[m] (or NULL) and the activation.  The paper's names: A is
 * N x K, B is K x M, C is N x M.  dense+bias is batch = 1, trans_b = 1 with the
 * weight stored [out, in]. */
int orc_batch_matmul(const float* a, const float* bm, const float* bias, float* c,
                     int batch, int N, int M, int K, int trans_b, int act, int mode, int threads) {
    threads = pick_threads(threads);
    const long rows = (long)batch * N;
#pragma omp parallel for schedule(dynamic, 1) num_threads(threads)
    for (long bn = 0; bn < rows; ++bn) {
        const long b = bn / N;
        const float* arow = a + bn * K;
        const float* bb = bm + b * (long)K * M;
        for (int m = 0; m < M; ++m) {
            double acc = 0.0;
            for (int k = 0; k < K; ++k) {
                const float bv = trans_b ? bb[(long)m * K + k] : bb[(long)k * M + m];
                acc += rd(arow[k], mode) * rd(bv, mode);
            }
            if (bias) acc += (double)bias[m];
            c[bn * M + m] = (float)activate(acc, act);
        }
    }
    return threads;
}

/* Row softmax over the last axis of scale * S[rows, cols]. */
int orc_softmax(const float* s, float* p, long rows, int cols, float scale, int threads) {
    threads = pick_threads(threads);
#pragma omp parallel for schedule(static) num_threads(threads)
    for (long i = 0; i < rows; ++i) {
        const float* si = s + i * cols;
        double mx = -INFINITY;
        for (int j = 0; j < cols; ++j) {
            const double v = (double)scale * (double)si[j];
            if (v > mx) mx = v;
        }
        double sum = 0.0;
        for (int j = 0; j < cols; ++j) sum += exp((double)scale * (double)si[j] - mx);
        for (int j = 0; j < cols; ++j)
            p[i * cols + j] = (float)(exp((double)scale * (double)si[j] - mx) / sum);
    }
    return threads;
}
