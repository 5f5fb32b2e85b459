/*
 * CPU oracle for the Per-Token-Static (PTS) W8A8 linear layer of PTQ4VM
 * (arXiv 2412.20386).  TEST INFRASTRUCTURE ONLY: this file exists so that the
 * GPU library can be checked against an independent, slow, plainly written
 * implementation.  Nothing in the product path may call it, and it shares no
 * code, header, table or constant with the CUDA sources.
 *
 * Every function is a scalar loop nest that follows the paper's equations in
 * the paper's order.  The only parallelism is an OpenMP "for" over independent
 * rows.  No intrinsics, no BLAS, no blocking, no fusion.
 *
 * Notation (Sec. 5.1): M = B*T token rows, token position t = m mod T,
 * x[m,k] fp16 activations (row-major), Wq[n,k] integer weights (row-major, the
 * paper's W-bar, already smoothed and quantized offline, Sec. 2.3 weight
 * quantizer), dw[n] = Delta_W per output channel, s[k] = smoothing scale
 * (Eq. smooth_scale), dx[t] = Delta_X per token position.
 *
 * Parity status of each function is listed in its comment; all of them are
 * pinned by tests that do not route through this file (numpy float32/float64
 * evaluations, closed forms, brute force).
 *
 * Build: gcc -O2 -fopenmp -ffp-contract=off -fno-fast-math -shared -fPIC
 */
#include <math.h>
#include <stdint.h>
#include <stddef.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#define PTQO_MAX_K 8192   /* row buffer of ptqo_linear_forward_rows */

int ptqo_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ------------------------------------------------------------------------- */
/* IEEE binary16 <-> wider formats, written out from the format definition.   */
/* Pinned against numpy's float16 conversions on all 65536 bit patterns and   */
/* on every rounding midpoint.                                                */
/* ------------------------------------------------------------------------- */

/* binary16 bits -> float (exact: every binary16 value is a binary32 value). */
float ptqo_half_to_float(uint16_t h)
{
    int sign = (h >> 15) & 1;
    int expo = (h >> 10) & 0x1f;
    int frac = h & 0x3ff;
    float v;
    if (expo == 0x1f) {
        v = frac ? NAN : INFINITY;
    } else if (expo == 0) {
        v = ldexpf((float)frac, -24);               /* subnormal: frac * 2^-24 */
    } else {
        v = ldexpf((float)(1024 + frac), expo - 25); /* (1+frac/1024) * 2^(expo-15) */
    }
    return sign ? -v : v;
}

/* double -> binary16 bits with ONE rounding (nearest, ties to even), overflow
 * to infinity as IEEE prescribes.  The scaling steps are by powers of two and
 * therefore exact; nearbyint() in the default rounding mode is ties-to-even. */
uint16_t ptqo_double_to_half(double v)
{
    uint16_t sign = 0;
    double a;
    if (isnan(v)) return 0x7e00;
    if (signbit(v)) sign = 0x8000;
    a = fabs(v);
    if (a >= 65520.0) return (uint16_t)(sign | 0x7c00);   /* 65520 = midpoint(65504, 2^16) ties to 2^16 = inf */
    if (a < 6.103515625e-05) {                            /* below 2^-14: subnormal grid, spacing 2^-24 */
        double m = nearbyint(ldexp(a, 24));               /* 0 .. 1024; 1024 is the smallest normal */
        return (uint16_t)(sign | (uint16_t)m);
    } else {
        int e;
        double f = frexp(a, &e);                          /* a = f * 2^e, f in [0.5,1) */
        double m = nearbyint(ldexp(f, 11));               /* 1024 .. 2048 */
        int be = e - 1 + 15;                              /* biased exponent of 2^(e-1) */
        if (m == 2048.0) { m = 1024.0; be += 1; }
        return (uint16_t)(sign | (uint16_t)(be << 10) | (uint16_t)((int)m - 1024));
    }
}

/* ------------------------------------------------------------------------- */
/* Step Q1: smoothing + PTS quantization.                                     */
/*   u = x / s[k]          smoothing, diag(s)^-1 X        (Eq. smooth)        */
/*   v = u / dx[t]         per-token-position step        (Sec. 5.1)          */
/*   q = clip(round(v))    round-to-nearest, ties to even (Sec. 2.3 form)     */
/* Both divisions and the rounding are IEEE binary32 (the precision in which  */
/* the integer decision is taken on both sides).  Range [-128, 127];          */
/* NaN -> 0, +inf -> 127, -inf -> -128.                                       */
/* Pinned: all fp16 inputs against numpy float32; ties; clamp; monotonicity.  */
/* ------------------------------------------------------------------------- */
int8_t ptqo_quantize_one(uint16_t x_half, float s, float dx)
{
    volatile float xf = ptqo_half_to_float(x_half);
    volatile float u = xf / s;
    volatile float v = u / dx;
    float r;
    if (isnan(v)) return 0;
    r = nearbyintf(v);
    if (r > 127.0f) r = 127.0f;
    if (r < -128.0f) r = -128.0f;
    return (int8_t)r;
}

void ptqo_quantize(const uint16_t *x, long M, int K, int T,
                   const float *s, const float *dx, int8_t *q)
{
    long m;
#pragma omp parallel for schedule(static)
    for (m = 0; m < M; ++m) {
        int t = (int)(m % T);
        int k;
        for (k = 0; k < K; ++k)
            q[m * K + k] = ptqo_quantize_one(x[m * K + k], s[k], dx[t]);
    }
}

/* ------------------------------------------------------------------------- */
/* Step G1: integer contraction  acc[m,n] = sum_k q[m,k] * Wq[n,k]            */
/* (W-bar . X-bar of Sec. 5.1, written row-major).  Accumulates in 64 bits    */
/* and reports through the return value whether every sum fits in int32.      */
/* Pinned: numpy int64 matmul, hand-checkable tiny cases, one-hot selection.  */
/* ------------------------------------------------------------------------- */
int ptqo_int_matmul(const int8_t *q, const int8_t *wq, long M, int K, int N, int32_t *acc)
{
    long m;
    int overflow = 0;
#pragma omp parallel for schedule(static) reduction(|:overflow)
    for (m = 0; m < M; ++m) {
        int n, k;
        for (n = 0; n < N; ++n) {
            int64_t sum = 0;
            for (k = 0; k < K; ++k)
                sum += (int64_t)q[m * K + k] * (int64_t)wq[(long)n * K + k];
            if (sum > INT32_MAX || sum < INT32_MIN) overflow = 1;
            acc[m * N + n] = (int32_t)sum;
        }
    }
    return overflow;
}

/* ------------------------------------------------------------------------- */
/* Step E1: dequantization  Y = diag(Delta_W) (W-bar X-bar) diag(Delta_X)     */
/* (Sec. 5.1), plus the optional per-output-channel bias, evaluated in        */
/* binary64 and rounded once to binary16.                                     */
/* Pinned: float64 product of the dequantized operands; power-of-two steps.   */
/* ------------------------------------------------------------------------- */
void ptqo_dequant(const int32_t *acc, long M, int N, int T,
                  const float *dx, const float *dw, const float *bias, uint16_t *y)
{
    long m;
#pragma omp parallel for schedule(static)
    for (m = 0; m < M; ++m) {
        int t = (int)(m % T);
        int n;
        for (n = 0; n < N; ++n) {
            double yd = (double)acc[m * N + n] * (double)dx[t] * (double)dw[n];
            if (bias) yd += (double)bias[n];
            y[m * N + n] = ptqo_double_to_half(yd);
        }
    }
}

/* The whole path on a contiguous range of rows [m0, m1) of x[M,K]:
 * Q1 -> G1 -> E1.  q_out / acc_out may be NULL; when given they are dense
 * [m1-m0, K] and [m1-m0, N].  Returns the overflow flag of the contraction,
 * or -1 when K exceeds the row buffer. */
int ptqo_linear_forward_rows(const uint16_t *x, long m0, long m1, int K, int N, int T,
                             const int8_t *wq, const float *dw, const float *s,
                             const float *dx, const float *bias,
                             uint16_t *y, int8_t *q_out, int32_t *acc_out)
{
    long m;
    int overflow = 0;
    if (K > PTQO_MAX_K) return -1;
#pragma omp parallel for schedule(static) reduction(|:overflow)
    for (m = m0; m < m1; ++m) {
        int t = (int)(m % T);
        int8_t qrow[PTQO_MAX_K];
        int n, k;
        for (k = 0; k < K; ++k) {
            qrow[k] = ptqo_quantize_one(x[m * K + k], s[k], dx[t]);
            if (q_out) q_out[(m - m0) * K + k] = qrow[k];
        }
        for (n = 0; n < N; ++n) {
            int64_t sum = 0;
            double yd;
            for (k = 0; k < K; ++k)
                sum += (int64_t)qrow[k] * (int64_t)wq[(long)n * K + k];
            if (sum > INT32_MAX || sum < INT32_MIN) overflow = 1;
            if (acc_out) acc_out[(m - m0) * N + n] = (int32_t)sum;
            yd = (double)(int32_t)sum * (double)dx[t] * (double)dw[n];
            if (bias) yd += (double)bias[n];
            y[(m - m0) * N + n] = ptqo_double_to_half(yd);
        }
    }
    return overflow;
}

/* ------------------------------------------------------------------------- */
/* Step Q0: min-max calibration of the static parameters.                     */
/*   maxX[k] = max_{b,t} |x[b,t,k]|                                            */
/*   maxW[k] = max_n |Wq[n,k]| * dw[n]      (magnitude of the given weights)  */
/*   s[k]    = sqrt( max(maxX,floor) / max(maxW,floor) )   (Eq. smooth_scale) */
/*   dx[t]   = max( max_{b,k} |x[b,t,k] / s[k]|, floor ) / 127                */
/* with floor = 1e-5 guarding all-zero channels and positions.  All binary32, */
/* each operation correctly rounded; max is order independent, so the result  */
/* has exactly one correct value.                                             */
/* Pinned: numpy float32 evaluation; no-clip invariant on the calibration set.*/
/* ------------------------------------------------------------------------- */
void ptqo_calibrate(const uint16_t *xcal, int Bc, int T, int K,
                    const int8_t *wq, const float *dw, int N,
                    float *s, float *dx)
{
    const float floor_ = 1e-5f;
    long M = (long)Bc * T;
    int k, t;
    for (k = 0; k < K; ++k) {
        float mx = 0.0f, mw = 0.0f;
        long m;
        int n;
        for (m = 0; m < M; ++m) {
            float a = fabsf(ptqo_half_to_float(xcal[m * K + k]));
            if (a > mx) mx = a;
        }
        for (n = 0; n < N; ++n) {
            volatile float a = fabsf((float)wq[(long)n * K + k]) * dw[n];
            if (a > mw) mw = a;
        }
        if (mx < floor_) mx = floor_;
        if (mw < floor_) mw = floor_;
        {
            volatile float ratio = mx / mw;
            s[k] = sqrtf(ratio);
        }
    }
    for (t = 0; t < T; ++t) {
        float mu = 0.0f;
        int b;
        for (b = 0; b < Bc; ++b) {
            long m = (long)b * T + t;
            for (k = 0; k < K; ++k) {
                volatile float u = ptqo_half_to_float(xcal[m * K + k]) / s[k];
                float a = fabsf(u);
                if (a > mu) mu = a;
            }
        }
        if (mu < floor_) mu = floor_;
        {
            volatile float d = mu / 127.0f;
            dx[t] = d;
        }
    }
}

/* Per-tensor static comparator (the coarsest granularity in the latency      */
/* table of Sec. 6 and in Fig. 5): the smoothing scales of ptqo_calibrate and */
/* ONE step for the whole activation tensor,                                  */
/*   delta = max( max_{b,t,k} |x[b,t,k] / s[k]|, 1e-5 ) / 127,                */
/* i.e. the min-max rule of Sec. 2.3 taken over every token position at once. */
/* Pinned: numpy float32; equals the largest per-position step; never clips   */
/* the calibration batch; degenerate (all-zero) batch gives the floor.        */
void ptqo_calibrate_per_tensor(const uint16_t *xcal, int Bc, int T, int K,
                               const int8_t *wq, const float *dw, int N,
                               float *s, float *delta)
{
    const float floor_ = 1e-5f;
    long M = (long)Bc * T, m;
    int k;
    float mu = 0.0f;
    float *dx_pos = (float *)malloc(sizeof(float) * (size_t)T);
    ptqo_calibrate(xcal, Bc, T, K, wq, dw, N, s, dx_pos);    /* s only; the per-position steps are discarded */
    free(dx_pos);
    for (m = 0; m < M; ++m)
        for (k = 0; k < K; ++k) {
            volatile float u = ptqo_half_to_float(xcal[m * K + k]) / s[k];
            float a = fabsf(u);
            if (a > mu) mu = a;
        }
    if (mu < floor_) mu = floor_;
    {
        volatile float d = mu / 127.0f;
        *delta = d;
    }
}

/* ========================================================================= */
/* Asymmetric PTS: step AND zero offset per token position (Sec. 5.1 gives    */
/* every token position both parameters; quantizer form of Sec. 2.3:         */
/*   X-hat = Delta (clip(round(X / Delta) + eps, 0, 2^b - 1) - eps) ).        */
/* Reading: the offset eps is an integer z[t] in [0, 255] (the codes must be  */
/* integers for the integer GEMM), the code is                                */
/*   c = clip( round((x / s[k]) / dx[t]) + z[t], 0, 255 )        (unsigned)   */
/* with the same two binary32 divisions and tie rule as the symmetric case,   */
/* NaN -> z[t] (the value zero), +inf -> 255, -inf -> 0, and the contraction  */
/* runs over the offset-free integers:                                        */
/*   acc[m,n] = sum_k (c[m,k] - z[t]) * Wq[n,k].                              */
/* Dequantization is unchanged.                                               */
/* Pinned: numpy float32 on all fp16 inputs; z = 128 reproduces the symmetric */
/* codes; closed form with integer inputs; reconstruction bound; calibration  */
/* against numpy and the never-clips invariant.                               */
/* ========================================================================= */
uint8_t ptqo_quantize_asym_one(uint16_t x_half, float s, float dx, int z)
{
    volatile float xf = ptqo_half_to_float(x_half);
    volatile float u = xf / s;
    volatile float v = u / dx;
    double r;
    if (isnan(v)) return (uint8_t)z;
    r = (double)nearbyintf(v) + (double)z;      /* exact in binary64, also for infinities */
    if (r > 255.0) r = 255.0;
    if (r < 0.0) r = 0.0;
    return (uint8_t)r;
}

void ptqo_quantize_asym(const uint16_t *x, long M, int K, int T,
                        const float *s, const float *dx, const int32_t *z, uint8_t *c)
{
    long m;
#pragma omp parallel for schedule(static)
    for (m = 0; m < M; ++m) {
        int t = (int)(m % T);
        int k;
        for (k = 0; k < K; ++k)
            c[m * K + k] = ptqo_quantize_asym_one(x[m * K + k], s[k], dx[t], z[t]);
    }
}

int ptqo_int_matmul_asym(const uint8_t *c, const int32_t *z, int T, const int8_t *wq,
                         long M, int K, int N, int32_t *acc)
{
    long m;
    int overflow = 0;
#pragma omp parallel for schedule(static) reduction(|:overflow)
    for (m = 0; m < M; ++m) {
        int t = (int)(m % T);
        int n, k;
        for (n = 0; n < N; ++n) {
            int64_t sum = 0;
            for (k = 0; k < K; ++k)
                sum += ((int64_t)c[m * K + k] - (int64_t)z[t]) * (int64_t)wq[(long)n * K + k];
            if (sum > INT32_MAX || sum < INT32_MIN) overflow = 1;
            acc[m * N + n] = (int32_t)sum;
        }
    }
    return overflow;
}

/* Min-max calibration with zero offset:                                      */
/*   s[k] as in ptqo_calibrate (Eq. smooth_scale)                             */
/*   lo[t] = min(0, min_{b,k} x/s),  hi[t] = max(0, max_{b,k} x/s)            */
/*   dx[t] = max(hi - lo, floor) / 255          (Delta_X of Sec. 2.3)         */
/*   z[t]  = clip(round(-lo / dx[t]), 0, 255)   (eps_X of Sec. 2.3, rounded)  */
/* The range always contains zero, so that zero is a code.                    */
void ptqo_calibrate_asym(const uint16_t *xcal, int Bc, int T, int K,
                         const int8_t *wq, const float *dw, int N,
                         float *s, float *dx, int32_t *z)
{
    const float floor_ = 1e-5f;
    float *dx_sym = (float *)malloc(sizeof(float) * (size_t)T);
    int t;
    ptqo_calibrate(xcal, Bc, T, K, wq, dw, N, s, dx_sym);    /* s only; the symmetric steps are discarded */
    free(dx_sym);
    for (t = 0; t < T; ++t) {
        float lo = 0.0f, hi = 0.0f;
        int b, k;
        for (b = 0; b < Bc; ++b) {
            long m = (long)b * T + t;
            for (k = 0; k < K; ++k) {
                volatile float u = ptqo_half_to_float(xcal[m * K + k]) / s[k];
                if (u < lo) lo = u;
                if (u > hi) hi = u;
            }
        }
        {
            volatile float range = hi - lo;
            volatile float d;
            volatile float zr;
            float r;
            if (range < floor_) range = floor_;
            d = range / 255.0f;
            zr = -lo / d;
            r = nearbyintf(zr);
            if (r > 255.0f) r = 255.0f;
            if (r < 0.0f) r = 0.0f;
            dx[t] = d;
            z[t] = (int32_t)r;
        }
    }
}

/* Whole asymmetric path on rows [m0, m1): codes, offset-free accumulators, fp16 output. */
int ptqo_linear_forward_rows_asym(const uint16_t *x, long m0, long m1, int K, int N, int T,
                                  const int8_t *wq, const float *dw, const float *s,
                                  const float *dx, const int32_t *z, const float *bias,
                                  uint16_t *y, uint8_t *c_out, int32_t *acc_out)
{
    long m;
    int overflow = 0;
    if (K > PTQO_MAX_K) return -1;
#pragma omp parallel for schedule(static) reduction(|:overflow)
    for (m = m0; m < m1; ++m) {
        int t = (int)(m % T);
        uint8_t crow[PTQO_MAX_K];
        int n, k;
        for (k = 0; k < K; ++k) {
            crow[k] = ptqo_quantize_asym_one(x[m * K + k], s[k], dx[t], z[t]);
            if (c_out) c_out[(m - m0) * K + k] = crow[k];
        }
        for (n = 0; n < N; ++n) {
            int64_t sum = 0;
            double yd;
            for (k = 0; k < K; ++k)
                sum += ((int64_t)crow[k] - (int64_t)z[t]) * (int64_t)wq[(long)n * K + k];
            if (sum > INT32_MAX || sum < INT32_MIN) overflow = 1;
            if (acc_out) acc_out[(m - m0) * N + n] = (int32_t)sum;
            yd = (double)(int32_t)sum * (double)dx[t] * (double)dw[n];
            if (bias) yd += (double)bias[n];
            y[(m - m0) * N + n] = ptqo_double_to_half(yd);
        }
    }
    return overflow;
}

/* ========================================================================= */
/* Comparator: per-token DYNAMIC quantization (the slower alternative the     */
/* paper measures against PTS, Sec. 4.1 and Table "Latency comparison"): the  */
/* step of a token row is computed from that row at run time,                 */
/*   u[m,k] = x[m,k] / s[k],  dx_row[m] = max( max_k |u[m,k]|, 1e-5 ) / 127,  */
/*   q[m,k] = clip( round(u[m,k] / dx_row[m]), -128, 127 ),                   */
/* all in binary32 with the tie and special-value rules of the static case.   */
/* The paper gives no formula for it; this is the usual symmetric min-max     */
/* per-token rule.  The contraction and dequantization are the static ones    */
/* with T = M and dx = dx_row.                                                */
/* Pinned: numpy float32; every row reaches +-127 and never -128; equals the  */
/* static quantizer fed with the row steps; power-of-two row scaling.         */
/* ========================================================================= */
void ptqo_quantize_dynamic(const uint16_t *x, long M, int K, const float *s, int8_t *q, float *dx_row)
{
    const float floor_ = 1e-5f;
    long m;
#pragma omp parallel for schedule(static)
    for (m = 0; m < M; ++m) {
        float mu = 0.0f;
        int k;
        for (k = 0; k < K; ++k) {
            volatile float u = ptqo_half_to_float(x[m * K + k]) / s[k];
            float a = fabsf(u);
            if (a > mu) mu = a;                 /* NaN never wins the comparison */
        }
        if (mu < floor_) mu = floor_;
        {
            volatile float d = mu / 127.0f;
            dx_row[m] = d;
        }
        for (k = 0; k < K; ++k)
            q[m * K + k] = ptqo_quantize_one(x[m * K + k], s[k], dx_row[m]);
    }
}

/* ========================================================================= */
/* Step-size search (Sec. 5.2, second stage; the "+Truncation" row of the     */
/* ablation table): per token position, the step that minimises the L2        */
/* distance between the smoothed calibration activations and their            */
/* dequantized codes, searched over a grid of truncation ratios.  The paper   */
/* states the loss and that it is a grid search, not the grid; here           */
/*   Delta[t,j] = base[t] * (j / n_grid)        j = j_lo .. n_grid            */
/*   u = x / s[k],  q = clip(round(u / Delta[t,j]), -128, 127)                */
/*   e = u - Delta[t,j] * q     (one rounding: fused multiply-add, binary32)  */
/*   loss[t,j] = sum_{b,k} e^2  (binary64 sum; non-finite u are skipped)      */
/*   best[t] = the j of least loss, the LARGEST such j on equal losses        */
/* with base[t] normally the min-max step (j = n_grid is "no truncation").    */
/* Pinned: exact rational brute force on tiny inputs; zero loss on grid       */
/* points; Delta^2/12 law without clipping; truncation wins with an outlier.  */
/* ========================================================================= */
void ptqo_search_act_step(const uint16_t *xcal, int Bc, int T, int K, const float *s, const float *base,
                          int n_grid, int j_lo, double *loss, int32_t *best, float *dx)
{
    const int C = n_grid - j_lo + 1;
    int t;
#pragma omp parallel for schedule(static)
    for (t = 0; t < T; ++t) {
        int j, best_j = n_grid;
        double best_loss = 0.0;
        for (j = n_grid; j >= j_lo; --j) {
            volatile float ratio = (float)j / (float)n_grid;
            volatile float delta = base[t] * ratio;
            double acc = 0.0;
            int b, k;
            for (b = 0; b < Bc; ++b) {
                long m = (long)b * T + t;
                for (k = 0; k < K; ++k) {
                    volatile float u = ptqo_half_to_float(xcal[m * K + k]) / s[k];
                    volatile float v;
                    float r, e;
                    if (!isfinite(u)) continue;
                    v = u / delta;
                    r = nearbyintf(v);
                    if (r > 127.0f) r = 127.0f;
                    if (r < -128.0f) r = -128.0f;
                    e = fmaf(-delta, r, u);
                    acc += (double)e * (double)e;
                }
            }
            loss[(long)t * C + (j - j_lo)] = acc;
            if (j == n_grid || acc < best_loss) {     /* descending j and strict '<': ties keep the larger j */
                best_loss = acc;
                best_j = j;
            }
        }
        best[t] = best_j;
        {
            volatile float ratio = (float)best_j / (float)n_grid;
            volatile float delta = base[t] * ratio;
            dx[t] = delta;
        }
    }
}

/* ========================================================================= */
/* 4-bit variant (W4A4 of the paper's latency table; Appendix B.1, part 2).   */
/* Same quantizer with the signed 4-bit range:                                */
/*   q4 = clip(round((x / s[k]) / dx[t]), -8, 7),   NaN -> 0, +-inf -> 7 / -8 */
/* and the min-max step dx[t] = max(max|x/s|, 1e-5) / 7.  Two adjacent 4-bit  */
/* values share a byte as the paper's packing step states: the value of even  */
/* index in the low nibble, the next one in the high nibble,                  */
/*   byte = (d[2i+1] << 4) | (d[2i] & 15);                                    */
/* an odd-length row ends with a zero high nibble.  Unpacking sign-extends.   */
/* The contraction and the dequantization are those of the 8-bit path.        */
/* Pinned: hand-evaluated bytes of the packing formula (tests/golden);        */
/* round trip over all nibble pairs; clip(q8) relation to the pinned 8-bit    */
/* quantizer; numpy float32; no-clip invariant of the calibration.            */
/* ========================================================================= */
int8_t ptqo_quantize4_one(uint16_t x_half, float s, float dx)
{
    volatile float xf = ptqo_half_to_float(x_half);
    volatile float u = xf / s;
    volatile float v = u / dx;
    float r;
    if (isnan(v)) return 0;
    r = nearbyintf(v);
    if (r > 7.0f) r = 7.0f;
    if (r < -8.0f) r = -8.0f;
    return (int8_t)r;
}

void ptqo_quantize4(const uint16_t *x, long M, int K, int T, const float *s, const float *dx, int8_t *q)
{
    long m;
#pragma omp parallel for schedule(static)
    for (m = 0; m < M; ++m) {
        int t = (int)(m % T);
        int k;
        for (k = 0; k < K; ++k)
            q[m * K + k] = ptqo_quantize4_one(x[m * K + k], s[k], dx[t]);
    }
}

/* rows of `cols` 4-bit values (each in [-8, 7], one per int8) -> rows of (cols + 1) / 2 bytes */
void ptqo_pack_int4(const int8_t *d, long rows, int cols, uint8_t *packed)
{
    const int pb = (cols + 1) / 2;
    long r;
    for (r = 0; r < rows; ++r) {
        int i;
        for (i = 0; i < pb; ++i) {
            int lo = d[r * cols + 2 * i];
            int hi = (2 * i + 1 < cols) ? d[r * cols + 2 * i + 1] : 0;
            packed[r * pb + i] = (uint8_t)(((hi << 4) | (lo & 15)) & 0xff);
        }
    }
}

void ptqo_unpack_int4(const uint8_t *packed, long rows, int cols, int8_t *d)
{
    const int pb = (cols + 1) / 2;
    long r;
    for (r = 0; r < rows; ++r) {
        int k;
        for (k = 0; k < cols; ++k) {
            int nib = (packed[r * pb + k / 2] >> ((k & 1) * 4)) & 15;
            d[r * cols + k] = (int8_t)(nib >= 8 ? nib - 16 : nib);
        }
    }
}

/* s[k] as in ptqo_calibrate (the weights are the unpacked 4-bit values); dx[t] = max(max|x/s|, floor) / 7 */
void ptqo_calibrate4(const uint16_t *xcal, int Bc, int T, int K, const int8_t *wq, const float *dw, int N,
                     float *s, float *dx)
{
    const float floor_ = 1e-5f;
    int t;
    ptqo_calibrate(xcal, Bc, T, K, wq, dw, N, s, dx);     /* s only; the 8-bit steps are replaced below */
    for (t = 0; t < T; ++t) {
        float mu = 0.0f;
        int b, k;
        for (b = 0; b < Bc; ++b) {
            long m = (long)b * T + t;
            for (k = 0; k < K; ++k) {
                volatile float u = ptqo_half_to_float(xcal[m * K + k]) / s[k];
                float a = fabsf(u);
                if (a > mu) mu = a;
            }
        }
        if (mu < floor_) mu = floor_;
        {
            volatile float d = mu / 7.0f;
            dx[t] = d;
        }
    }
}
