/*
 * CPU oracle for local-operator chains: TEST INFRASTRUCTURE, not part of the product.
 *
 * Plain direct-loop definitions of the block-wise local operators of Sec. IV-A of the
 * paper (convolution and max pooling: an output element reads a block of the input whose
 * extent follows from kernel size, padding, dilation and stride) with the element-wise local
 * operators (ReLU, SiLU) and the residual addition applied per output element.
 * Nothing here is blocked, fused or reordered; nothing here is shared with the CUDA
 * library.  Only tests, the smoke check and the benchmark's CPU-baseline leg call it.
 *
 * Layout: activations NHWC, weights [cout][kh][kw][cin], all float32 in memory.  On the
 * "bf16 path" every stored value is a float32 that is exactly representable in bfloat16:
 * inputs arrive that way and each layer output is rounded (nearest, ties to even) when it
 * is stored.
 *
 * Each routine computes the output rows oh in [oh_lo, oh_hi) of the FULL output tensor
 * and leaves every other row untouched, so the same routine serves whole-tensor
 * execution (oh_lo = 0, oh_hi = H_out) and band-wise execution.
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

/* float -> nearest bfloat16-representable float, ties to even (NaN passed through). */
float lop_oracle_bf16_rne(float v)
{
    uint32_t u;
    memcpy(&u, &v, 4);
    if ((u & 0x7F800000u) == 0x7F800000u && (u & 0x007FFFFFu)) {   /* NaN: keep it a NaN */
        u |= 0x00400000u;
        u &= 0xFFFF0000u;
    } else {
        uint32_t lsb = (u >> 16) & 1u;
        u += 0x7FFFu + lsb;
        u &= 0xFFFF0000u;
    }
    memcpy(&v, &u, 4);
    return v;
}

static float activate(float t, int act)
{
    if (act == 1) return t > 0.0f ? t : 0.0f;                /* ReLU */
    if (act == 2) return t / (1.0f + expf(-t));              /* SiLU */
    if (act == 3) return 0.5f * t * (1.0f + erff(t * 0.70710678118654752f));   /* GELU, t * Phi(t) with the exact normal CDF */
    return t;
}

/*
 * y[n,oh,ow,co] = epilogue( sum_{kh,kw,ci} x[n, oh*sh-ph+kh*dh, ow*sw-pw+kw*dw, ci] * w[co,kh,kw,ci] )
 * taps outside the input contribute zero.  Accumulation in double, in the order kh, kw, ci.
 * epilogue: t = scale[co]*(float)acc + shift[co]; res_pos==1: t += res; t = act(t); res_pos==2: t += res.
 * scale / shift / res may be NULL (1 / 0 / none).  res has the output's shape.
 */
void lop_oracle_conv2d(const float *x, int N, int H, int W, int Cin,
                       const float *w, int Cout, int kh, int kw, int sh, int sw,
                       int ph, int pw, int dh, int dw,
                       const float *scale, const float *shift,
                       const float *res, int res_pos, int act, int round_bf16,
                       int oh_lo, int oh_hi, float *y)
{
    const int Ho = (H + 2 * ph - dh * (kh - 1) - 1) / sh + 1;
    const int Wo = (W + 2 * pw - dw * (kw - 1) - 1) / sw + 1;
    if (oh_lo < 0) oh_lo = 0;
    if (oh_hi > Ho) oh_hi = Ho;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int n = 0; n < N; ++n)
        for (int oh = oh_lo; oh < oh_hi; ++oh)
            for (int ow = 0; ow < Wo; ++ow)
                for (int co = 0; co < Cout; ++co) {
                    double acc = 0.0;
                    for (int a = 0; a < kh; ++a) {
                        const int ih = oh * sh - ph + a * dh;
                        if (ih < 0 || ih >= H) continue;
                        for (int b = 0; b < kw; ++b) {
                            const int iw = ow * sw - pw + b * dw;
                            if (iw < 0 || iw >= W) continue;
                            const float *xp = x + (((size_t)n * H + ih) * W + iw) * Cin;
                            const float *wp = w + (((size_t)co * kh + a) * kw + b) * Cin;
                            for (int ci = 0; ci < Cin; ++ci) acc += (double)xp[ci] * (double)wp[ci];
                        }
                    }
                    const size_t o = (((size_t)n * Ho + oh) * Wo + ow) * Cout + co;
                    float t = (float)acc;
                    t = (scale ? scale[co] : 1.0f) * t + (shift ? shift[co] : 0.0f);
                    if (res && res_pos == 1) t += res[o];
                    t = activate(t, act);
                    if (res && res_pos == 2) t += res[o];
                    y[o] = round_bf16 ? lop_oracle_bf16_rne(t) : t;
                }
}

/*
 * y[n,oh,ow,c] = max over the taps (kh,kw) that fall inside the input; padding never wins
 * (it behaves as minus infinity).  A window with no in-bounds tap yields -inf.
 */
void lop_oracle_maxpool2d(const float *x, int N, int H, int W, int C,
                          int kh, int kw, int sh, int sw, int ph, int pw, int dh, int dw,
                          int oh_lo, int oh_hi, float *y)
{
    const int Ho = (H + 2 * ph - dh * (kh - 1) - 1) / sh + 1;
    const int Wo = (W + 2 * pw - dw * (kw - 1) - 1) / sw + 1;
    if (oh_lo < 0) oh_lo = 0;
    if (oh_hi > Ho) oh_hi = Ho;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int n = 0; n < N; ++n)
        for (int oh = oh_lo; oh < oh_hi; ++oh)
            for (int ow = 0; ow < Wo; ++ow)
                for (int c = 0; c < C; ++c) {
                    float m = -INFINITY;
                    for (int a = 0; a < kh; ++a) {
                        const int ih = oh * sh - ph + a * dh;
                        if (ih < 0 || ih >= H) continue;
                        for (int b = 0; b < kw; ++b) {
                            const int iw = ow * sw - pw + b * dw;
                            if (iw < 0 || iw >= W) continue;
                            const float v = x[(((size_t)n * H + ih) * W + iw) * C + c];
                            if (v > m) m = v;
                        }
                    }
                    y[(((size_t)n * Ho + oh) * Wo + ow) * C + c] = m;
                }
}

/*
 * Row-wise local operator (Sec. IV-A, Eq. 1 of the paper): Y = X * W^T, every row of X multiplied by the same
 * parameter matrix W, so a block of rows of Y depends on the same block of rows of X and on nothing else.
 * x: [M][K], w: [Cout][K], y: [M][Cout], all row-major; rows [r_lo, r_hi) of y are computed, the others left alone.
 * Accumulation in double over k ascending; epilogue as for the convolution (res has y's shape).
 */
void lop_oracle_linear(const float *x, long long M, int K, const float *w, int Cout,
                       const float *scale, const float *shift, const float *res, int res_pos, int act,
                       int round_bf16, long long r_lo, long long r_hi, float *y)
{
    if (r_lo < 0) r_lo = 0;
    if (r_hi > M) r_hi = M;
#pragma omp parallel for schedule(dynamic, 16)
    for (long long r = r_lo; r < r_hi; ++r)
        for (int co = 0; co < Cout; ++co) {
            double acc = 0.0;
            for (int k = 0; k < K; ++k) acc += (double)x[(size_t)r * K + k] * (double)w[(size_t)co * K + k];
            const size_t o = (size_t)r * Cout + co;
            float t = (float)acc;
            t = (scale ? scale[co] : 1.0f) * t + (shift ? shift[co] : 0.0f);
            if (res && res_pos == 1) t += res[o];
            t = activate(t, act);
            if (res && res_pos == 2) t += res[o];
            y[o] = round_bf16 ? lop_oracle_bf16_rne(t) : t;
        }
}

/*
 * Depth-wise convolution, a block-wise local operator like the convolution (Sec. IV-A): every channel is filtered by
 * its own kh x kw kernel,  y[n,oh,ow,c] = epilogue( sum_{a,b} x[n, oh*sh-ph+a*dh, ow*sw-pw+b*dw, c] * w[c,a,b] ),
 * taps outside the input contribute zero.  w: [C][kh][kw].  Accumulation in double over (a, b); epilogue as above.
 */
void lop_oracle_dwconv2d(const float *x, int N, int H, int W, int C, const float *w, int kh, int kw, int sh, int sw,
                         int ph, int pw, int dh, int dw, const float *scale, const float *shift,
                         const float *res, int res_pos, int act, int round_bf16, int oh_lo, int oh_hi, float *y)
{
    const int Ho = (H + 2 * ph - dh * (kh - 1) - 1) / sh + 1;
    const int Wo = (W + 2 * pw - dw * (kw - 1) - 1) / sw + 1;
    if (oh_lo < 0) oh_lo = 0;
    if (oh_hi > Ho) oh_hi = Ho;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int n = 0; n < N; ++n)
        for (int oh = oh_lo; oh < oh_hi; ++oh)
            for (int ow = 0; ow < Wo; ++ow)
                for (int c = 0; c < C; ++c) {
                    double acc = 0.0;
                    for (int a = 0; a < kh; ++a) {
                        const int ih = oh * sh - ph + a * dh;
                        if (ih < 0 || ih >= H) continue;
                        for (int b = 0; b < kw; ++b) {
                            const int iw = ow * sw - pw + b * dw;
                            if (iw < 0 || iw >= W) continue;
                            acc += (double)x[(((size_t)n * H + ih) * W + iw) * C + c] * (double)w[((size_t)c * kh + a) * kw + b];
                        }
                    }
                    const size_t o = (((size_t)n * Ho + oh) * Wo + ow) * C + c;
                    float t = (float)acc;
                    t = (scale ? scale[c] : 1.0f) * t + (shift ? shift[c] : 0.0f);
                    if (res && res_pos == 1) t += res[o];
                    t = activate(t, act);
                    if (res && res_pos == 2) t += res[o];
                    y[o] = round_bf16 ? lop_oracle_bf16_rne(t) : t;
                }
}

/*
 * Layer normalisation over the channels of every pixel (an element-wise-per-row local operator in the sense of
 * Sec. IV-A: a row of the [pixels][C] matrix depends on that row alone):
 *   y[r][c] = gamma[c] * (x[r][c] - mean_r) / sqrt(var_r + eps) + beta[c],  var_r the biased variance.
 * Mean and variance in double; gamma / beta may be NULL (1 / 0).  Rows [r_lo, r_hi) of y are computed.
 */
void lop_oracle_layernorm(const float *x, long long M, int C, const float *gamma, const float *beta, float eps,
                          int round_bf16, long long r_lo, long long r_hi, float *y)
{
    if (r_lo < 0) r_lo = 0;
    if (r_hi > M) r_hi = M;
#pragma omp parallel for schedule(dynamic, 16)
    for (long long r = r_lo; r < r_hi; ++r) {
        const float *xr = x + (size_t)r * C;
        double mean = 0.0, var = 0.0;
        for (int c = 0; c < C; ++c) mean += xr[c];
        mean /= C;
        for (int c = 0; c < C; ++c) var += ((double)xr[c] - mean) * ((double)xr[c] - mean);
        var /= C;
        const double rstd = 1.0 / sqrt(var + (double)eps);
        for (int c = 0; c < C; ++c) {
            float t = (float)(((double)xr[c] - mean) * rstd);
            t = (gamma ? gamma[c] : 1.0f) * t + (beta ? beta[c] : 0.0f);
            y[(size_t)r * C + c] = round_bf16 ? lop_oracle_bf16_rne(t) : t;
        }
    }
}

/* Channel concatenation: y[r] = (a[r][0..Ca), b[r][0..Cb)) for the rows [r_lo, r_hi) of the [pixels][C] matrices. */
void lop_oracle_concat(const float *a, int Ca, const float *b, int Cb, long long M, long long r_lo, long long r_hi, float *y)
{
    if (r_lo < 0) r_lo = 0;
    if (r_hi > M) r_hi = M;
    for (long long r = r_lo; r < r_hi; ++r) {
        memcpy(y + (size_t)r * (Ca + Cb), a + (size_t)r * Ca, sizeof(float) * (size_t)Ca);
        memcpy(y + (size_t)r * (Ca + Cb) + Ca, b + (size_t)r * Cb, sizeof(float) * (size_t)Cb);
    }
}

int lop_oracle_num_threads(void)
{
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}
