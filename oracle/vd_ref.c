/*
 * vd_ref — the oracle: a plain, slow CPU restatement of the operators of the convolutional
 * frame decoder (latent in, frame out).  TEST INFRASTRUCTURE ONLY: nothing on the product
 * path may call, link or load this file; it shares no code with the CUDA library.
 *
 * The paper names the operator set (Conv2d, GroupNorm, SiLU; Section IV-A, text before Eq. 8)
 * and the decoder's fused chain Upsample -> Conv2d -> GroupNorm -> SiLU (Section IV-B.1, Eq. 9);
 * it states that fusion changes data movement only, so the result is the plain definition of
 * each operator.  Each function below is that definition written out as direct loops.
 *
 * Conventions: every tensor is fp32, NCHW, contiguous, host memory.  Every reduction (a
 * convolution's dot product, GroupNorm's mean and variance, softmax's row sum, attention's
 * weighted sum) accumulates in fp64 and is rounded to fp32 once when stored, so that the order
 * of summation is immaterial at fp32 resolution.  OpenMP only splits independent outputs
 * between threads; each output element is reduced by one thread in a fixed order, so results
 * do not depend on the thread count.
 *
 * Return value: 0 on success, -1 on an invalid argument.
 */
#include <math.h>
#include <stddef.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define VD_REF_API __attribute__((visibility("default")))

VD_REF_API int vd_ref_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

VD_REF_API void vd_ref_set_num_threads(int n) {
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/*
 * Conv2d (operator set of Section IV-A; second link of the chain of Section IV-B.1).
 * Cross-correlation, stride 1, zero padding ksize/2, ksize in {1,3}:
 *   y[n,o,i,j] = b[o] + sum_{c,ky,kx} w[o,c,ky,kx] * x[n,c,i+ky-p,j+kx-p],   x = 0 outside the image.
 * w is [Cout,Cin,ksize,ksize]; b may be NULL (no bias).
 */
VD_REF_API int vd_ref_conv2d(const float* x, const float* w, const float* b, float* y,
                             int N, int Cin, int H, int W, int Cout, int ksize) {
    if (!x || !w || !y || N < 0 || Cin <= 0 || Cout <= 0 || H <= 0 || W <= 0) return -1;
    if (ksize != 1 && ksize != 3) return -1;
    const int p = ksize / 2;
    const long rows = (long)N * Cout * H;
#pragma omp parallel
    {
        double* acc = (double*)malloc(sizeof(double) * (size_t)W);
#pragma omp for schedule(dynamic, 4)
        for (long r = 0; r < rows; ++r) {
            const int i = (int)(r % H);
            const int o = (int)((r / H) % Cout);
            const int n = (int)(r / ((long)H * Cout));
            const double bias = b ? (double)b[o] : 0.0;
            for (int j = 0; j < W; ++j) acc[j] = bias;
            for (int c = 0; c < Cin; ++c) {
                const float* xc = x + ((size_t)n * Cin + c) * H * W;
                const float* wc = w + ((size_t)o * Cin + c) * ksize * ksize;
                for (int ky = 0; ky < ksize; ++ky) {
                    const int ii = i + ky - p;
                    if (ii < 0 || ii >= H) continue;          /* zero padding: the row adds nothing */
                    const float* xr = xc + (size_t)ii * W;
                    for (int kx = 0; kx < ksize; ++kx) {
                        const double wv = (double)wc[ky * ksize + kx];
                        const int d = kx - p;
                        const int j0 = d < 0 ? -d : 0;            /* first j with 0 <= j+d */
                        const int j1 = d > 0 ? W - d : W;         /* one past the last j with j+d < W */
                        for (int j = j0; j < j1; ++j) acc[j] += wv * (double)xr[j + d];
                    }
                }
            }
            float* yr = y + (((size_t)n * Cout + o) * H + i) * W;
            for (int j = 0; j < W; ++j) yr[j] = (float)acc[j];
        }
        free(acc);
    }
    return 0;
}

/*
 * GroupNorm (operator set of Section IV-A; third link of the chain of Section IV-B.1).
 * Per sample n and group g of C/G contiguous channels, over the (C/G)*H*W values of the group:
 *   pass 1: mu = mean(x);   pass 2: var = mean((x-mu)^2)  (biased);
 *   y = (x-mu)/sqrt(var+eps) * gamma[c] + beta[c].
 * gamma/beta may be NULL (treated as 1 and 0).  mean_out/rstd_out, when non-NULL, receive
 * the [N,G] statistics (mu and 1/sqrt(var+eps)) in fp64.
 */
VD_REF_API int vd_ref_groupnorm(const float* x, const float* gamma, const float* beta, float* y,
                                int N, int C, int H, int W, int G, float eps,
                                double* mean_out, double* rstd_out) {
    if (!x || !y || N < 0 || C <= 0 || H <= 0 || W <= 0 || G <= 0 || C % G != 0) return -1;
    const int cg = C / G;
    const size_t hw = (size_t)H * W;
    const size_t cnt = (size_t)cg * hw;
#pragma omp parallel for schedule(dynamic, 1)
    for (long ng = 0; ng < (long)N * G; ++ng) {
        const int g = (int)(ng % G);
        const int n = (int)(ng / G);
        const float* xg = x + ((size_t)n * C + (size_t)g * cg) * hw;
        float* yg = y + ((size_t)n * C + (size_t)g * cg) * hw;
        double s = 0.0;
        for (size_t t = 0; t < cnt; ++t) s += (double)xg[t];
        const double mu = s / (double)cnt;
        double m2 = 0.0;
        for (size_t t = 0; t < cnt; ++t) {
            const double d = (double)xg[t] - mu;
            m2 += d * d;
        }
        const double var = m2 / (double)cnt;
        const double rstd = 1.0 / sqrt(var + (double)eps);
        if (mean_out) mean_out[ng] = mu;
        if (rstd_out) rstd_out[ng] = rstd;
        for (int cc = 0; cc < cg; ++cc) {
            const int c = g * cg + cc;
            const double ga = gamma ? (double)gamma[c] : 1.0;
            const double be = beta ? (double)beta[c] : 0.0;
            for (size_t t = 0; t < hw; ++t)
                yg[cc * hw + t] = (float)(((double)xg[cc * hw + t] - mu) * rstd * ga + be);
        }
    }
    return 0;
}

/* SiLU (last link of the chain of Section IV-B.1): y = x / (1 + exp(-x)). */
VD_REF_API int vd_ref_silu(const float* x, float* y, long count) {
    if (!x || !y || count < 0) return -1;
#pragma omp parallel for
    for (long t = 0; t < count; ++t) {
        const double v = (double)x[t];
        y[t] = (float)(v / (1.0 + exp(-v)));
    }
    return 0;
}

/* Nearest-neighbour 2x upsample (first link of the chain of Section IV-B.1):
 * y[n,c,i,j] = x[n,c,i>>1,j>>1];  y is [N,C,2H,2W]. */
VD_REF_API int vd_ref_upsample2x(const float* x, float* y, int N, int C, int H, int W) {
    if (!x || !y || N < 0 || C <= 0 || H <= 0 || W <= 0) return -1;
    const int H2 = 2 * H, W2 = 2 * W;
#pragma omp parallel for
    for (long nc = 0; nc < (long)N * C; ++nc) {
        const float* xp = x + (size_t)nc * H * W;
        float* yp = y + (size_t)nc * H2 * W2;
        for (int i = 0; i < H2; ++i)
            for (int j = 0; j < W2; ++j) yp[(size_t)i * W2 + j] = xp[(size_t)(i >> 1) * W + (j >> 1)];
    }
    return 0;
}

/* Elementwise sum, the skip connection of a residual block: y = a + b (fp32 add, one rounding). */
VD_REF_API int vd_ref_add(const float* a, const float* b, float* y, long count) {
    if (!a || !b || !y || count < 0) return -1;
#pragma omp parallel for
    for (long t = 0; t < count; ++t) y[t] = a[t] + b[t];
    return 0;
}

/*
 * Single-head softmax attention over T = H*W tokens of C channels (the decoder's mid-block
 * attention; the paper does not describe it, the workload definition does).  q, k, v, o are
 * [N,C,T] (an NCHW map with its pixels flattened row-major, token t = i*W + j):
 *   s[t,u] = scale * sum_c q[c,t]*k[c,u];   p[t,:] = softmax_u(s[t,:]) with the row maximum
 *   subtracted first;   o[c,t] = sum_u p[t,u] * v[c,u].
 * p_out, when non-NULL, receives the [N,T,T] probabilities in fp64 (small T only).
 */
VD_REF_API int vd_ref_attention_core(const float* q, const float* k, const float* v, float* o,
                                     int N, int C, int T, float scale, double* p_out) {
    if (!q || !k || !v || !o || N < 0 || C <= 0 || T <= 0) return -1;
    for (int n = 0; n < N; ++n) {
        const float* qn = q + (size_t)n * C * T;
        const float* kn = k + (size_t)n * C * T;
        const float* vn = v + (size_t)n * C * T;
        float* on = o + (size_t)n * C * T;
#pragma omp parallel
        {
            double* s = (double*)malloc(sizeof(double) * (size_t)T);
#pragma omp for schedule(dynamic, 8)
            for (int t = 0; t < T; ++t) {
                for (int u = 0; u < T; ++u) s[u] = 0.0;
                for (int c = 0; c < C; ++c) {
                    const double qv = (double)qn[(size_t)c * T + t];
                    const float* kc = kn + (size_t)c * T;
                    for (int u = 0; u < T; ++u) s[u] += qv * (double)kc[u];
                }
                double mx = -INFINITY;
                for (int u = 0; u < T; ++u) {
                    s[u] *= (double)scale;
                    if (s[u] > mx) mx = s[u];
                }
                double den = 0.0;
                for (int u = 0; u < T; ++u) {
                    s[u] = exp(s[u] - mx);
                    den += s[u];
                }
                for (int u = 0; u < T; ++u) s[u] /= den;
                if (p_out) memcpy(p_out + ((size_t)n * T + t) * T, s, sizeof(double) * (size_t)T);
                for (int c = 0; c < C; ++c) {
                    const float* vc = vn + (size_t)c * T;
                    double a = 0.0;
                    for (int u = 0; u < T; ++u) a += s[u] * (double)vc[u];
                    on[(size_t)c * T + t] = (float)a;
                }
            }
            free(s);
        }
    }
    return 0;
}

/*
 * Latent extrapolation, the hit branch of Algorithm 2 / Eq. 10: the next latent is the
 * previous one advanced along the last motion vector, z = z_prev + lambda * v_prev,
 * and the motion vector kept for the next step is v = z - z_prev.
 */
VD_REF_API int vd_ref_extrapolate(const float* z_prev, const float* v_prev, float lambda, float* z,
                                  float* v, long count) {
    if (!z_prev || !v_prev || !z || count < 0) return -1;
    for (long t = 0; t < count; ++t) {
        const double zn = (double)z_prev[t] + (double)lambda * (double)v_prev[t];
        z[t] = (float)zn;
        if (v) v[t] = (float)((double)z[t] - (double)z_prev[t]);
    }
    return 0;
}

/*
 * Display packing of a decoded frame for transport to the host (the output side of the decode step of
 * Algorithm 1, Q_out.push(I_t); Table II lists the frame transport as a component of its own).  The
 * paper does not print the mapping; the reading taken is the usual one for a decoder whose frames live in
 * [-1, 1]: q = round(clamp(x * 0.5 + 0.5, 0, 1) * 255), channels interleaved per pixel (NHWC), 8 bits.
 * A floating-point value decides an integer here, so the arithmetic is fixed to what the kernels do, in
 * fp32: t = fma(x, 127.5, 127.5) (one rounding), clamped to [0, 255], rounded to nearest with ties to
 * even.  NaN packs to 0.
 *   x: [N,C,H,W] fp32     q: [N,H,W,C] uint8
 */
VD_REF_API int vd_ref_pack_u8(const float* x, unsigned char* q, int N, int C, int H, int W) {
    if (!x || !q || N < 0 || C <= 0 || H <= 0 || W <= 0) return -1;
    for (int n = 0; n < N; ++n)
        for (int c = 0; c < C; ++c)
            for (int i = 0; i < H; ++i)
                for (int j = 0; j < W; ++j) {
                    float t = fmaf(x[(((size_t)n * C + c) * H + i) * W + j], 127.5f, 127.5f);
                    if (!(t > 0.0f)) t = 0.0f;              /* also NaN */
                    if (t > 255.0f) t = 255.0f;
                    q[(((size_t)n * H + i) * W + j) * C + c] = (unsigned char)rintf(t);
                }
    return 0;
}
