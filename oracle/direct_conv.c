/*
 * ORACLE — test infrastructure only.  Nothing in the product path may call,
 * link or import this file; only tests, the smoke check and the benchmark's
 * CPU-baseline leg do.
 *
 * 2-D convolution (cross-correlation, no kernel flip) by its plain definition,
 * the "sliding window" scheme of the paper's Section 3.2 (scheme pool, item 1-3)
 * and the quantity that the Winograd identity of Eq. 6 must reproduce:
 *
 *   y[n,co,oh,ow] = act( bias[co] +
 *        sum_{ci in group(co)} sum_{a<k} sum_{b<k}
 *            w[co,ci,a,b] * xpad[n, ci, oh*stride - pad + a*dil, ow*stride - pad + b*dil] )
 *
 * xpad is x inside the image and 0 outside.  OH = floor((H + 2 pad - dil (k-1) - 1)/stride) + 1.
 * Inputs are fp32 (the precision the paper's engine computes in), promoted to
 * fp64; every product and sum is fp64; the result is returned in fp64.
 * No blocking, no reordering: seven nested loops in the order of the formula.
 *
 * Layouts: x [N][Cin][H][W], w [Cout][Cin/groups][k][k], bias [Cout] or NULL,
 * y [N][Cout][OH][OW]; all dense row-major host arrays.
 */
#include <stddef.h>

#ifdef _OPENMP
#include <omp.h>
#endif

static int out_extent(int in, int k, int stride, int pad, int dil)
{
    if (stride <= 0) return 0;
    int span = in + 2 * pad - dil * (k - 1) - 1;
    if (span < 0) return 0;
    return span / stride + 1;
}

int oracle_conv_out_extent(int in, int k, int stride, int pad, int dil)
{
    return out_extent(in, k, stride, pad, dil);
}

int oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* One output element, straight from the definition. */
static double conv_point(const float* x, const float* w, const float* bias,
                         int Cin, int Cout, int H, int W, int k,
                         int stride, int pad, int dil, int groups, int relu,
                         int n, int co, int oh, int ow)
{
    const int cpg = Cin / groups;          /* input channels per group  */
    const int opg = Cout / groups;         /* output channels per group */
    const int g = co / opg;
    double acc = bias ? (double)bias[co] : 0.0;
    for (int c = 0; c < cpg; ++c) {
        const int ci = g * cpg + c;
        for (int a = 0; a < k; ++a) {
            const int ih = oh * stride - pad + a * dil;
            if (ih < 0 || ih >= H) continue;
            for (int b = 0; b < k; ++b) {
                const int iw = ow * stride - pad + b * dil;
                if (iw < 0 || iw >= W) continue;
                const double xv = (double)x[(((size_t)n * Cin + ci) * H + ih) * W + iw];
                const double wv = (double)w[(((size_t)co * cpg + c) * k + a) * k + b];
                acc += wv * xv;
            }
        }
    }
    if (relu && acc < 0.0) acc = 0.0;
    return acc;
}

/* Full output tensor.  Returns 0, or -1 on an argument the definition has no meaning for. */
int oracle_direct_conv_f64(const float* x, const float* w, const float* bias, double* y,
                           int N, int Cin, int Cout, int H, int W, int k,
                           int stride, int pad, int dil, int groups, int relu)
{
    if (N < 0 || Cin <= 0 || Cout <= 0 || H <= 0 || W <= 0 || k <= 0 || stride <= 0 ||
        pad < 0 || dil <= 0 || groups <= 0 || Cin % groups || Cout % groups)
        return -1;
    const int OH = out_extent(H, k, stride, pad, dil);
    const int OW = out_extent(W, k, stride, pad, dil);
    const long long planes = (long long)N * Cout;
#pragma omp parallel for schedule(dynamic, 1)
    for (long long p = 0; p < planes; ++p) {
        const int n = (int)(p / Cout), co = (int)(p % Cout);
        for (int oh = 0; oh < OH; ++oh)
            for (int ow = 0; ow < OW; ++ow)
                y[((size_t)p * OH + oh) * OW + ow] =
                    conv_point(x, w, bias, Cin, Cout, H, W, k, stride, pad, dil, groups, relu,
                               n, co, oh, ow);
    }
    return 0;
}

/* Selected images only: images[i] (i < n_images) are computed in full into
 * y_out[i][Cout][OH][OW].  Used when the whole batch is too much CPU work. */
int oracle_direct_conv_f64_images(const float* x, const float* w, const float* bias, double* y_out,
                                  const int* images, int n_images,
                                  int N, int Cin, int Cout, int H, int W, int k,
                                  int stride, int pad, int dil, int groups, int relu)
{
    if (N < 0 || Cin <= 0 || Cout <= 0 || H <= 0 || W <= 0 || k <= 0 || stride <= 0 ||
        pad < 0 || dil <= 0 || groups <= 0 || Cin % groups || Cout % groups)
        return -1;
    for (int i = 0; i < n_images; ++i)
        if (images[i] < 0 || images[i] >= N) return -1;
    const int OH = out_extent(H, k, stride, pad, dil);
    const int OW = out_extent(W, k, stride, pad, dil);
    const long long planes = (long long)n_images * Cout;
#pragma omp parallel for schedule(dynamic, 1)
    for (long long p = 0; p < planes; ++p) {
        const int n = images[p / Cout], co = (int)(p % Cout);
        for (int oh = 0; oh < OH; ++oh)
            for (int ow = 0; ow < OW; ++ow)
                y_out[((size_t)p * OH + oh) * OW + ow] =
                    conv_point(x, w, bias, Cin, Cout, H, W, k, stride, pad, dil, groups, relu,
                               n, co, oh, ow);
    }
    return 0;
}

/* Selected output elements only: flat[i] indexes y as [N][Cout][OH][OW]. */
int oracle_direct_conv_f64_at(const float* x, const float* w, const float* bias,
                              const long long* flat, long long n_flat, double* out,
                              int N, int Cin, int Cout, int H, int W, int k,
                              int stride, int pad, int dil, int groups, int relu)
{
    if (N < 0 || Cin <= 0 || Cout <= 0 || H <= 0 || W <= 0 || k <= 0 || stride <= 0 ||
        pad < 0 || dil <= 0 || groups <= 0 || Cin % groups || Cout % groups)
        return -1;
    const int OH = out_extent(H, k, stride, pad, dil);
    const int OW = out_extent(W, k, stride, pad, dil);
    const long long total = (long long)N * Cout * OH * OW;
    for (long long i = 0; i < n_flat; ++i)
        if (flat[i] < 0 || flat[i] >= total) return -1;
#pragma omp parallel for schedule(static)
    for (long long i = 0; i < n_flat; ++i) {
        long long f = flat[i];
        const int ow = (int)(f % OW); f /= OW;
        const int oh = (int)(f % OH); f /= OH;
        const int co = (int)(f % Cout); f /= Cout;
        const int n = (int)f;
        out[i] = conv_point(x, w, bias, Cin, Cout, H, W, k, stride, pad, dil, groups, relu,
                            n, co, oh, ow);
    }
    return 0;
}

/*
 * Rectangular kernels (the paper's Section 4.2 names the 1 x 7 and 7 x 1 convolutions of Inception-v3):
 * the same definition with its own kernel height and width and its own padding per axis, stride 1,
 * no dilation, one group:
 *
 *   y[n,co,oh,ow] = act( bias[co] + sum_ci sum_{a<kh} sum_{b<kw}
 *                        w[co,ci,a,b] * xpad[n, ci, oh - pad_h + a, ow - pad_w + b] )
 *   OH = H + 2 pad_h - kh + 1,  OW = W + 2 pad_w - kw + 1;   w is [Cout][Cin][kh][kw].
 */
int oracle_direct_conv_rect_f64(const float* x, const float* w, const float* bias, double* y,
                                int N, int Cin, int Cout, int H, int W, int kh, int kw,
                                int pad_h, int pad_w, int relu)
{
    if (N < 0 || Cin <= 0 || Cout <= 0 || H <= 0 || W <= 0 || kh <= 0 || kw <= 0 || pad_h < 0 || pad_w < 0)
        return -1;
    const int OH = H + 2 * pad_h - kh + 1, OW = W + 2 * pad_w - kw + 1;
    if (OH <= 0 || OW <= 0) return -1;
    const long long planes = (long long)N * Cout;
#pragma omp parallel for schedule(dynamic, 1)
    for (long long p = 0; p < planes; ++p) {
        const int n = (int)(p / Cout), co = (int)(p % Cout);
        for (int oh = 0; oh < OH; ++oh)
            for (int ow = 0; ow < OW; ++ow) {
                double acc = bias ? (double)bias[co] : 0.0;
                for (int ci = 0; ci < Cin; ++ci)
                    for (int a = 0; a < kh; ++a) {
                        const int ih = oh - pad_h + a;
                        if (ih < 0 || ih >= H) continue;
                        for (int b = 0; b < kw; ++b) {
                            const int iw = ow - pad_w + b;
                            if (iw < 0 || iw >= W) continue;
                            acc += (double)w[(((size_t)co * Cin + ci) * kh + a) * kw + b] *
                                   (double)x[(((size_t)n * Cin + ci) * H + ih) * W + iw];
                        }
                    }
                if (relu && acc < 0.0) acc = 0.0;
                y[((size_t)p * OH + oh) * OW + ow] = acc;
            }
    }
    return 0;
}
