/*
 * dc_oracle.c -- TEST INFRASTRUCTURE, not product code.
 *
 * Plain, slow, fp64 CPU statement of what the convolution-merging path of
 * arXiv 2301.12187 computes (Sec. 3 "Preliminary", Eq. 1, App. E.1 "Skip
 * Addition", App. E.2 "Padding Reordering Technique").  Only the tests, the
 * smoke check and the benchmark's CPU-baseline leg may call it.  It shares no
 * source, header, table or helper with the CUDA library.
 *
 * Conventions (the oracle's own):
 *   feature maps   x[n][c][h][w]            (NCHW, row-major, double)
 *   conv kernels   W[o][i][u][v]            (out, in-per-group, row tap, col tap)
 *   forward        y[n,o,Y,X] = b[o] + sum_{i,u,v} W[o,i,u,v] *
 *                               xpad[n, g(o)*Cg+i, Y*s+u-p, X*s+v-p]
 *                  (cross-correlation: no kernel flip; zero outside the image)
 *   H_out = floor((H + 2p - k)/s) + 1
 *
 * Every loop nest below is the definition written out; nothing is blocked,
 * fused or reordered beyond skipping taps that fall on the zero padding.
 */
#include <math.h>
#include <stddef.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int dco_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void dco_set_num_threads(int t)
{
#ifdef _OPENMP
    if (t > 0) omp_set_num_threads(t);
#else
    (void)t;
#endif
}

/* Output extent of one convolution: floor((h + 2p - k)/s) + 1, or 0 when the
 * kernel does not fit. */
int dco_out_extent(int h, int k, int s, int p)
{
    int a = h + 2 * p - k;
    if (a < 0) return 0;
    return a / s + 1;
}

/*
 * BN fusion into the preceding convolution (Sec. 2 "TensorRT"; Sec. 5.1
 * "Evaluation"): y = gamma*(conv(x)+b-mean)/sqrt(var+eps)+beta is the
 * convolution with W~[o,.] = g[o]*W[o,.] and b~[o] = beta[o]+(b[o]-mean[o])*g[o],
 * g[o] = gamma[o]/sqrt(var[o]+eps).  `per_out` = weights per output channel.
 * `b` may be NULL (no conv bias).
 */
void dco_fold_bn(const double *W, const double *b, const double *gamma, const double *beta,
                 const double *mean, const double *var, double eps, int c_out, int per_out,
                 double *W_out, double *b_out)
{
    for (int o = 0; o < c_out; ++o) {
        double g = gamma[o] / sqrt(var[o] + eps);
        for (int j = 0; j < per_out; ++j) W_out[(size_t)o * per_out + j] = g * W[(size_t)o * per_out + j];
        b_out[o] = beta[o] + ((b ? b[o] : 0.0) - mean[o]) * g;
    }
}

/*
 * Eval-mode batch normalisation applied literally to a feature map (the
 * operation dco_fold_bn is checked against): per channel
 * y = gamma*(x-mean)/sqrt(var+eps)+beta, in place.
 */
void dco_batchnorm(double *x, int n, int c, int hw, const double *gamma, const double *beta,
                   const double *mean, const double *var, double eps)
{
    for (int in = 0; in < n; ++in)
        for (int ic = 0; ic < c; ++ic) {
            double inv = 1.0 / sqrt(var[ic] + eps);
            double *p = x + ((size_t)in * c + ic) * hw;
            for (int j = 0; j < hw; ++j) p[j] = gamma[ic] * (p[j] - mean[ic]) * inv + beta[ic];
        }
}

/*
 * Direct convolution, the forward definition above (Sec. 3: f_theta).
 * groups == 1 (dense) or any divisor of c_in and c_out (depthwise when
 * groups == c_in == c_out).  bias may be NULL.  Zero padding p on every side.
 * y must hold n*c_out*ho*wo doubles.
 */
void dco_conv_direct(const double *x, int n, int c_in, int h, int w, const double *W,
                     const double *bias, int c_out, int k, int s, int p, int groups, double *y)
{
    const int ho = dco_out_extent(h, k, s, p), wo = dco_out_extent(w, k, s, p);
    const int cg_in = c_in / groups, cg_out = c_out / groups;
    if (ho <= 0 || wo <= 0) return;
#pragma omp parallel for collapse(2) schedule(static)
    for (int in = 0; in < n; ++in)
        for (int o = 0; o < c_out; ++o) {
            double *yo = y + ((size_t)in * c_out + o) * ho * wo;
            const double b0 = bias ? bias[o] : 0.0;
            for (int j = 0; j < ho * wo; ++j) yo[j] = b0;
            const int g = o / cg_out;
            for (int i = 0; i < cg_in; ++i) {
                const double *xi = x + ((size_t)in * c_in + (size_t)g * cg_in + i) * h * w;
                for (int u = 0; u < k; ++u)
                    for (int v = 0; v < k; ++v) {
                        const double wt = W[(((size_t)o * cg_in + i) * k + u) * k + v];
                        for (int Y = 0; Y < ho; ++Y) {
                            const int yy = Y * s + u - p;
                            if (yy < 0 || yy >= h) continue; /* row lies in the zero padding */
                            for (int X = 0; X < wo; ++X) {
                                const int xx = X * s + v - p;
                                if (xx < 0 || xx >= w) continue; /* column lies in the zero padding */
                                yo[(size_t)Y * wo + X] += wt * xi[(size_t)yy * w + xx];
                            }
                        }
                    }
            }
        }
}

/* Depthwise kernel Wdw[c][1][k][k] written as the dense kernel it stands for:
 * W[o][i][u][v] = delta(o,i) * Wdw[o][u][v]. */
void dco_lift_depthwise(const double *Wdw, int c, int k, double *W)
{
    memset(W, 0, sizeof(double) * (size_t)c * c * k * k);
    for (int o = 0; o < c; ++o)
        for (int u = 0; u < k; ++u)
            for (int v = 0; v < k; ++v)
                W[(((size_t)o * c + o) * k + u) * k + v] = Wdw[((size_t)o * k + u) * k + v];
}

/*
 * Merging two consecutive convolutions (Sec. 3: f_{theta2}(f_{theta1}(X)) =
 * f_{theta2 (*) theta1}(X); Eq. 1).  Substituting layer 1 (kernel k1, stride
 * s1) into layer 2 (kernel k2) gives, with u' = u1 + s1*u2 and v' = v1 + s1*v2,
 *   W'[o,i,u',v'] = sum_c sum_{u1+s1*u2=u'} sum_{v1+s1*v2=v'} W2[o,c,u2,v2]*W1[c,i,u1,v1]
 *   k' = k1 + (k2-1)*s1.
 * Both operands dense: W1[c1][c0][k1][k1], W2[c2][c1][k2][k2]; out[c2][c0][k'][k'].
 */
void dco_merge_pair(const double *W1, int c0, int c1, int k1, int s1, const double *W2, int c2,
                    int k2, double *out)
{
    const int kk = k1 + (k2 - 1) * s1;
    memset(out, 0, sizeof(double) * (size_t)c2 * c0 * kk * kk);
#pragma omp parallel for schedule(static)
    for (int o = 0; o < c2; ++o)
        for (int i = 0; i < c0; ++i)
            for (int c = 0; c < c1; ++c)
                for (int u2 = 0; u2 < k2; ++u2)
                    for (int v2 = 0; v2 < k2; ++v2)
                        for (int u1 = 0; u1 < k1; ++u1)
                            for (int v1 = 0; v1 < k1; ++v1) {
                                const int up = u1 + s1 * u2, vp = v1 + s1 * v2;
                                out[(((size_t)o * c0 + i) * kk + up) * kk + vp] +=
                                    W2[(((size_t)o * c1 + c) * k2 + u2) * k2 + v2] *
                                    W1[(((size_t)c * c0 + i) * k1 + u1) * k1 + v1];
                            }
}

/* Bias of the merged pair: layer 2 sees the constant b1[c] on every tap, so
 * b'[o] = b2[o] + sum_c (sum_{u2,v2} W2[o,c,u2,v2]) * b1[c]. */
void dco_merge_bias(const double *b1, int c1, const double *W2, const double *b2, int c2, int k2,
                    double *out)
{
    for (int o = 0; o < c2; ++o) {
        double acc = b2 ? b2[o] : 0.0;
        for (int c = 0; c < c1; ++c) {
            double ws = 0.0;
            for (int t = 0; t < k2 * k2; ++t) ws += W2[((size_t)o * c1 + c) * k2 * k2 + t];
            acc += ws * (b1 ? b1[c] : 0.0);
        }
        out[o] = acc;
    }
}
