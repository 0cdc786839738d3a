/*
 * CPU oracle for column-wise N:M pruning and the sparse convolution it feeds.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain restatement of what the
 * method computes; it shares nothing with the CUDA library (no headers, helpers,
 * tables or constants) and the product path never calls it.  Only the tests, the
 * smoke check and the CPU-baseline leg of the benchmark may load it.
 *
 * What the paper fixes and what is a stated reading:
 *   - Weight matrix [C_out, K], K = Kh*Kw*C_in, column k = (kh*Kw + kw)*C_in + c
 *     (OHWI kernel layout, Fig. 4 caption).
 *   - Rows are cut into tiles of T output channels; inside a tile one column (its
 *     T weights) is the pruning unit, scored by its L1 norm (Sec. 3.1).
 *   - In every group of M consecutive columns N units are RETAINED (Sec. 2.1,
 *     Sec. 3.1: N = (1 - sparsity) * M; Algorithm 1 takes N as the retained count).
 *   - Compressed form: values W[T, kept] per tile plus the index array Idx[kept]
 *     holding the surviving column positions (Sec. 2.1, Algorithm 1 inputs).
 *   - The product is the plain matrix product on the retained columns
 *     (Algorithm 1, read with W[t, n] and C + t*V), i.e. the dense convolution
 *     with the pruned columns set to zero.
 *   Readings where the paper is silent: scores are summed in fp64 over the tile's
 *   rows in ascending row order; a score that is NaN ranks as +infinity; equal scores keep the
 *   lower column; a tail group of
 *   m' < M columns keeps min(N, m'); a tail tile sums over the rows that exist;
 *   bias is added before an optional ReLU; out-of-range taps read zero.
 *
 * Pins (tests, CPU only): textbook row-wise N:M for T = 1; exhaustive subset search
 * on tiny inputs; hand-worked examples; count/order invariants; N = M identity;
 * zero-expansion round trip; conv against a brute-force 7-loop dense conv, against a
 * library fp64 conv, 1x1 against a plain matrix product, hand-worked 3x3 cases; the
 * shortcut-adding form against the plain form (zero residual: identical; integer inputs:
 * exact sum; a library fp64 conv plus the residual).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* Number of columns the pruner retains out of k: N per full group of M, and
 * min(N, m') for a tail group of m' columns (Sec. 2.1: N retained per M). */
int nm_oracle_kept_count(int k, int n_keep, int m_group)
{
    int full = k / m_group, tail = k % m_group;
    return full * n_keep + (tail < n_keep ? tail : n_keep);
}

int nm_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * Column-wise N:M pruning at tile level (Sec. 3.1).
 *   w        [c_out][k] fp32, row-major (k flattened OHWI)
 *   values   [c_out][kk] fp32 out: values[o][j] = w[o][indices[o / tile_t][j]], copied bit for bit
 *   indices  [n_tiles][kk] uint16 out: retained column positions, ascending
 * Returns kk, or -1 on a bad argument.
 */
int nm_oracle_prune(const float* w, int c_out, int k, int n_keep, int m_group, int tile_t,
                    float* values, uint16_t* indices)
{
    if (!w || !values || !indices || c_out < 1 || k < 1 || k > 65535 || n_keep < 1 ||
        m_group < n_keep || tile_t < 1)
        return -1;
    const int kk = nm_oracle_kept_count(k, n_keep, m_group);
    const int n_tiles = (c_out + tile_t - 1) / tile_t;
    double* score = (double*)malloc(sizeof(double) * (size_t)m_group);
    char* keep = (char*)malloc((size_t)m_group);
    if (!score || !keep) { free(score); free(keep); return -1; }

    for (int r = 0; r < n_tiles; ++r) {
        const int row0 = r * tile_t;
        const int row1 = row0 + tile_t < c_out ? row0 + tile_t : c_out;
        int j = 0;
        for (int g0 = 0; g0 < k; g0 += m_group) {
            const int gsz = g0 + m_group <= k ? m_group : k - g0;
            const int take = n_keep < gsz ? n_keep : gsz;
            /* L1 norm of each column of the tile */
            for (int i = 0; i < gsz; ++i) {
                double s = 0.0;
                for (int o = row0; o < row1; ++o) s += fabs((double)w[(size_t)o * k + g0 + i]);
                /* a NaN score (a NaN weight) would make the comparisons below depend on position;
                 * it ranks as +infinity, which keeps the order total (ties by column as usual) */
                score[i] = isnan(s) ? (double)INFINITY : s;
                keep[i] = 0;
            }
            /* retain the `take` largest; a later column wins only if strictly larger */
            for (int n = 0; n < take; ++n) {
                int best = -1;
                for (int i = 0; i < gsz; ++i) {
                    if (keep[i]) continue;
                    if (best < 0 || score[i] > score[best]) best = i;
                }
                keep[best] = 1;
            }
            for (int i = 0; i < gsz; ++i)
                if (keep[i]) indices[(size_t)r * kk + j++] = (uint16_t)(g0 + i);
        }
        for (int o = row0; o < row1; ++o)
            for (int jj = 0; jj < kk; ++jj)
                values[(size_t)o * kk + jj] = w[(size_t)o * k + indices[(size_t)r * kk + jj]];
    }
    free(score);
    free(keep);
    return kk;
}

/* Zero-expansion of the compressed form back to [c_out][k] (Fig. 1 read backwards). */
int nm_oracle_expand(const float* values, const uint16_t* indices, int c_out, int k, int kk,
                     int tile_t, float* w_out)
{
    if (!values || !indices || !w_out || c_out < 1 || k < 1 || kk < 0 || tile_t < 1) return -1;
    memset(w_out, 0, sizeof(float) * (size_t)c_out * k);
    for (int o = 0; o < c_out; ++o) {
        const uint16_t* idx = indices + (size_t)(o / tile_t) * kk;
        for (int j = 0; j < kk; ++j) w_out[(size_t)o * k + idx[j]] = values[(size_t)o * kk + j];
    }
    return 0;
}

/*
 * Sparse convolution on the compressed weights: Algorithm 1 applied to the
 * patch matrix of Sec. 2.2 without building it.
 *   x [batch][h][w][c_in] fp32 (NHWC), y [batch][ho][wo][c_out] fp32 (NHWC)
 *   y = act(bias[o] + sum_j values[o][j] * x[n][oh*s - p + kh_j*d][ow*s - p + kw_j*d][c_j])
 * with k_j = indices[o / tile_t][j] = (kh_j*Kw + kw_j)*c_in + c_j, products and the
 * running sum in fp64 in ascending j, one rounding to fp32 at the end.
 * Returns 0, or -1 on a bad argument.
 */
int nm_oracle_conv2d(const float* values, const uint16_t* indices, int c_out, int kh, int kw,
                     int c_in, int kk, int tile_t, const float* x, int batch, int h, int w,
                     int stride_h, int stride_w, int pad_h, int pad_w, int dil_h, int dil_w,
                     const float* bias, int relu, float* y)
{
    if (!values || !indices || !x || !y || c_out < 1 || kh < 1 || kw < 1 || c_in < 1 || kk < 0 ||
        tile_t < 1 || batch < 1 || h < 1 || w < 1 || stride_h < 1 || stride_w < 1 || pad_h < 0 ||
        pad_w < 0 || dil_h < 1 || dil_w < 1)
        return -1;
    const int ho = (h + 2 * pad_h - dil_h * (kh - 1) - 1) / stride_h + 1;
    const int wo = (w + 2 * pad_w - dil_w * (kw - 1) - 1) / stride_w + 1;
    if (h + 2 * pad_h - dil_h * (kh - 1) - 1 < 0 || w + 2 * pad_w - dil_w * (kw - 1) - 1 < 0) return -1;

#pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < batch; ++n) {
        for (int oh = 0; oh < ho; ++oh) {
            for (int ow = 0; ow < wo; ++ow) {
                float* yp = y + (((size_t)n * ho + oh) * wo + ow) * c_out;
                for (int o = 0; o < c_out; ++o) {
                    const uint16_t* idx = indices + (size_t)(o / tile_t) * kk;
                    const float* val = values + (size_t)o * kk;
                    double acc = bias ? (double)bias[o] : 0.0;
                    for (int j = 0; j < kk; ++j) {
                        const int kcol = idx[j];
                        const int c = kcol % c_in;
                        const int tap = kcol / c_in;
                        const int ih = oh * stride_h - pad_h + (tap / kw) * dil_h;
                        const int iw = ow * stride_w - pad_w + (tap % kw) * dil_w;
                        if (ih < 0 || ih >= h || iw < 0 || iw >= w) continue;
                        acc += (double)val[j] * (double)x[(((size_t)n * h + ih) * w + iw) * c_in + c];
                    }
                    if (relu && acc < 0.0) acc = 0.0;
                    yp[o] = (float)acc;
                }
            }
        }
    }
    return 0;
}

/*
 * The same convolution followed by the shortcut addition of a residual block: the networks the
 * paper measures end to end (Sec. 4.5, torchvision ResNets) add the block input to the last
 * convolution's output before the ReLU.
 *   y = act(bias[o] + sum_j values[o][j] * x[...] + residual[n][oh][ow][o])
 * residual has the output's shape (NHWC fp32) and may be NULL (then this is nm_oracle_conv2d).
 * Products, the running sum and the shortcut addition in fp64, one rounding to fp32 at the end.
 */
int nm_oracle_conv2d_res(const float* values, const uint16_t* indices, int c_out, int kh, int kw,
                         int c_in, int kk, int tile_t, const float* x, int batch, int h, int w,
                         int stride_h, int stride_w, int pad_h, int pad_w, int dil_h, int dil_w,
                         const float* bias, const float* residual, int relu, float* y)
{
    if (!values || !indices || !x || !y || c_out < 1 || kh < 1 || kw < 1 || c_in < 1 || kk < 0 ||
        tile_t < 1 || batch < 1 || h < 1 || w < 1 || stride_h < 1 || stride_w < 1 || pad_h < 0 ||
        pad_w < 0 || dil_h < 1 || dil_w < 1)
        return -1;
    const int ho = (h + 2 * pad_h - dil_h * (kh - 1) - 1) / stride_h + 1;
    const int wo = (w + 2 * pad_w - dil_w * (kw - 1) - 1) / stride_w + 1;
    if (h + 2 * pad_h - dil_h * (kh - 1) - 1 < 0 || w + 2 * pad_w - dil_w * (kw - 1) - 1 < 0) return -1;

#pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < batch; ++n) {
        for (int oh = 0; oh < ho; ++oh) {
            for (int ow = 0; ow < wo; ++ow) {
                const size_t pix = ((size_t)n * ho + oh) * wo + ow;
                for (int o = 0; o < c_out; ++o) {
                    const uint16_t* idx = indices + (size_t)(o / tile_t) * kk;
                    const float* val = values + (size_t)o * kk;
                    double acc = bias ? (double)bias[o] : 0.0;
                    for (int j = 0; j < kk; ++j) {
                        const int kcol = idx[j];
                        const int c = kcol % c_in;
                        const int tap = kcol / c_in;
                        const int ih = oh * stride_h - pad_h + (tap / kw) * dil_h;
                        const int iw = ow * stride_w - pad_w + (tap % kw) * dil_w;
                        if (ih < 0 || ih >= h || iw < 0 || iw >= w) continue;
                        acc += (double)val[j] * (double)x[(((size_t)n * h + ih) * w + iw) * c_in + c];
                    }
                    if (residual) acc += (double)residual[pix * c_out + o];
                    if (relu && acc < 0.0) acc = 0.0;
                    y[pix * c_out + o] = (float)acc;
                }
            }
        }
    }
    return 0;
}

/*
 * Max pooling over NHWC fp32 (the layer between the stem and the first residual block of the
 * ResNets of Sec. 4.5): y[n][oh][ow][c] = max of x over the kh x kw window whose corner is
 * (oh*stride_h - pad_h, ow*stride_w - pad_w); positions outside the image do not take part.
 * Returns 0, -1 on a bad argument (padding must be smaller than the window).
 */
int nm_oracle_maxpool2d(const float* x, int batch, int h, int w, int c, int kh, int kw, int stride_h,
                        int stride_w, int pad_h, int pad_w, float* y)
{
    if (!x || !y || batch < 1 || h < 1 || w < 1 || c < 1 || kh < 1 || kw < 1 || stride_h < 1 ||
        stride_w < 1 || pad_h < 0 || pad_w < 0 || pad_h >= kh || pad_w >= kw || h + 2 * pad_h < kh ||
        w + 2 * pad_w < kw)
        return -1;
    const int ho = (h + 2 * pad_h - kh) / stride_h + 1, wo = (w + 2 * pad_w - kw) / stride_w + 1;
    for (int n = 0; n < batch; ++n)
        for (int oh = 0; oh < ho; ++oh)
            for (int ow = 0; ow < wo; ++ow)
                for (int ch = 0; ch < c; ++ch) {
                    int seen = 0;
                    float m = 0.0f;
                    for (int i = 0; i < kh; ++i)
                        for (int j = 0; j < kw; ++j) {
                            const int ih = oh * stride_h - pad_h + i, iw = ow * stride_w - pad_w + j;
                            if (ih < 0 || ih >= h || iw < 0 || iw >= w) continue;
                            const float v = x[(((size_t)n * h + ih) * w + iw) * c + ch];
                            if (!seen || v > m) m = v;
                            seen = 1;
                        }
                    y[(((size_t)n * ho + oh) * wo + ow) * c + ch] = m;
                }
    return 0;
}
