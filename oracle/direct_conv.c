/* CPU oracle: direct convolution in fp64 -- TEST INFRASTRUCTURE ONLY.
 *
 * The definition every execution kernel must reproduce (the paper's notion of
 * one operator with many interchangeable kernels, its Section 3.1.1, and its
 * "general" kernel row of Table 2):
 *
 *   Y[k,oh,ow] = b[k] + sum_{c in group(k)} sum_{r<R} sum_{s<S}
 *                X[c, oh*st + r - pad, ow*st + s - pad] * W[k,c,r,s]
 *
 * with X = 0 outside the image, cross-correlation (no filter flip), and
 * OH = floor((H + 2*pad - R)/st) + 1.  Inputs are fp32, all arithmetic fp64.
 * Plain loops; OpenMP over output channels only.
 */
#include <stddef.h>

void oracle_direct_conv(const float *x, const float *w, const float *bias, double *y,
                        int C, int H, int W, int K, int R, int S,
                        int stride, int pad, int groups)
{
    const int OH = (H + 2 * pad - R) / stride + 1;
    const int OW = (W + 2 * pad - S) / stride + 1;
    const int Cg = C / groups;
    const int Kg = K / groups;
#pragma omp parallel for schedule(dynamic, 1)
    for (int k = 0; k < K; ++k) {
        const int g = k / Kg;
        for (int oh = 0; oh < OH; ++oh) {
            for (int ow = 0; ow < OW; ++ow) {
                double acc = bias ? (double)bias[k] : 0.0;
                for (int cc = 0; cc < Cg; ++cc) {
                    const int c = g * Cg + cc;
                    for (int r = 0; r < R; ++r) {
                        const int ih = oh * stride + r - pad;
                        if (ih < 0 || ih >= H) continue;
                        for (int s = 0; s < S; ++s) {
                            const int iw = ow * stride + s - pad;
                            if (iw < 0 || iw >= W) continue;
                            acc += (double)x[((size_t)c * H + ih) * W + iw] *
                                   (double)w[(((size_t)k * Cg + cc) * R + r) * S + s];
                        }
                    }
                }
                y[((size_t)k * OH + oh) * OW + ow] = acc;
            }
        }
    }
}

/* Same definition with an fp64 input (used when chaining layers in fp64). */
void oracle_direct_conv_f64(const double *x, const float *w, const float *bias, double *y,
                            int C, int H, int W, int K, int R, int S,
                            int stride, int pad, int groups)
{
    const int OH = (H + 2 * pad - R) / stride + 1;
    const int OW = (W + 2 * pad - S) / stride + 1;
    const int Cg = C / groups;
    const int Kg = K / groups;
#pragma omp parallel for schedule(dynamic, 1)
    for (int k = 0; k < K; ++k) {
        const int g = k / Kg;
        for (int oh = 0; oh < OH; ++oh) {
            for (int ow = 0; ow < OW; ++ow) {
                double acc = bias ? (double)bias[k] : 0.0;
                for (int cc = 0; cc < Cg; ++cc) {
                    const int c = g * Cg + cc;
                    for (int r = 0; r < R; ++r) {
                        const int ih = oh * stride + r - pad;
                        if (ih < 0 || ih >= H) continue;
                        for (int s = 0; s < S; ++s) {
                            const int iw = ow * stride + s - pad;
                            if (iw < 0 || iw >= W) continue;
                            acc += x[((size_t)c * H + ih) * W + iw] *
                                   (double)w[(((size_t)k * Cg + cc) * R + r) * S + s];
                        }
                    }
                }
                y[((size_t)k * OH + oh) * OW + ow] = acc;
            }
        }
    }
}
