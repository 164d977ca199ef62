/*
 * Reference oracle for the forward grouped 2-D convolution. TEST INFRASTRUCTURE ONLY.
 *
 * This file is the slow, plain, obviously-correct statement of what the library computes.  It is
 * used by the tests, the smoke check and the CPU-baseline leg of the benchmark, never by the
 * product path, and it shares no code with the CUDA kernels.
 *
 * What it computes (grouped convolution as defined in Section II of the paper; index form of the
 * convolution stage of Algorithm 1, i.e. input row oh*S_h + kh and column ow*S_w + kw on the
 * zero-padded input, no kernel flip):
 *
 *   y[n, g*Kg + k, p, q] = sum_{c < Cg} sum_{r < KH} sum_{s < KW}
 *        x[n, g*Cg + c, p*stride + r*dilation - pad, q*stride + s*dilation - pad] * w[g*Kg + k, c, r, s]
 *
 *   Cg = C_in / groups (the paper's CPG), Kg = C_out / groups (the paper's KPG); both divisions
 *   must be exact (Section III-B).  x is NCHW, w is [C_out, Cg, KH, KW], y is NCHW.
 *   Reads outside [0,H) x [0,W) contribute zero (the paper convolves a padded input).
 *   H_out = floor((H + 2*pad - dilation*(KH-1) - 1) / stride) + 1, likewise W_out.
 *
 *   Algorithm 1 carries one stride per axis (S_h for rows, S_w for columns); gconv_ref_f64_2d takes stride, padding
 *   and dilation per axis (row index p*stride_h + r*dilation_h - pad_h, column index q*stride_w + s*dilation_w - pad_w)
 *   and gconv_ref_f64 is the same sum with both axes given the same values.
 *
 * Arithmetic: inputs are fp32, every product and the running sum are fp64 (an fp32 x fp32 product
 * is exact in fp64), the result is returned in fp64.  Seven loops: four over the output, three
 * over the reduction.
 *
 * MAC counter: one per (output element, c, r, s) visited, including taps that fall in the padding,
 * so that it equals Eq. (2) of the paper: N*C_in*C_out*KH*KW*H_out*W_out / groups.
 *
 * The optional thread count only spreads the two outermost loops (n, output channel) over cores
 * with OpenMP; each output element is still computed by one thread in the order above.
 */
#include <stddef.h>

#ifdef _OPENMP
#include <omp.h>
#endif

int gconv_ref_out_dim(int in, int k, int stride, int pad, int dilation)
{
    int span = in + 2 * pad - dilation * (k - 1) - 1;
    if (span < 0) return 0;
    return span / stride + 1;
}

/* returns 0 on success, -1 on an invalid problem */
int gconv_ref_f64_2d(const float *x, const float *w, double *y,
                     int N, int C_in, int H, int W, int C_out, int KH, int KW,
                     int stride_h, int stride_w, int pad_h, int pad_w, int dilation_h, int dilation_w, int groups,
                     int threads, long long *macs_out)
{
    if (N < 1 || C_in < 1 || H < 1 || W < 1 || C_out < 1 || KH < 1 || KW < 1) return -1;
    if (stride_h < 1 || stride_w < 1 || pad_h < 0 || pad_w < 0 || dilation_h < 1 || dilation_w < 1 || groups < 1) return -1;
    if (C_in % groups != 0 || C_out % groups != 0) return -1;
    const int Cg = C_in / groups;
    const int Kg = C_out / groups;
    const int H_out = gconv_ref_out_dim(H, KH, stride_h, pad_h, dilation_h);
    const int W_out = gconv_ref_out_dim(W, KW, stride_w, pad_w, dilation_w);
    if (H_out < 1 || W_out < 1) return -1;
    long long macs = 0;
    if (threads < 1) threads = 1;

#ifdef _OPENMP
#pragma omp parallel for collapse(2) num_threads(threads) reduction(+ : macs) schedule(static)
#endif
    for (int n = 0; n < N; ++n) {
        for (int ko = 0; ko < C_out; ++ko) {
            const int g = ko / Kg;
            for (int p = 0; p < H_out; ++p) {
                for (int q = 0; q < W_out; ++q) {
                    double acc = 0.0;
                    for (int c = 0; c < Cg; ++c) {
                        for (int r = 0; r < KH; ++r) {
                            for (int s = 0; s < KW; ++s) {
                                const int h = p * stride_h + r * dilation_h - pad_h;
                                const int v = q * stride_w + s * dilation_w - pad_w;
                                macs += 1;
                                if (h >= 0 && h < H && v >= 0 && v < W) {
                                    const size_t xi = (((size_t)n * C_in + (size_t)(g * Cg + c)) * H + h) * W + v;
                                    const size_t wi = (((size_t)ko * Cg + c) * KH + r) * KW + s;
                                    acc += (double)x[xi] * (double)w[wi];
                                }
                            }
                        }
                    }
                    y[(((size_t)n * C_out + ko) * H_out + p) * W_out + q] = acc;
                }
            }
        }
    }
    if (macs_out) *macs_out = macs;
    return 0;
}

/* the square case: one stride, padding and dilation for both axes */
int gconv_ref_f64(const float *x, const float *w, double *y,
                  int N, int C_in, int H, int W, int C_out, int KH, int KW,
                  int stride, int pad, int dilation, int groups,
                  int threads, long long *macs_out)
{
    return gconv_ref_f64_2d(x, w, y, N, C_in, H, W, C_out, KH, KW, stride, stride, pad, pad, dilation, dilation, groups,
                            threads, macs_out);
}

int gconv_ref_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
