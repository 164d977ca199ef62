/*
 * Grouped Spatial Pack Convolution (Algorithm 1, Section III-B of the paper) on the CPU.  TEST INFRASTRUCTURE ONLY:
 * a second CPU implementation, used by the tests (cross-check of the oracle) and timed by the benchmark as the
 * paper's own method on the host cores.  It shares no code with the CUDA path and none with gconv_ref.c.
 *
 * The method, in the paper's four stages and notation (CPG = C_in/g channels per group, KPG = C_out/g kernels per
 * group, tile sizes T_I and T_O, which by Eq. (1) lie in (0, CPG] and (0, KPG]; here they must also divide CPG and
 * KPG, which is what the floor-divided volume shapes of Section III-B need to hold every channel):
 *
 *   1. kernel reshaping    W [C_out][CPG][K_h][K_w]      ->  W'[g][KPG/T_O][CPG/T_I][K_h][K_w][T_I][T_O]
 *   2. input reshaping     X [N][C_in][H][W], zero-padded ->  X'[g][N][CPG/T_I][H_i][T_I][W_i]     (H_i = H + 2 pad)
 *   3. convolution         Y'[g][N][KPG/T_O][H_o][W_o][T_O] += X'[..][oh*S + kh*D][ti][ow*S + kw*D] * W'[..][kh][kw][ti][:]
 *   4. output reshaping    Y'                             ->  Y [N][C_out][H_o][W_o]
 *
 * Stage 1 does not depend on the input ("computed ahead of time"), so it has its own entry point and the timed call
 * runs stages 2-4.  The T_O outputs of one pixel sit next to each other in W' and Y', which is what the method wants
 * for SIMD lanes: the innermost loop below runs over them.  Arithmetic is float32 throughout, as in the paper's
 * experiments (Section IV-A); the tests compare it with the fp64 oracle at an fp32 tolerance.
 * Dilation D is not in the paper; D = 1 gives the printed algorithm.
 */
#include <stddef.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

static int out_dim(int in, int k, int stride, int pad, int dil)
{
    int span = in + 2 * pad - dil * (k - 1) - 1;
    return span < 0 ? 0 : span / stride + 1;
}

/* floats in W' */
size_t gspc_packed_kernel_elems(int C_in, int C_out, int KH, int KW, int groups)
{
    return (size_t)C_out * (size_t)(C_in / groups) * KH * KW;
}

/* stage 1: wp[g][ko][ct][kh][kw][ti][to] = w[g*KPG + ko*T_O + to][ct*T_I + ti][kh][kw] */
int gspc_pack_kernels(const float *w, float *wp, int C_in, int C_out, int KH, int KW, int groups, int T_I, int T_O)
{
    if (groups < 1 || C_in % groups || C_out % groups) return -1;
    const int CPG = C_in / groups, KPG = C_out / groups;
    if (T_I < 1 || T_O < 1 || CPG % T_I || KPG % T_O) return -1;
    const int nct = CPG / T_I, nko = KPG / T_O;
    for (int g = 0; g < groups; ++g)
        for (int ko = 0; ko < nko; ++ko)
            for (int ct = 0; ct < nct; ++ct)
                for (int kh = 0; kh < KH; ++kh)
                    for (int kw = 0; kw < KW; ++kw)
                        for (int ti = 0; ti < T_I; ++ti)
                            for (int to = 0; to < T_O; ++to) {
                                const size_t dst = ((((((size_t)g * nko + ko) * nct + ct) * KH + kh) * KW + kw) * T_I + ti) * T_O + to;
                                const size_t src = (((size_t)(g * KPG + ko * T_O + to) * CPG + (ct * T_I + ti)) * KH + kh) * KW + kw;
                                wp[dst] = w[src];
                            }
    return 0;
}

/* stage 3 for one (g, n, ko) slab: all T_O filters of the tile for every output pixel */
#if defined(__x86_64__) && defined(__GNUC__)
__attribute__((target_clones("avx512f", "avx2,fma", "default")))
#endif
static void conv_slab(const float *xg, const float *wk, float *yk, int nct, int T_I, int T_O, int KH, int KW, int Hi, int Wi,
                      int Ho, int Wo, int stride, int dil)
{
    for (int oh = 0; oh < Ho; ++oh)
        for (int ow = 0; ow < Wo; ++ow) {
            float *acc = yk + ((size_t)oh * Wo + ow) * T_O;
            for (int to = 0; to < T_O; ++to) acc[to] = 0.0f;
            for (int ct = 0; ct < nct; ++ct)
                for (int kh = 0; kh < KH; ++kh)
                    for (int kw = 0; kw < KW; ++kw)
                        for (int ti = 0; ti < T_I; ++ti) {
                            const float xv = xg[(((size_t)ct * Hi + (oh * stride + kh * dil)) * T_I + ti) * Wi + (ow * stride + kw * dil)];
                            const float *wv = wk + ((((size_t)ct * KH + kh) * KW + kw) * T_I + ti) * T_O;
#pragma omp simd
                            for (int to = 0; to < T_O; ++to) acc[to] += xv * wv[to];
                        }
        }
}

/*
 * Stages 2-4.  x [N][C_in][H][W], wp from gspc_pack_kernels with the same tiles, y [N][C_out][H_o][W_o] (float32).
 * stage_seconds, if not NULL, receives the wall time of stages 2, 3 and 4.  Returns 0, or -1 for an invalid problem
 * or tile pair, -2 when the temporary volumes cannot be allocated.
 */
int gspc_forward_f32(const float *x, const float *wp, float *y, int N, int C_in, int H, int W, int C_out, int KH, int KW,
                     int stride, int pad, int dilation, int groups, int T_I, int T_O, int threads, double *stage_seconds)
{
    if (N < 1 || C_in < 1 || H < 1 || W < 1 || C_out < 1 || KH < 1 || KW < 1) return -1;
    if (stride < 1 || pad < 0 || dilation < 1 || groups < 1 || C_in % groups || C_out % groups) return -1;
    const int CPG = C_in / groups, KPG = C_out / groups;
    if (T_I < 1 || T_O < 1 || CPG % T_I || KPG % T_O) return -1;
    const int Ho = out_dim(H, KH, stride, pad, dilation), Wo = out_dim(W, KW, stride, pad, dilation);
    if (Ho < 1 || Wo < 1) return -1;
    const int Hi = H + 2 * pad, Wi = W + 2 * pad;
    const int nct = CPG / T_I, nko = KPG / T_O;
    if (threads < 1) threads = 1;
    float *xp = (float *)malloc(sizeof(float) * (size_t)groups * N * CPG * Hi * Wi);
    float *yp = (float *)malloc(sizeof(float) * (size_t)groups * N * KPG * Ho * Wo);
    if (xp == NULL || yp == NULL) {
        free(xp);
        free(yp);
        return -2;
    }
    double t0 = 0, t1 = 0, t2 = 0, t3 = 0;
#ifdef _OPENMP
    t0 = omp_get_wtime();
#endif
    /* stage 2: xp[g][n][ct][h][ti][wcol] = padded x[n][g*CPG + ct*T_I + ti][h - pad][wcol - pad] */
#ifdef _OPENMP
#pragma omp parallel for collapse(2) num_threads(threads) schedule(static)
#endif
    for (int g = 0; g < groups; ++g)
        for (int n = 0; n < N; ++n)
            for (int ct = 0; ct < nct; ++ct)
                for (int h = 0; h < Hi; ++h)
                    for (int ti = 0; ti < T_I; ++ti) {
                        float *dst = xp + (((((size_t)g * N + n) * nct + ct) * Hi + h) * T_I + ti) * Wi;
                        const int hs = h - pad;
                        if (hs < 0 || hs >= H) {
                            memset(dst, 0, sizeof(float) * Wi);
                            continue;
                        }
                        const float *src = x + (((size_t)n * C_in + (g * CPG + ct * T_I + ti)) * H + hs) * W;
                        for (int c = 0; c < pad; ++c) dst[c] = 0.0f;
                        memcpy(dst + pad, src, sizeof(float) * W);
                        for (int c = pad + W; c < Wi; ++c) dst[c] = 0.0f;
                    }
#ifdef _OPENMP
    t1 = omp_get_wtime();
#endif
    /* stage 3: the convolution on the packed volumes */
#ifdef _OPENMP
#pragma omp parallel for collapse(3) num_threads(threads) schedule(static)
#endif
    for (int g = 0; g < groups; ++g)
        for (int n = 0; n < N; ++n)
            for (int ko = 0; ko < nko; ++ko) {
                const float *xg = xp + ((size_t)g * N + n) * (size_t)nct * Hi * T_I * Wi;
                const float *wk = wp + ((size_t)g * nko + ko) * (size_t)nct * KH * KW * T_I * T_O;
                float *yk = yp + (((size_t)g * N + n) * nko + ko) * (size_t)Ho * Wo * T_O;
                conv_slab(xg, wk, yk, nct, T_I, T_O, KH, KW, Hi, Wi, Ho, Wo, stride, dilation);
            }
#ifdef _OPENMP
    t2 = omp_get_wtime();
#endif
    /* stage 4: y[n][g*KPG + ko*T_O + to][oh][ow] = yp[g][n][ko][oh][ow][to] */
#ifdef _OPENMP
#pragma omp parallel for collapse(2) num_threads(threads) schedule(static)
#endif
    for (int n = 0; n < N; ++n)
        for (int c = 0; c < C_out; ++c) {
            const int g = c / KPG, ko = (c % KPG) / T_O, to = c % T_O;
            const float *src = yp + (((size_t)g * N + n) * nko + ko) * (size_t)Ho * Wo * T_O + to;
            float *dst = y + ((size_t)n * C_out + c) * (size_t)Ho * Wo;
            for (size_t p = 0; p < (size_t)Ho * Wo; ++p) dst[p] = src[p * T_O];
        }
#ifdef _OPENMP
    t3 = omp_get_wtime();
#endif
    if (stage_seconds != NULL) {
        stage_seconds[0] = t1 - t0;
        stage_seconds[1] = t2 - t1;
        stage_seconds[2] = t3 - t2;
    }
    free(xp);
    free(yp);
    return 0;
}
