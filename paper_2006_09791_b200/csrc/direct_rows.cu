// DIRECT_TILED, narrow-group kernel ("rows"): groups with at most 8 filters, down to depthwise.
//
// These layers move far more bytes than they compute (2.25 to 18 FLOP per byte), so the kernel is
// built around the load/store stream: no shared memory and no barrier.  One thread owns all Kg
// filters of one group for a strip of PR output rows x 4 adjacent output pixels.  For every input
// channel of the group it streams the strip's input rows from global memory (one aligned 16-byte
// load plus the halo scalars, which hit L1 because the neighbouring thread loads them as its
// vector), applies each row to every (output row, r) pair it feeds, and finally writes Kg x PR
// float4 results straight into NCHW.  Weights come from the packed [g][c][r][s][Kg] layout, so the
// Kg filters of a tap are one vector load that is uniform across most of a warp.
// Sum order per output: (c, r, s) as in the convolution stage of Algorithm 1.
#include "gconv_internal.h"

namespace gconv {

namespace {

template <int KT>
__device__ __forceinline__ void load_filters(const float* __restrict__ p, float (&wv)[KT]) {
    if constexpr (KT == 8) {
        const float4 a = __ldg(reinterpret_cast<const float4*>(p));
        const float4 b = __ldg(reinterpret_cast<const float4*>(p) + 1);
        wv[0] = a.x; wv[1] = a.y; wv[2] = a.z; wv[3] = a.w; wv[4] = b.x; wv[5] = b.y; wv[6] = b.z; wv[7] = b.w;
    } else if constexpr (KT == 4) {
        const float4 a = __ldg(reinterpret_cast<const float4*>(p));
        wv[0] = a.x; wv[1] = a.y; wv[2] = a.z; wv[3] = a.w;
    } else if constexpr (KT == 2) {
        const float2 a = __ldg(reinterpret_cast<const float2*>(p));
        wv[0] = a.x; wv[1] = a.y;
    } else {
        wv[0] = __ldg(p);
    }
}

// One input row segment for 4 output pixels: columns [b, b + NIN), b = ox*S - pad, zero outside.
template <int S, int NIN, bool VEC>
__device__ __forceinline__ void load_row(const float* __restrict__ row, bool row_ok, int b, int pad, int W,
                                         float (&in)[NIN]) {
    if constexpr (VEC) {
        // W % 4 == 0, pad <= 1, ox % 4 == 0: column a = b + pad is 16-byte aligned and a + 3 < W
        const int a = b + pad;
        float4 v0 = make_float4(0.f, 0.f, 0.f, 0.f), v1 = v0;
        float left = 0.f, r0 = 0.f, r1 = 0.f;
        if (row_ok) {
            v0 = __ldg(reinterpret_cast<const float4*>(row + a));
            if (S == 2 && a + 4 < W) v1 = __ldg(reinterpret_cast<const float4*>(row + a + 4));
            if (pad == 1 && a > 0) left = __ldg(row + a - 1);
            constexpr int after = (S == 1) ? 4 : 8;  // first column after the vector part
            if (a + after < W) r0 = __ldg(row + a + after);
            if (pad == 0 && S == 1 && a + after + 1 < W) r1 = __ldg(row + a + after + 1);
        }
        // assemble columns b .. b+NIN-1
        float tmp[NIN + 2];
        int o = 0;
        if (pad == 1) tmp[o++] = left;
        tmp[o++] = v0.x; tmp[o++] = v0.y; tmp[o++] = v0.z; tmp[o++] = v0.w;
        if (S == 2) { tmp[o++] = v1.x; tmp[o++] = v1.y; tmp[o++] = v1.z; tmp[o++] = v1.w; }
        tmp[o++] = r0;
        if (o < NIN + 2) tmp[o++] = r1;
#pragma unroll
        for (int j = 0; j < NIN; ++j) in[j] = tmp[j];
    } else {
#pragma unroll
        for (int j = 0; j < NIN; ++j) {
            const int v = b + j;
            in[j] = (row_ok && v >= 0 && v < W) ? __ldg(row + v) : 0.f;
        }
    }
}

template <int S, int KT, int PR, bool VEC>
__global__ void __launch_bounds__(128, (KT <= 2 && VEC) ? 8 : 1)
direct_rows_kernel(const Shape s, const RowsCfg c, const float* __restrict__ x, const uint32_t* __restrict__ packed,
                   float* __restrict__ y, Status* status, uint32_t tag) {
    // The header tag is loaded now but only examined right before the stores, so the check costs no
    // memory round trip ahead of the input loads; a mismatch still leaves y untouched.
    const uint32_t tag_seen = __ldg(packed);
    const float* __restrict__ wpk = reinterpret_cast<const float*>(packed + kHeaderBytes / 4);
    const uint32_t item = blockIdx.x * blockDim.x + threadIdx.x;
    if (item >= c.items) return;
    // item = ((n*G + g)*YT + yt)*XQ + xq
    uint32_t t, xq, yt, g, n;
    c.div_xq.divmod(item, t, xq);
    c.div_yt.divmod(t, t, yt);
    c.div_g.divmod(t, n, g);
    const int ox = (int)xq * 4;
    const int oy0 = (int)yt * PR;
    const int pad = VEC ? c.pad01 : s.pad;
    const int b = ox * S - s.pad;
    const int h0 = oy0 * S - s.pad;
    constexpr int NIN = 3 * S + 3;            // (4-1)*S + 3
    constexpr int NROWS = (PR - 1) * S + 3;

    float acc[KT][PR][4];
#pragma unroll
    for (int k = 0; k < KT; ++k)
#pragma unroll
        for (int p = 0; p < PR; ++p)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[k][p][j] = 0.f;

    const size_t plane = (size_t)s.H * s.W;
    const float* xc = x + ((size_t)n * s.C_in + (size_t)g * s.Cg) * plane;
    const float* wg = wpk + (size_t)g * s.Cg * 9 * KT;

    for (int ch = 0; ch < s.Cg; ++ch, xc += plane, wg += 9 * KT) {
        float wv[KT <= 2 ? 9 : 1][KT];
        if constexpr (KT <= 2) {
#pragma unroll
            for (int rs = 0; rs < 9; ++rs) load_filters<KT>(wg + rs * KT, wv[rs]);
        }
#pragma unroll
        for (int i = 0; i < NROWS; ++i) {
            const int h = h0 + i;
            const bool row_ok = (h >= 0) && (h < s.H);
            float in[NIN];
            load_row<S, NIN, VEC>(xc + (size_t)(row_ok ? h : 0) * s.W, row_ok, b, pad, s.W, in);
#pragma unroll
            for (int p = 0; p < PR; ++p) {
                const int r = i - p * S;
                if (r < 0 || r > 2) continue;
#pragma unroll
                for (int ss = 0; ss < 3; ++ss) {
                    if constexpr (KT <= 2) {
#pragma unroll
                        for (int k = 0; k < KT; ++k)
#pragma unroll
                            for (int j = 0; j < 4; ++j) acc[k][p][j] = fmaf(in[j * S + ss], wv[r * 3 + ss][k], acc[k][p][j]);
                    } else {
                        float wq[KT];
                        load_filters<KT>(wg + (r * 3 + ss) * KT, wq);
#pragma unroll
                        for (int k = 0; k < KT; ++k)
#pragma unroll
                            for (int j = 0; j < 4; ++j) acc[k][p][j] = fmaf(in[j * S + ss], wq[k], acc[k][p][j]);
                    }
                }
            }
        }
    }

    if (tag_seen != tag) {
        if (threadIdx.x == 0) record_status(status, GCONV_ERR_PACK_MISMATCH, (int)blockIdx.x);
        return;
    }
    const size_t oplane = (size_t)s.H_out * s.W_out;
    float* yb = y + ((size_t)n * s.C_out + (size_t)g * KT) * oplane;
    const bool vec_store = ((s.W_out & 3) == 0);
#pragma unroll
    for (int k = 0; k < KT; ++k) {
#pragma unroll
        for (int p = 0; p < PR; ++p) {
            const int oy = oy0 + p;
            if (oy >= s.H_out) continue;
            float* dst = yb + (size_t)k * oplane + (size_t)oy * s.W_out + ox;
            if (vec_store) {
                *reinterpret_cast<float4*>(dst) = make_float4(acc[k][p][0], acc[k][p][1], acc[k][p][2], acc[k][p][3]);
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    if (ox + j < s.W_out) dst[j] = acc[k][p][j];
            }
        }
    }
}

template <int S, int KT, int PR>
cudaError_t launch_rows(const Shape& s, const RowsCfg& c, const float* x, const void* packed, float* y, Status* status,
                        cudaStream_t st) {
    const unsigned blocks = (c.items + 127) / 128;
    const uint32_t tag = pack_tag(s, GCONV_VARIANT_DIRECT_TILED);
    if (c.vec)
        direct_rows_kernel<S, KT, PR, true><<<blocks, 128, 0, st>>>(s, c, x, reinterpret_cast<const uint32_t*>(packed), y, status, tag);
    else
        direct_rows_kernel<S, KT, PR, false><<<blocks, 128, 0, st>>>(s, c, x, reinterpret_cast<const uint32_t*>(packed), y, status, tag);
    return cudaGetLastError();
}

}  // namespace

FastDiv make_fastdiv(uint32_t d) {
    FastDiv f;
    f.div = d;
    if (d == 1) {
        f.mul = 0;
        f.shr = 0;
        return f;
    }
    uint32_t lg = 0;
    while ((1ull << lg) < d) ++lg;  // ceil(log2 d)
    const uint32_t p = 31 + lg;
    f.mul = (uint32_t)(((1ull << p) + d - 1) / d);
    f.shr = p - 32;
    return f;
}

bool rows_supported(const Shape& s) {
    if (!s.square()) return false;   // one stride, padding and dilation for both axes
    if (!(s.KH == 3 && s.KW == 3 && s.dilation == 1 && (s.stride == 1 || s.stride == 2))) return false;
    if (!(s.Kg == 1 || s.Kg == 2 || s.Kg == 4 || s.Kg == 8)) return false;
    if (s.Cg > 16) return false;
    const unsigned long long items = (unsigned long long)s.N * s.groups * ((s.H_out + 1) / 2) * ((s.W_out + 3) / 4);
    return items < (1ull << 31);
}

static int rows_pr(const Shape& s) {
    if (s.Kg >= 4) return 2;
    return s.H_out >= 4 ? 4 : 2;
}

RowsCfg rows_config(const Shape& s) {
    RowsCfg c;
    c.PR = rows_pr(s);
    const uint32_t XQ = (s.W_out + 3) / 4, YT = (s.H_out + c.PR - 1) / c.PR;
    c.div_xq = make_fastdiv(XQ);
    c.div_yt = make_fastdiv(YT);
    c.div_g = make_fastdiv((uint32_t)s.groups);
    c.items = (uint32_t)((unsigned long long)s.N * s.groups * YT * XQ);
    c.vec = (s.W % 4 == 0) && (s.pad <= 1);
    c.pad01 = s.pad;
    return c;
}

cudaError_t rows_forward(const Shape& s, const float* x, const void* packed, float* y, Status* status, cudaStream_t st) {
    const RowsCfg c = rows_config(s);
#define GCONV_ROWS_CASE(S, K, P) \
    if (s.stride == S && s.Kg == K && c.PR == P) return launch_rows<S, K, P>(s, c, x, packed, y, status, st);
    GCONV_ROWS_CASE(1, 1, 4) GCONV_ROWS_CASE(1, 1, 2) GCONV_ROWS_CASE(1, 2, 4) GCONV_ROWS_CASE(1, 2, 2)
    GCONV_ROWS_CASE(1, 4, 2) GCONV_ROWS_CASE(1, 8, 2)
    GCONV_ROWS_CASE(2, 1, 4) GCONV_ROWS_CASE(2, 1, 2) GCONV_ROWS_CASE(2, 2, 4) GCONV_ROWS_CASE(2, 2, 2)
    GCONV_ROWS_CASE(2, 4, 2) GCONV_ROWS_CASE(2, 8, 2)
#undef GCONV_ROWS_CASE
    return cudaErrorInvalidValue;
}

}  // namespace gconv
