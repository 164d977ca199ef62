// Variant DIRECT_TILED: FP32 FFMA direct grouped convolution for narrow groups down to depthwise.
//
// One CTA computes, for one image, GB consecutive groups x KB output channels of each group x a
// TH x TW patch of output pixels.  The input halo patch of the CTA's channels is staged once in
// shared memory with zero fill outside the image (this plays the role of Algorithm 1's padded,
// group-split input reshape, without a pass over HBM), the CTA's slice of the packed weights
// [g][c][r][s][Kg] (Kg innermost, so a thread's KT filters are one vector load) sits beside it,
// and every thread accumulates a register tile of KT output channels x 4 adjacent output pixels
// over (c, r, s) in the order of the convolution stage of Algorithm 1.  y is written directly in
// NCHW.  3x3 kernels, dilation 1, stride 1 or 2, any padding.
#include "gconv_internal.h"

namespace gconv {

namespace {

constexpr int PW = 4;  // output pixels per thread along W

template <int STRIDE, int KT>
__global__ void __launch_bounds__(256)
direct_tiled_kernel(const Shape s, const TiledCfg c, const float* __restrict__ x, const uint32_t* __restrict__ packed,
                    float* __restrict__ y, Status* status, uint32_t tag) {
    extern __shared__ __align__(16) float smem[];
    if (packed[0] != tag) {
        if (threadIdx.x == 0) record_status(status, GCONV_ERR_PACK_MISMATCH, (int)blockIdx.x);
        return;
    }
    const float* __restrict__ wpk = reinterpret_cast<const float*>(packed + kHeaderBytes / 4);

    // ---- which tile --------------------------------------------------------------------------
    int b = blockIdx.x;
    const int tile_x = b % c.tiles_x;  b /= c.tiles_x;
    const int tile_y = b % c.tiles_y;  b /= c.tiles_y;
    const int kblock = b % c.kblocks;  b /= c.kblocks;
    const int gblock = b;
    const int n = blockIdx.y;
    const int g0 = gblock * c.GB;
    const int gcount = min(c.GB, s.groups - g0);
    const int KB = c.KQ * KT;
    const int kb0 = kblock * KB;
    const int x0 = tile_x * (c.TXT * PW);
    const int y0 = tile_y * c.TY;
    const int in_x0 = x0 * STRIDE - s.pad;
    const int in_y0 = y0 * STRIDE - s.pad;

    float* s_in = smem;                                 // [GB][CCH][IH][IWP]
    float* s_w = smem + c.GB * c.CCH * c.IH * c.IWP;    // [GB][CCH][3][3][KB]

    // ---- which outputs this thread owns ------------------------------------------------------
    const int tid = threadIdx.x;
    int t = tid;
    const int tx = t % c.TXT;  t /= c.TXT;
    const int ty = t % c.TY;   t /= c.TY;
    const int kq = t % c.KQ;   t /= c.KQ;
    const int gl = t;
    const bool active = (gl < gcount);

    float acc[KT][PW];
#pragma unroll
    for (int k = 0; k < KT; ++k)
#pragma unroll
        for (int j = 0; j < PW; ++j) acc[k][j] = 0.f;

    const int lanes_per_row = c.LPR;            // power of two <= 32 covering IW
    const int row_in_pass = tid / lanes_per_row;
    const int ix0 = tid % lanes_per_row;
    const int rows_per_pass = blockDim.x / lanes_per_row;
    const size_t plane = (size_t)s.H * s.W;
    const float* xn = x + ((size_t)n * s.C_in + (size_t)g0 * s.Cg) * plane;

    for (int c0 = 0; c0 < s.Cg; c0 += c.CCH) {
        const int cch = min(c.CCH, s.Cg - c0);
        if (c0 > 0) __syncthreads();
        // stage the input halo patch: rows = (group, channel, iy), zero outside the image
        const int nrows = gcount * cch * c.IH;
        for (int row = row_in_pass; row < nrows; row += rows_per_pass) {
            const int iy = row % c.IH;
            const int gc = row / c.IH;       // gl * cch + cc
            const int cc = gc % cch;
            const int gll = gc / cch;
            const int h = in_y0 + iy;
            const bool hin = (h >= 0) && (h < s.H);
            const float* src = xn + ((size_t)(gll * s.Cg + c0 + cc)) * plane + (size_t)(hin ? h : 0) * s.W;
            float* dst = s_in + ((gll * c.CCH + cc) * c.IH + iy) * c.IWP;
            for (int ix = ix0; ix < c.IWP; ix += lanes_per_row) {
                const int v = in_x0 + ix;
                float val = 0.f;
                if (hin && v >= 0 && v < s.W && ix < c.IW) val = __ldg(src + v);
                dst[ix] = val;
            }
        }
        // stage the weights of this channel chunk: [gl][cc][r][s][KB]
        const int wrows = gcount * cch * 9;
        for (int e = tid; e < wrows * KB; e += blockDim.x) {
            const int k = e % KB;
            const int rr = e / KB;           // (gl*cch + cc)*9 + rs
            const int rs = rr % 9;
            const int gc = rr / 9;
            const int cc = gc % cch;
            const int gll = gc / cch;
            const size_t srci = (((size_t)(g0 + gll) * s.Cg + (c0 + cc)) * 9 + rs) * s.Kg + kb0 + k;
            s_w[((gll * c.CCH + cc) * 9 + rs) * KB + k] = (kb0 + k < s.Kg) ? __ldg(wpk + srci) : 0.f;
        }
        __syncthreads();

        if (active) {
            for (int cc = 0; cc < cch; ++cc) {
                const float* in_c = s_in + ((gl * c.CCH + cc) * c.IH + ty * STRIDE) * c.IWP + tx * (PW * STRIDE);
                const float* w_c = s_w + ((gl * c.CCH + cc) * 9) * KB + kq * KT;
#pragma unroll
                for (int r = 0; r < 3; ++r) {
                    constexpr int NIN = (PW - 1) * STRIDE + 3;
                    float in[NIN + 3];
                    const float* row = in_c + r * c.IWP;
                    {
                        const float4 a = *reinterpret_cast<const float4*>(row);
                        in[0] = a.x; in[1] = a.y; in[2] = a.z; in[3] = a.w;
                        if (STRIDE == 1) {
                            const float2 bq = *reinterpret_cast<const float2*>(row + 4);
                            in[4] = bq.x; in[5] = bq.y;
                        } else {
                            const float4 bq = *reinterpret_cast<const float4*>(row + 4);
                            in[4] = bq.x; in[5] = bq.y; in[6] = bq.z; in[7] = bq.w;
                            in[8] = row[8];
                        }
                    }
#pragma unroll
                    for (int ss = 0; ss < 3; ++ss) {
                        float wv[KT];
                        const float* wp = w_c + (r * 3 + ss) * KB;
                        if (KT % 4 == 0) {
#pragma unroll
                            for (int k4 = 0; k4 < KT / 4; ++k4) {
                                const float4 q = *reinterpret_cast<const float4*>(wp + 4 * k4);
                                wv[4 * k4 + 0] = q.x; wv[4 * k4 + 1] = q.y; wv[4 * k4 + 2] = q.z; wv[4 * k4 + 3] = q.w;
                            }
                        } else if (KT == 2) {
                            const float2 q = *reinterpret_cast<const float2*>(wp);
                            wv[0] = q.x; wv[KT - 1] = q.y;
                        } else {
#pragma unroll
                            for (int k = 0; k < KT; ++k) wv[k] = wp[k];
                        }
#pragma unroll
                        for (int k = 0; k < KT; ++k)
#pragma unroll
                            for (int j = 0; j < PW; ++j) acc[k][j] = fmaf(in[j * STRIDE + ss], wv[k], acc[k][j]);
                    }
                }
            }
        }
    }

    if (!active) return;
    const int oy = y0 + ty;
    const int ox = x0 + tx * PW;
    if (oy >= s.H_out || ox >= s.W_out) return;
    const size_t oplane = (size_t)s.H_out * s.W_out;
    const int kbase = kb0 + kq * KT;
    const bool vec = ((s.W_out & 3) == 0);  // then ox + 3 < W_out and the row start is 16-byte aligned
#pragma unroll
    for (int k = 0; k < KT; ++k) {
        if (kbase + k >= s.Kg) break;
        float* dst = y + ((size_t)n * s.C_out + (size_t)(g0 + gl) * s.Kg + kbase + k) * oplane + (size_t)oy * s.W_out + ox;
        if (vec) {
            *reinterpret_cast<float4*>(dst) = make_float4(acc[k][0], acc[k][1], acc[k][2], acc[k][3]);
        } else {
#pragma unroll
            for (int j = 0; j < PW; ++j)
                if (ox + j < s.W_out) dst[j] = acc[k][j];
        }
    }
}

__global__ void tiled_pack_kernel(Shape s, const float* __restrict__ w, uint32_t* __restrict__ packed, uint32_t tag) {
    const int taps = s.KH * s.KW;               // 9, or 25 for the 5x5 depthwise layers
    const size_t n = (size_t)s.C_out * s.Cg * taps;
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i == 0) {
        packed[0] = tag;
        for (int j = 1; j < kHeaderBytes / 4; ++j) packed[j] = 0;
    }
    float* dst = reinterpret_cast<float*>(packed + kHeaderBytes / 4);
    for (; i < n; i += (size_t)gridDim.x * blockDim.x) {
        // destination index i = (((g*Cg + c)*taps + rs)*Kg + k)
        const int k = (int)(i % s.Kg);
        size_t t = i / s.Kg;
        const int rs = (int)(t % taps);
        t /= taps;
        const int c = (int)(t % s.Cg);
        const int g = (int)(t / s.Cg);
        dst[i] = w[(((size_t)g * s.Kg + k) * s.Cg + c) * taps + rs];
    }
}

int largest_kt(int Kg) {
    if (Kg % 8 == 0) return 8;
    if (Kg % 4 == 0) return 4;
    if (Kg % 2 == 0) return 2;
    return 1;
}

}  // namespace

bool tiled_supported(const Shape& s) {
    if (!s.square()) return false;   // one stride, padding and dilation for both axes
    if (s.KH == 5 && s.KW == 5) return dw_supported(s);   // 5x5: only the depthwise stream kernel
    return s.KH == 3 && s.KW == 3 && s.dilation == 1 && (s.stride == 1 || s.stride == 2) && s.N <= 65535;
}

size_t tiled_packed_bytes(const Shape& s) { return kHeaderBytes + sizeof(float) * (size_t)s.C_out * s.Cg * s.KH * s.KW; }

cudaError_t tiled_pack(const Shape& s, const float* w, void* packed, cudaStream_t st) {
    const size_t n = (size_t)s.C_out * s.Cg * s.KH * s.KW;
    int blocks = (int)((n + 255) / 256 < 1184 ? (n + 255) / 256 : 1184);
    tiled_pack_kernel<<<blocks, 256, 0, st>>>(s, w, reinterpret_cast<uint32_t*>(packed), pack_tag(s, GCONV_VARIANT_DIRECT_TILED));
    return cudaGetLastError();
}

TiledCfg tiled_config(const Shape& s, int sm_count) {
    TiledCfg c;
    const int S = s.stride;
    c.KT = largest_kt(s.Kg);
    const int kq_full = s.Kg / c.KT;
    // x threads: split W_out into equal tiles of at most 8 threads (32 pixels)
    const int xthreads = (s.W_out + PW - 1) / PW;
    const int ntx = (xthreads + 7) / 8;
    c.TXT = (xthreads + ntx - 1) / ntx;
    // rows: up to 8 per tile when several filters share the patch, up to a whole CTA otherwise
    int ty_max = 256 / (c.TXT * (kq_full < 8 ? kq_full : 8));
    if (ty_max < 4) ty_max = 4;
    if (ty_max > 32) ty_max = 32;
    const int nty = (s.H_out + ty_max - 1) / ty_max;
    c.TY = (s.H_out + nty - 1) / nty;
    int kq = 256 / (c.TXT * c.TY);
    if (kq < 1) kq = 1;
    if (kq > kq_full) kq = kq_full;
    c.KQ = kq;
    c.kblocks = (kq_full + kq - 1) / kq;
    c.tiles_x = ntx;
    c.tiles_y = nty;
    c.CCH = s.Cg < 8 ? s.Cg : 8;
    c.IH = (c.TY - 1) * S + 3;
    c.IW = (c.TXT * PW - 1) * S + 3;
    c.IWP = ((c.TXT * PW * S + (S == 1 ? 2 : 1)) + 3) & ~3;  // covers the widest vector read of the last thread
    if (c.IWP < c.IW) c.IWP = (c.IW + 3) & ~3;
    int lpr = 1;
    while (lpr < c.IWP && lpr < 32) lpr <<= 1;
    c.LPR = lpr;
    // several groups per CTA when one group does not fill it, as long as the grid still covers the chip
    int gb = 1;
    if (c.kblocks == 1) {
        const int per_group = c.TXT * c.TY * c.KQ;
        gb = 256 / per_group;
        if (gb < 1) gb = 1;
        if (gb > s.groups) gb = s.groups;
        const long long ctas1 = (long long)ntx * nty * s.N * s.groups;
        while (gb > 1 && ctas1 / gb < 4LL * sm_count) gb >>= 1;
        const size_t per_g_smem = sizeof(float) * ((size_t)c.CCH * c.IH * c.IWP + (size_t)c.CCH * 9 * c.KQ * c.KT);
        while (gb > 1 && gb * per_g_smem > 96 * 1024) gb >>= 1;
    }
    c.GB = gb;
    c.gblocks = (s.groups + gb - 1) / gb;
    const int nt = c.TXT * c.TY * c.KQ * c.GB;
    c.threads = (nt + 31) & ~31;
    c.smem = sizeof(float) * ((size_t)c.GB * c.CCH * c.IH * c.IWP + (size_t)c.GB * c.CCH * 9 * c.KQ * c.KT);
    return c;
}

template <int STRIDE, int KT>
static cudaError_t launch_tiled(const Shape& s, const TiledCfg& c, const float* x, const void* packed, float* y,
                                Status* status, cudaStream_t st) {
    auto kern = direct_tiled_kernel<STRIDE, KT>;
    if (c.smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)c.smem);
        if (e != cudaSuccess) return e;
    }
    dim3 grid((unsigned)(c.tiles_x * c.tiles_y * c.kblocks * c.gblocks), (unsigned)s.N);
    kern<<<grid, c.threads, c.smem, st>>>(s, c, x, reinterpret_cast<const uint32_t*>(packed), y, status,
                                          pack_tag(s, GCONV_VARIANT_DIRECT_TILED));
    return cudaGetLastError();
}

cudaError_t tiled_forward(const Shape& s, const float* x, const void* packed, float* y, Status* status, int sm_count,
                          cudaStream_t st) {
    if (dw_supported(s)) return dw_forward(s, x, packed, y, status, sm_count, st);
    if (rows_supported(s)) return rows_forward(s, x, packed, y, status, st);
    const TiledCfg c = tiled_config(s, sm_count);
#define GCONV_TILED_CASE(S, K) \
    if (s.stride == S && c.KT == K) return launch_tiled<S, K>(s, c, x, packed, y, status, st);
    GCONV_TILED_CASE(1, 1) GCONV_TILED_CASE(1, 2) GCONV_TILED_CASE(1, 4) GCONV_TILED_CASE(1, 8)
    GCONV_TILED_CASE(2, 1) GCONV_TILED_CASE(2, 2) GCONV_TILED_CASE(2, 4) GCONV_TILED_CASE(2, 8)
#undef GCONV_TILED_CASE
    return cudaErrorInvalidValue;
}

}  // namespace gconv
