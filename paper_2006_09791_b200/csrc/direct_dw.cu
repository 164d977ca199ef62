// DIRECT_TILED, depthwise kernel ("stream"): groups = C_in = C_out, 3x3, pad 1, stride 1 or 2, W <= 128 (256 for stride 2).
//
// Depthwise layers do 9 MACs per output and are bound by the HBM stream (2.25 FLOP per byte), so the
// kernel is a software-pipelined stream: a thread owns a strip of 4 output columns of one plane and
// walks down RH output rows.  Input rows arrive as aligned 16-byte loads (four scalar loads when W is not a
// multiple of 4) that are issued one block of
// rows ahead of their use (the next block's loads are in flight while the current block is computed),
// the one-pixel left/right halos come from the neighbouring lanes by warp shuffle (a warp holds whole
// rows: lane = strip-within-row, several rows' strips per warp), and every output row leaves as one
// 16-byte store.  No shared memory, no barrier.  Sum order per output: (r, s) as in Algorithm 1.
#include "gconv_internal.h"

namespace gconv {

namespace {

constexpr int U = 4;   // output rows per pipeline block (strip lengths are multiples of it)

// Four consecutive pixels of row h starting at column col (zero outside the image).  VEC = 4: W % 4 == 0, so the
// address is 16-byte aligned and the four pixels are in range; VEC = 2: W is even, two 8-byte loads (the second pair
// may be past the row); VEC = 0: four bounds-checked scalar loads.
template <int VEC>
__device__ __forceinline__ float4 ldrow(const float* __restrict__ plane, int h, int H, int W, int col) {
    if (h < 0 || h >= H) return make_float4(0.f, 0.f, 0.f, 0.f);
    const float* p = plane + (size_t)h * W + col;
    if constexpr (VEC == 4) {
        return __ldg(reinterpret_cast<const float4*>(p));
    } else if constexpr (VEC == 2) {
        const float2 a = __ldg(reinterpret_cast<const float2*>(p));
        const float2 b = col + 2 < W ? __ldg(reinterpret_cast<const float2*>(p + 2)) : make_float2(0.f, 0.f);
        return make_float4(a.x, a.y, b.x, b.y);
    } else {
        float4 v;
        v.x = col + 0 < W ? __ldg(p + 0) : 0.f;
        v.y = col + 1 < W ? __ldg(p + 1) : 0.f;
        v.z = col + 2 < W ? __ldg(p + 2) : 0.f;
        v.w = col + 3 < W ? __ldg(p + 3) : 0.f;
        return v;
    }
}
template <int VEC>
__device__ __forceinline__ void strow(float* __restrict__ dst, int col, int W, const float (&acc)[4]) {
    if constexpr (VEC == 4) {
        *reinterpret_cast<float4*>(dst) = make_float4(acc[0], acc[1], acc[2], acc[3]);
    } else if constexpr (VEC == 2) {
        *reinterpret_cast<float2*>(dst) = make_float2(acc[0], acc[1]);
        if (col + 2 < W) *reinterpret_cast<float2*>(dst + 2) = make_float2(acc[2], acc[3]);
    } else {
#pragma unroll
        for (int j = 0; j < 4; ++j)
            if (col + j < W) dst[j] = acc[j];
    }
}

// ---- stride 1 -------------------------------------------------------------------------------------
// One input row's contribution to an output row: v = the strip's own four columns, l / r = the columns just left and
// right of it (from the neighbouring lanes, zero at the image border).
__device__ __forceinline__ void row_taps1(const float4 v, const float l, const float r, const float (&w)[3], float (&acc)[4]) {
    acc[0] = fmaf(l, w[0], acc[0]);   acc[0] = fmaf(v.x, w[1], acc[0]); acc[0] = fmaf(v.y, w[2], acc[0]);
    acc[1] = fmaf(v.x, w[0], acc[1]); acc[1] = fmaf(v.y, w[1], acc[1]); acc[1] = fmaf(v.z, w[2], acc[1]);
    acc[2] = fmaf(v.y, w[0], acc[2]); acc[2] = fmaf(v.z, w[1], acc[2]); acc[2] = fmaf(v.w, w[2], acc[2]);
    acc[3] = fmaf(v.z, w[0], acc[3]); acc[3] = fmaf(v.w, w[1], acc[3]); acc[3] = fmaf(r, w[2], acc[3]);
}

// UB = output rows per pipeline block: 4 on planes of 28 rows and more (80 registers, three blocks per SM), 2 on smaller
// ones (64 registers, four blocks per SM: short strips want more warps rather than more rows in flight per thread).
template <int VEC, int UB>
__global__ void __launch_bounds__(256, VEC == 0 ? 2 : (UB == 4 ? 3 : 4))
dw_stream_s1_kernel(const Shape s, const DwCfg c, const float* __restrict__ x, const uint32_t* __restrict__ packed,
                    float* __restrict__ y, Status* status, uint32_t tag) {
    const uint32_t tag_seen = __ldg(packed);
    const float* __restrict__ wpk = reinterpret_cast<const float*>(packed + kHeaderBytes / 4);
    const int lane = threadIdx.x & 31;
    const uint32_t warp_global = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int sub = lane / c.XQ;                 // which of the warp's strips-of-rows this lane belongs to
    const int xq = lane - sub * c.XQ;
    // item = plane * chunks + chunk ; the warp holds `subs` consecutive items
    const uint32_t item = warp_global * (uint32_t)c.subs + (uint32_t)sub;
    const bool live = (sub < c.subs) && (item < c.items);
    uint32_t plane_idx = 0, chunk = 0;
    c.div_chunks.divmod(live ? item : 0u, plane_idx, chunk);
    const int ch = (int)(plane_idx % (uint32_t)s.C_in);
    const float* __restrict__ xp = x + (size_t)plane_idx * s.H * s.W;
    float* __restrict__ yp = y + (size_t)plane_idx * s.H * s.W;
    const int col = xq * 4;
    const int p0 = (int)chunk * c.RH;
    const int p1 = min(p0 + c.RH, s.H);
    const bool has_l = xq > 0, has_r = xq < c.XQ - 1;
    float w[3][3];
#pragma unroll
    for (int i = 0; i < 9; ++i) w[i / 3][i % 3] = live ? __ldg(wpk + (size_t)ch * 9 + i) : 0.f;

    // rows p-1 .. p+UB of the current block; `live` only gates memory traffic, every lane runs the shuffles.  A row
    // feeds three output rows, so its two halo columns are fetched from the neighbouring lanes once, when the row
    // enters the block, and kept (hl, hr).
    float4 cur[UB + 2], nxt[UB];
    float hl[UB + 2], hr[UB + 2];
    auto halo = [&](const float4 v, float& l, float& r) {
        const float a = __shfl_up_sync(0xffffffffu, v.w, 1), b = __shfl_down_sync(0xffffffffu, v.x, 1);
        l = has_l ? a : 0.f;
        r = has_r ? b : 0.f;
    };
#pragma unroll
    for (int j = 0; j < UB + 2; ++j) cur[j] = live ? ldrow<VEC>(xp, p0 - 1 + j, s.H, s.W, col) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int j = 0; j < UB + 2; ++j) halo(cur[j], hl[j], hr[j]);
    for (int p = p0; p < p0 + c.RH; p += UB) {        // warp-uniform trip count
#pragma unroll
        for (int j = 0; j < UB; ++j) {                  // next block's new rows, in flight during this block's math
            const int h = p + UB + 1 + j;
            nxt[j] = (live && h <= p1) ? ldrow<VEC>(xp, h, s.H, s.W, col) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int j = 0; j < UB; ++j) {
            float acc[4] = {0.f, 0.f, 0.f, 0.f};
            row_taps1(cur[j], hl[j], hr[j], w[0], acc);
            row_taps1(cur[j + 1], hl[j + 1], hr[j + 1], w[1], acc);
            row_taps1(cur[j + 2], hl[j + 2], hr[j + 2], w[2], acc);
            if (live && p + j < p1 && tag_seen == tag) strow<VEC>(yp + (size_t)(p + j) * s.W + col, col, s.W, acc);
        }
        cur[0] = cur[UB];
        cur[1] = cur[UB + 1];
        hl[0] = hl[UB]; hr[0] = hr[UB];
        hl[1] = hl[UB + 1]; hr[1] = hr[UB + 1];
#pragma unroll
        for (int j = 0; j < UB; ++j) {
            cur[2 + j] = nxt[j];
            halo(nxt[j], hl[2 + j], hr[2 + j]);
        }
    }
    if (tag_seen != tag && threadIdx.x == 0) record_status(status, GCONV_ERR_PACK_MISMATCH, (int)blockIdx.x);
}

// ---- stride 2 -------------------------------------------------------------------------------------
// Four outputs q..q+3 read input columns 2q-1 .. 2q+7: two aligned float4 (a, b) and the previous lane's b.w.
// (l = the column just left of the strip: the previous lane's b.w, zero at the image border)
__device__ __forceinline__ void row_taps2(const float4 a, const float4 b, const float l, const float (&w)[3], float (&acc)[4]) {
    acc[0] = fmaf(l, w[0], acc[0]);   acc[0] = fmaf(a.x, w[1], acc[0]); acc[0] = fmaf(a.y, w[2], acc[0]);
    acc[1] = fmaf(a.y, w[0], acc[1]); acc[1] = fmaf(a.z, w[1], acc[1]); acc[1] = fmaf(a.w, w[2], acc[1]);
    acc[2] = fmaf(a.w, w[0], acc[2]); acc[2] = fmaf(b.x, w[1], acc[2]); acc[2] = fmaf(b.y, w[2], acc[2]);
    acc[3] = fmaf(b.y, w[0], acc[3]); acc[3] = fmaf(b.z, w[1], acc[3]); acc[3] = fmaf(b.w, w[2], acc[3]);
}

template <int VEC>
__global__ void __launch_bounds__(256)
dw_stream_s2_kernel(const Shape s, const DwCfg c, const float* __restrict__ x, const uint32_t* __restrict__ packed,
                    float* __restrict__ y, Status* status, uint32_t tag) {
    const uint32_t tag_seen = __ldg(packed);
    const float* __restrict__ wpk = reinterpret_cast<const float*>(packed + kHeaderBytes / 4);
    const int lane = threadIdx.x & 31;
    const uint32_t warp_global = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int sub = lane / c.XQ;
    const int xq = lane - sub * c.XQ;
    const uint32_t item = warp_global * (uint32_t)c.subs + (uint32_t)sub;
    const bool live = (sub < c.subs) && (item < c.items);
    uint32_t plane_idx = 0, chunk = 0;
    c.div_chunks.divmod(live ? item : 0u, plane_idx, chunk);
    const int ch = (int)(plane_idx % (uint32_t)s.C_in);
    const float* __restrict__ xp = x + (size_t)plane_idx * s.H * s.W;
    float* __restrict__ yp = y + (size_t)plane_idx * s.H_out * s.W_out;
    const int col = xq * 8;                      // first of the 8 input columns of this strip
    const int p0 = (int)chunk * c.RH;
    const int p1 = min(p0 + c.RH, s.H_out);
    const bool has_l = xq > 0;
    const bool second_ok = col + 4 < s.W;        // the last strip of a row may have only one group of four columns
    float w[3][3];
#pragma unroll
    for (int i = 0; i < 9; ++i) w[i / 3][i % 3] = live ? __ldg(wpk + (size_t)ch * 9 + i) : 0.f;
    const float4 z4 = make_float4(0.f, 0.f, 0.f, 0.f);
    // input rows 2p-1, 2p, 2p+1 feed output row p; row 2p+1 is row 2(p+1)-1 of the next output
    float4 ta = live ? ldrow<VEC>(xp, 2 * p0 - 1, s.H, s.W, col) : z4;
    float4 tb = (live && second_ok) ? ldrow<VEC>(xp, 2 * p0 - 1, s.H, s.W, col + 4) : z4;
    float4 ca[2], cb[2], na[2], nb[2];
#pragma unroll
    for (int j = 0; j < 2; ++j) {
        ca[j] = live ? ldrow<VEC>(xp, 2 * p0 + j, s.H, s.W, col) : z4;
        cb[j] = (live && second_ok) ? ldrow<VEC>(xp, 2 * p0 + j, s.H, s.W, col + 4) : z4;
    }
    // the left halo of a row is fetched from the neighbouring lane once; the bottom row of one output is the top row of the next
    auto halo = [&](const float4 b) { const float v = __shfl_up_sync(0xffffffffu, b.w, 1); return has_l ? v : 0.f; };
    float lt = halo(tb), lc[2] = {halo(cb[0]), halo(cb[1])};
    for (int p = p0; p < p0 + c.RH; ++p) {
#pragma unroll
        for (int j = 0; j < 2; ++j) {                  // rows of the next output, in flight during this one's math
            const int h = 2 * (p + 1) + j;
            const bool need = live && (p + 1 < p1);
            na[j] = need ? ldrow<VEC>(xp, h, s.H, s.W, col) : z4;
            nb[j] = (need && second_ok) ? ldrow<VEC>(xp, h, s.H, s.W, col + 4) : z4;
        }
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        row_taps2(ta, tb, lt, w[0], acc);
        row_taps2(ca[0], cb[0], lc[0], w[1], acc);
        row_taps2(ca[1], cb[1], lc[1], w[2], acc);
        if (live && p < p1 && tag_seen == tag) {
            float* dst = yp + (size_t)p * s.W_out + xq * 4;
            if ((s.W_out & 3) == 0) {
                *reinterpret_cast<float4*>(dst) = make_float4(acc[0], acc[1], acc[2], acc[3]);
            } else if ((s.W_out & 1) == 0) {
                *reinterpret_cast<float2*>(dst) = make_float2(acc[0], acc[1]);
                if (xq * 4 + 2 < s.W_out) *reinterpret_cast<float2*>(dst + 2) = make_float2(acc[2], acc[3]);
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    if (xq * 4 + j < s.W_out) dst[j] = acc[j];
            }
        }
        ta = ca[1];
        tb = cb[1];
        lt = lc[1];
#pragma unroll
        for (int j = 0; j < 2; ++j) { ca[j] = na[j]; cb[j] = nb[j]; lc[j] = halo(nb[j]); }
    }
    if (tag_seen != tag && threadIdx.x == 0) record_status(status, GCONV_ERR_PACK_MISMATCH, (int)blockIdx.x);
}


// ---- 5x5 depthwise (pad 2) ----------------------------------------------------------------------------
// The same stream for 5x5 filters: a strip of four output columns reads eight (stride 2: eleven) input columns, its
// own aligned float4 (stride 2: two) plus two columns from the lane on the left and two (stride 2: one) from the lane
// on the right; five input rows feed an output row.  Sum order per output: (r, s) as in Algorithm 1.
__device__ __forceinline__ void row_taps5_s1(const float4 v, bool has_l, bool has_r, const float (&w)[5], float (&acc)[4]) {
    float l0 = __shfl_up_sync(0xffffffffu, v.z, 1), l1 = __shfl_up_sync(0xffffffffu, v.w, 1);
    float r0 = __shfl_down_sync(0xffffffffu, v.x, 1), r1 = __shfl_down_sync(0xffffffffu, v.y, 1);
    if (!has_l) { l0 = 0.f; l1 = 0.f; }
    if (!has_r) { r0 = 0.f; r1 = 0.f; }
    const float in[8] = {l0, l1, v.x, v.y, v.z, v.w, r0, r1};
#pragma unroll
    for (int j = 0; j < 4; ++j)
#pragma unroll
        for (int t = 0; t < 5; ++t) acc[j] = fmaf(in[j + t], w[t], acc[j]);
}
__device__ __forceinline__ void row_taps5_s2(const float4 a, const float4 b, bool has_l, bool has_r, const float (&w)[5],
                                             float (&acc)[4]) {
    float l0 = __shfl_up_sync(0xffffffffu, b.z, 1), l1 = __shfl_up_sync(0xffffffffu, b.w, 1);
    float r0 = __shfl_down_sync(0xffffffffu, a.x, 1);
    if (!has_l) { l0 = 0.f; l1 = 0.f; }
    if (!has_r) r0 = 0.f;
    const float in[11] = {l0, l1, a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w, r0};
#pragma unroll
    for (int j = 0; j < 4; ++j)
#pragma unroll
        for (int t = 0; t < 5; ++t) acc[j] = fmaf(in[2 * j + t], w[t], acc[j]);
}

template <int VEC, int STRIDE>
__global__ void __launch_bounds__(256)
dw5_stream_kernel(const Shape s, const DwCfg c, const float* __restrict__ x, const uint32_t* __restrict__ packed,
                  float* __restrict__ y, Status* status, uint32_t tag) {
    const uint32_t tag_seen = __ldg(packed);
    const float* __restrict__ wpk = reinterpret_cast<const float*>(packed + kHeaderBytes / 4);
    const int lane = threadIdx.x & 31;
    const uint32_t warp_global = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int sub = lane / c.XQ;
    const int xq = lane - sub * c.XQ;
    const uint32_t item = warp_global * (uint32_t)c.subs + (uint32_t)sub;
    const bool live = (sub < c.subs) && (item < c.items);
    uint32_t plane_idx = 0, chunk = 0;
    c.div_chunks.divmod(live ? item : 0u, plane_idx, chunk);
    const int ch = (int)(plane_idx % (uint32_t)s.C_in);
    const float* __restrict__ xp = x + (size_t)plane_idx * s.H * s.W;
    float* __restrict__ yp = y + (size_t)plane_idx * s.H_out * s.W_out;
    const int col = xq * 4 * STRIDE;             // first input column of this strip
    const int p0 = (int)chunk * c.RH;
    const int p1 = min(p0 + c.RH, s.H_out);
    const bool has_l = xq > 0, has_r = xq < c.XQ - 1;
    const bool second_ok = STRIDE == 2 && col + 4 < s.W;
    float w[5][5];
#pragma unroll
    for (int i = 0; i < 25; ++i) w[i / 5][i % 5] = live ? __ldg(wpk + (size_t)ch * 25 + i) : 0.f;
    const float4 z4 = make_float4(0.f, 0.f, 0.f, 0.f);
    // input rows STRIDE*p - 2 .. STRIDE*p + 2 feed output row p; STRIDE new rows per output row
    float4 ra[5], rb[5], na[STRIDE], nb[STRIDE];
#pragma unroll
    for (int j = 0; j < 5; ++j) {
        ra[j] = live ? ldrow<VEC>(xp, STRIDE * p0 - 2 + j, s.H, s.W, col) : z4;
        rb[j] = (live && second_ok) ? ldrow<VEC>(xp, STRIDE * p0 - 2 + j, s.H, s.W, col + 4) : z4;
    }
    for (int p = p0; p < p0 + c.RH; ++p) {       // warp-uniform trip count
#pragma unroll
        for (int j = 0; j < STRIDE; ++j) {         // the next output row's new input rows, in flight during this row's math
            const int h = STRIDE * (p + 1) + 3 - STRIDE + j;
            const bool need = live && (p + 1 < p1);
            na[j] = need ? ldrow<VEC>(xp, h, s.H, s.W, col) : z4;
            nb[j] = (need && second_ok) ? ldrow<VEC>(xp, h, s.H, s.W, col + 4) : z4;
        }
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int r = 0; r < 5; ++r) {
            if constexpr (STRIDE == 1) row_taps5_s1(ra[r], has_l, has_r, w[r], acc);
            else row_taps5_s2(ra[r], rb[r], has_l, has_r, w[r], acc);
        }
        if (live && p < p1 && tag_seen == tag) {
            float* dst = yp + (size_t)p * s.W_out + xq * 4;
            if ((s.W_out & 3) == 0) {
                *reinterpret_cast<float4*>(dst) = make_float4(acc[0], acc[1], acc[2], acc[3]);
            } else if ((s.W_out & 1) == 0) {
                *reinterpret_cast<float2*>(dst) = make_float2(acc[0], acc[1]);
                if (xq * 4 + 2 < s.W_out) *reinterpret_cast<float2*>(dst + 2) = make_float2(acc[2], acc[3]);
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    if (xq * 4 + j < s.W_out) dst[j] = acc[j];
            }
        }
#pragma unroll
        for (int j = 0; j + STRIDE < 5; ++j) { ra[j] = ra[j + STRIDE]; rb[j] = rb[j + STRIDE]; }
#pragma unroll
        for (int j = 0; j < STRIDE; ++j) { ra[5 - STRIDE + j] = na[j]; rb[5 - STRIDE + j] = nb[j]; }
    }
    if (tag_seen != tag && threadIdx.x == 0) record_status(status, GCONV_ERR_PACK_MISMATCH, (int)blockIdx.x);
}

// 5x5, stride 1: U5 output rows per block, the raw input rows of the next two blocks in flight during the block's
// math (four 16-byte loads per thread).  An input row feeds five output rows, so its eight-column window (own four
// columns plus two from each neighbouring lane) is built once, when the row enters the block, and kept in registers:
// four shuffles per input row instead of twenty.
constexpr int U5 = 2;   // output rows per block of the 5x5 kernel
constexpr int D5 = 4;   // raw rows in flight beyond the current block
template <int VEC>
__global__ void __launch_bounds__(256, 2)
dw5_stream_s1_kernel(const Shape s, const DwCfg c, const float* __restrict__ x, const uint32_t* __restrict__ packed,
                     float* __restrict__ y, Status* status, uint32_t tag) {
    const uint32_t tag_seen = __ldg(packed);
    const float* __restrict__ wpk = reinterpret_cast<const float*>(packed + kHeaderBytes / 4);
    const int lane = threadIdx.x & 31;
    const uint32_t warp_global = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int sub = lane / c.XQ;
    const int xq = lane - sub * c.XQ;
    const uint32_t item = warp_global * (uint32_t)c.subs + (uint32_t)sub;
    const bool live = (sub < c.subs) && (item < c.items);
    uint32_t plane_idx = 0, chunk = 0;
    c.div_chunks.divmod(live ? item : 0u, plane_idx, chunk);
    const int ch = (int)(plane_idx % (uint32_t)s.C_in);
    const float* __restrict__ xp = x + (size_t)plane_idx * s.H * s.W;
    float* __restrict__ yp = y + (size_t)plane_idx * s.H * s.W;
    const int col = xq * 4;
    const int p0 = (int)chunk * c.RH;
    const int p1 = min(p0 + c.RH, s.H);
    const bool has_l = xq > 0, has_r = xq < c.XQ - 1;
    const float4 z4 = make_float4(0.f, 0.f, 0.f, 0.f);
    // rows p0-2 .. p0+U5+1 fill the first block's windows, rows up to p0+U5+1+D5 wait in the queue; row h is needed
    // only if it feeds an output row of this strip (h <= p1+1)
    float4 first[U5 + 4], queue[D5];
#pragma unroll
    for (int j = 0; j < U5 + 4; ++j) first[j] = live ? ldrow<VEC>(xp, p0 - 2 + j, s.H, s.W, col) : z4;
#pragma unroll
    for (int j = 0; j < D5; ++j) {
        const int h = p0 + U5 + 2 + j;
        queue[j] = (live && h <= p1 + 1) ? ldrow<VEC>(xp, h, s.H, s.W, col) : z4;
    }
    float w[5][5];
#pragma unroll
    for (int i = 0; i < 25; ++i) w[i / 5][i % 5] = live ? __ldg(wpk + (size_t)ch * 25 + i) : 0.f;
    auto widen = [&](const float4 v, float (&o)[8]) {   // every lane runs the shuffles; `live` only gates memory traffic
        const float l0 = __shfl_up_sync(0xffffffffu, v.z, 1), l1 = __shfl_up_sync(0xffffffffu, v.w, 1);
        const float r0 = __shfl_down_sync(0xffffffffu, v.x, 1), r1 = __shfl_down_sync(0xffffffffu, v.y, 1);
        o[0] = has_l ? l0 : 0.f;
        o[1] = has_l ? l1 : 0.f;
        o[2] = v.x; o[3] = v.y; o[4] = v.z; o[5] = v.w;
        o[6] = has_r ? r0 : 0.f;
        o[7] = has_r ? r1 : 0.f;
    };
    float win[U5 + 4][8];                              // input rows p-2 .. p+U5+1 of the current block
#pragma unroll
    for (int j = 0; j < U5 + 4; ++j) widen(first[j], win[j]);
    for (int p = p0; p < p0 + c.RH; p += U5) {         // warp-uniform trip count
        float4 fresh[U5];
#pragma unroll
        for (int j = 0; j < U5; ++j) {
            const int h = p + U5 + 2 + D5 + j;
            fresh[j] = (live && h <= p1 + 1) ? ldrow<VEC>(xp, h, s.H, s.W, col) : z4;
        }
#pragma unroll
        for (int j = 0; j < U5; ++j) {
            float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int r = 0; r < 5; ++r)
#pragma unroll
                for (int q = 0; q < 4; ++q)
#pragma unroll
                    for (int t = 0; t < 5; ++t) acc[q] = fmaf(win[j + r][q + t], w[r][t], acc[q]);
            if (live && p + j < p1 && tag_seen == tag) strow<VEC>(yp + (size_t)(p + j) * s.W + col, col, s.W, acc);
        }
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
            for (int i = 0; i < 8; ++i) win[j][i] = win[j + U5][i];
#pragma unroll
        for (int j = 0; j < U5; ++j) widen(queue[j], win[4 + j]);
#pragma unroll
        for (int j = 0; j + U5 < D5; ++j) queue[j] = queue[j + U5];
#pragma unroll
        for (int j = 0; j < U5; ++j) queue[D5 - U5 + j] = fresh[j];
    }
    if (tag_seen != tag && threadIdx.x == 0) record_status(status, GCONV_ERR_PACK_MISMATCH, (int)blockIdx.x);
}

}  // namespace

bool dw_supported(const Shape& s) {
    if (!s.square()) return false;   // one stride, padding and dilation for both axes
    const bool k3 = s.KH == 3 && s.KW == 3 && s.pad == 1, k5 = s.KH == 5 && s.KW == 5 && s.pad == 2;
    if (!((k3 || k5) && s.dilation == 1 && (s.stride == 1 || s.stride == 2))) return false;
    if (!(s.Cg == 1 && s.Kg == 1)) return false;
    const int xq = s.stride == 1 ? (s.W + 3) / 4 : (s.W + 7) / 8;
    if (xq > 32) return false;
    return (unsigned long long)s.N * s.C_in * s.H_out < (1ull << 30);
}

DwCfg dw_config(const Shape& s, int sm_count) {
    DwCfg c;
    c.XQ = s.stride == 1 ? (s.W + 3) / 4 : (s.W + 7) / 8;
    c.subs = 32 / c.XQ;
    // rows per thread: long strips amortise the two halo rows, short ones give more parallelism; aim for
    // at least ~6 waves of 1024 threads per SM.  5x5: four halo rows per strip and 25 FMAs per output make the strip
    // length matter more than the thread count (measured): split only below ~0.4 waves.
    const long long planes = (long long)s.N * s.C_in;
    const long long want = s.KH == 5 ? 410LL * sm_count : 6LL * 1024 * sm_count;
    int rh = s.H_out;
    if (s.KH == 3 && s.stride == 1 && s.H_out >= 28) {
        // 3x3 stride 1 on planes of 28 rows and more: strips of 28 rows measured best at 28x28, 56x56 and 112x112
        // (7 % halo rows, long enough to amortise the set-up) as long as about half a wave of lanes remains
        rh = 28;
        while (rh > 8 && planes * ((s.H_out + rh - 1) / rh) * c.XQ < 512LL * sm_count) rh = (rh + 1) / 2;
    } else {
        while (rh > 8 && planes * ((s.H_out + rh - 1) / rh) * c.XQ < want) rh = (rh + 1) / 2;
        if (s.KH == 3 && s.stride == 1 && s.H_out <= 8 && planes * c.XQ * 2 >= 512LL * sm_count) rh = 4;   // 7x7, 8x8: two short strips
    }
    rh = ((rh + U - 1) / U) * U;
    c.RH = rh;
    c.chunks = (s.H_out + rh - 1) / rh;
    c.div_chunks = make_fastdiv((uint32_t)c.chunks);
    c.items = (uint32_t)(planes * c.chunks);
    const uint32_t warps = (c.items + c.subs - 1) / c.subs;
    c.blocks = (warps + 7) / 8;
    return c;
}

cudaError_t dw_forward(const Shape& s, const float* x, const void* packed, float* y, Status* status, int sm_count,
                       cudaStream_t st) {
    // small planes go through shared memory in batches of whole planes (direct_dw_plane.cu); 3x3 stride 1 on 28x28 planes
    // measured the same on both kernels (16.5 us on 192 planes, N = 64) and stays on the stream
    if (dw_plane_supported(s) && !(s.KH == 3 && s.stride == 1 && s.W == 28)) return dw_plane_forward(s, x, packed, y, status, sm_count, st);
    const DwCfg c = dw_config(s, sm_count);
    const uint32_t tag = pack_tag(s, GCONV_VARIANT_DIRECT_TILED);
    const uint32_t* pk = reinterpret_cast<const uint32_t*>(packed);
    const int vec = s.W % 4 == 0 ? 4 : (s.W % 2 == 0 ? 2 : 0);
#define GCONV_DW_LAUNCH(KERNEL) \
    do { \
        if (vec == 4) KERNEL(4); else if (vec == 2) KERNEL(2); else KERNEL(0); \
    } while (0)
#define GCONV_DW5_S1(V) dw5_stream_s1_kernel<V><<<c.blocks, 256, 0, st>>>(s, c, x, pk, y, status, tag)
#define GCONV_DW5_S2(V) dw5_stream_kernel<V, 2><<<c.blocks, 256, 0, st>>>(s, c, x, pk, y, status, tag)
#define GCONV_DW3_S1(V) \
    do { \
        if (s.H_out >= 28) dw_stream_s1_kernel<V, 4><<<c.blocks, 256, 0, st>>>(s, c, x, pk, y, status, tag); \
        else dw_stream_s1_kernel<V, 2><<<c.blocks, 256, 0, st>>>(s, c, x, pk, y, status, tag); \
    } while (0)
#define GCONV_DW3_S2(V) dw_stream_s2_kernel<V><<<c.blocks, 256, 0, st>>>(s, c, x, pk, y, status, tag)
    if (s.KH == 5) {
        if (s.stride == 1) GCONV_DW_LAUNCH(GCONV_DW5_S1);
        else GCONV_DW_LAUNCH(GCONV_DW5_S2);
    } else if (s.stride == 1) {
        GCONV_DW_LAUNCH(GCONV_DW3_S1);
    } else {
        GCONV_DW_LAUNCH(GCONV_DW3_S2);
    }
#undef GCONV_DW_LAUNCH
#undef GCONV_DW5_S1
#undef GCONV_DW5_S2
#undef GCONV_DW3_S1
#undef GCONV_DW3_S2
    return cudaGetLastError();
}

}  // namespace gconv
