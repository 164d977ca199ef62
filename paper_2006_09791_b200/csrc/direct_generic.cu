// Variant DIRECT_GENERIC: FP32 FFMA direct grouped convolution, one thread per output element.
// Handles every shape the descriptor accepts (any kernel size; stride, padding and dilation per axis); it is
// the safety net of the selector, not a fast path.  Grouped convolution of Section II of the paper,
// summed in the (c, r, s) order of the convolution stage of Algorithm 1.
#include "gconv_internal.h"

namespace gconv {

size_t generic_packed_bytes(const Shape& s) {
    return kHeaderBytes + sizeof(float) * (size_t)s.C_out * s.Cg * s.KH * s.KW;
}

__global__ void generic_pack_kernel(const float* __restrict__ w, uint32_t* __restrict__ packed, size_t n, uint32_t tag) {
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i == 0) {
        packed[0] = tag;
        for (int j = 1; j < kHeaderBytes / 4; ++j) packed[j] = 0;
    }
    float* dst = reinterpret_cast<float*>(packed + kHeaderBytes / 4);
    for (; i < n; i += (size_t)gridDim.x * blockDim.x) dst[i] = w[i];
}

cudaError_t generic_pack(const Shape& s, const float* w, void* packed, cudaStream_t st) {
    size_t n = (size_t)s.C_out * s.Cg * s.KH * s.KW;
    int blocks = (int)((n + 255) / 256 < 1184 ? (n + 255) / 256 : 1184);
    generic_pack_kernel<<<blocks, 256, 0, st>>>(w, reinterpret_cast<uint32_t*>(packed), n,
                                                pack_tag(s, GCONV_VARIANT_DIRECT_GENERIC));
    return cudaGetLastError();
}

__global__ void __launch_bounds__(256)
generic_forward_kernel(Shape s, const float* __restrict__ x, const uint32_t* __restrict__ packed,
                       float* __restrict__ y, Status* status, uint32_t tag) {
    if (packed[0] != tag) {
        if (threadIdx.x == 0) record_status(status, GCONV_ERR_PACK_MISMATCH, (int)blockIdx.x);
        return;
    }
    const float* __restrict__ w = reinterpret_cast<const float*>(packed + kHeaderBytes / 4);
    const size_t total = (size_t)s.N * s.C_out * s.H_out * s.W_out;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const int q = (int)(i % s.W_out);
        size_t t = i / s.W_out;
        const int p = (int)(t % s.H_out);
        t /= s.H_out;
        const int ko = (int)(t % s.C_out);
        const int n = (int)(t / s.C_out);
        const int g = ko / s.Kg;
        const float* xg = x + ((size_t)n * s.C_in + (size_t)g * s.Cg) * s.H * s.W;
        const float* wk = w + (size_t)ko * s.Cg * s.KH * s.KW;
        float acc = 0.f;
        for (int c = 0; c < s.Cg; ++c) {
            for (int r = 0; r < s.KH; ++r) {
                const int h = p * s.stride + r * s.dilation - s.pad;
                if (h < 0 || h >= s.H) continue;
                for (int ss = 0; ss < s.KW; ++ss) {
                    const int v = q * s.stride_w + ss * s.dilation_w - s.pad_w;
                    if (v < 0 || v >= s.W) continue;
                    acc = fmaf(__ldg(xg + ((size_t)c * s.H + h) * s.W + v), __ldg(wk + (c * s.KH + r) * s.KW + ss), acc);
                }
            }
        }
        y[i] = acc;
    }
}

cudaError_t generic_forward(const Shape& s, const float* x, const void* packed, float* y, Status* status,
                            int sm_count, cudaStream_t st) {
    const size_t total = (size_t)s.N * s.C_out * s.H_out * s.W_out;
    size_t want = (total + 255) / 256;
    size_t cap = (size_t)sm_count * 8 * 4;
    int blocks = (int)(want < cap ? want : cap);
    generic_forward_kernel<<<blocks, 256, 0, st>>>(s, x, reinterpret_cast<const uint32_t*>(packed), y, status,
                                                   pack_tag(s, GCONV_VARIANT_DIRECT_GENERIC));
    return cudaGetLastError();
}

}  // namespace gconv
