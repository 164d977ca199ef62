// Internal declarations shared by the host API and the kernel translation units of libgconv.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/gconv.h"

namespace gconv {

constexpr int kHeaderBytes = 64;  // packed-weight blob header; keeps the payload 16-byte aligned
constexpr uint32_t kMagic = 0x47434e56u;  // "GCNV"

struct Shape {
    int N, C_in, H, W, C_out, KH, KW, stride, pad, dilation, groups;
    int Cg, Kg, H_out, W_out;
};

// Device status block: word 0 = first error recorded by a kernel (0 = none), word 1 = detail.
struct Status {
    int code;
    int detail;
    int pad[2];
};

// Tag stored in word 0 of the packed blob; forward kernels compare it before touching the payload.
__host__ __device__ inline uint32_t pack_tag(const Shape& s, int variant) {
    uint32_t h = kMagic;
    const int v[7] = {variant, s.C_out, s.Cg, s.KH, s.KW, s.groups, s.Kg};
    for (int i = 0; i < 7; ++i) {
        h ^= (uint32_t)v[i] + 0x9e3779b9u + (h << 6) + (h >> 2);
    }
    return h;
}

__device__ inline void record_status(Status* st, int code, int detail) {
    if (atomicCAS(&st->code, 0, code) == 0) st->detail = detail;
}

// ---- per-variant entry points (host side launchers) --------------------------------------------
size_t generic_packed_bytes(const Shape& s);
cudaError_t generic_pack(const Shape& s, const float* w, void* packed, cudaStream_t st);
cudaError_t generic_forward(const Shape& s, const float* x, const void* packed, float* y, Status* status,
                            int sm_count, cudaStream_t st);

}  // namespace gconv
