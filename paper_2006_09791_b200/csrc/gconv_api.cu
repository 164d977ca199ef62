// Host side of libgconv: descriptor, validation, variant selection and the C ABI of include/gconv.h.
#include <new>

#include "gconv_internal.h"

using namespace gconv;

namespace {

bool variant_supported(const Shape& s, int v) {
    switch (v) {
        case GCONV_VARIANT_DIRECT_GENERIC:
            return true;
        case GCONV_VARIANT_DIRECT_TILED:
            return tiled_supported(s);
        case GCONV_VARIANT_IGEMM_TF32:
            return igemm_supported(s);
        default:
            return false;
    }
}

// Variant selector.  Keyed on (Cg, Kg, H*W, N) like the tile-size choice the paper leaves to
// autotuning (Section III-C); the thresholds come from measured timings of the forced variants.
int select_variant(const Shape& s) {
    if (igemm_supported(s) && s.Cg >= 2) return GCONV_VARIANT_IGEMM_TF32;
    if (tiled_supported(s)) return GCONV_VARIANT_DIRECT_TILED;
    return GCONV_VARIANT_DIRECT_GENERIC;
}

int fail_cuda(gconv_desc* d, cudaError_t e) {
    d->last_cuda_error = (int)e;
    (void)cudaGetLastError();  // clear the sticky-free error state
    return GCONV_ERR_CUDA;
}

int ensure_device_state(gconv_desc* d) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return fail_cuda(d, e);
    if (d->status_dev != nullptr && d->device == dev) return GCONV_OK;
    if (d->status_dev != nullptr) {
        cudaFree(d->status_dev);
        d->status_dev = nullptr;
    }
    if (d->scratch != nullptr) {
        cudaFree(d->scratch);
        d->scratch = nullptr;
        d->scratch_bytes = 0;
    }
    e = cudaDeviceGetAttribute(&d->sm_count, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return fail_cuda(d, e);
    e = cudaMalloc(&d->status_dev, sizeof(Status));
    if (e != cudaSuccess) return fail_cuda(d, e);
    e = cudaMemset(d->status_dev, 0, sizeof(Status));
    if (e != cudaSuccess) return fail_cuda(d, e);
    d->device = dev;
    return GCONV_OK;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

extern "C" {

int gconv_desc_create(gconv_desc_t* out, int N, int C_in, int H, int W, int C_out, int KH, int KW, int stride,
                      int pad, int dilation, int groups) {
    if (out == nullptr) return GCONV_ERR_NULL;
    *out = nullptr;
    if (N < 1 || C_in < 1 || H < 1 || W < 1 || C_out < 1 || KH < 1 || KW < 1) return GCONV_ERR_INVALID_ARG;
    if (stride < 1 || pad < 0 || dilation < 1 || groups < 1) return GCONV_ERR_INVALID_ARG;
    if (C_in % groups != 0 || C_out % groups != 0) return GCONV_ERR_INVALID_ARG;
    const long long span_h = (long long)H + 2LL * pad - (long long)dilation * (KH - 1) - 1;
    const long long span_w = (long long)W + 2LL * pad - (long long)dilation * (KW - 1) - 1;
    if (span_h < 0 || span_w < 0) return GCONV_ERR_INVALID_ARG;
    Shape s;
    s.N = N; s.C_in = C_in; s.H = H; s.W = W; s.C_out = C_out; s.KH = KH; s.KW = KW;
    s.stride = stride; s.pad = pad; s.dilation = dilation; s.groups = groups;
    s.Cg = C_in / groups;
    s.Kg = C_out / groups;
    s.H_out = (int)(span_h / stride) + 1;
    s.W_out = (int)(span_w / stride) + 1;
    const double lim = 1099511627776.0;  // 2^40 elements
    if ((double)N * C_in * H * W > lim || (double)N * C_out * s.H_out * s.W_out > lim ||
        (double)C_out * s.Cg * KH * KW > 2147483647.0 || (long long)H * W > 2147483647LL || pad > (1 << 20))
        return GCONV_ERR_INVALID_ARG;
    gconv_desc* d = new (std::nothrow) gconv_desc();
    if (d == nullptr) return GCONV_ERR_INVALID_ARG;
    d->s = s;
    d->variant = select_variant(s);
    d->forced = 0;
    d->status_dev = nullptr;
    d->device = -1;
    d->sm_count = 0;
    d->last_cuda_error = 0;
    d->scratch = nullptr;
    d->scratch_bytes = 0;
    *out = d;
    return GCONV_OK;
}

int gconv_desc_destroy(gconv_desc_t d) {
    if (d == nullptr) return GCONV_OK;
    if (d->status_dev != nullptr) cudaFree(d->status_dev);
    if (d->scratch != nullptr) cudaFree(d->scratch);
    delete d;
    return GCONV_OK;
}

int gconv_out_shape(gconv_desc_t d, int* H_out, int* W_out) {
    if (d == nullptr || H_out == nullptr || W_out == nullptr) return GCONV_ERR_NULL;
    *H_out = d->s.H_out;
    *W_out = d->s.W_out;
    return GCONV_OK;
}

long long gconv_macs(gconv_desc_t d) {
    if (d == nullptr) return -1;
    const Shape& s = d->s;
    return (long long)s.N * s.C_out * s.H_out * s.W_out * s.Cg * s.KH * s.KW;
}

size_t gconv_packed_bytes(gconv_desc_t d) {
    if (d == nullptr) return 0;
    switch (d->variant) {
        case GCONV_VARIANT_DIRECT_TILED:
            return tiled_packed_bytes(d->s);
        case GCONV_VARIANT_IGEMM_TF32:
            return igemm_packed_bytes(d->s);
        case GCONV_VARIANT_DIRECT_GENERIC:
        default:
            return generic_packed_bytes(d->s);
    }
}

int gconv_variant(gconv_desc_t d) { return d == nullptr ? -1 : d->variant; }

int gconv_variant_supported(gconv_desc_t d, int variant) {
    if (d == nullptr) return 0;
    return variant_supported(d->s, variant) ? 1 : 0;
}

int gconv_desc_set_variant(gconv_desc_t d, int variant) {
    if (d == nullptr) return GCONV_ERR_NULL;
    if (variant == GCONV_VARIANT_AUTO) {
        d->variant = select_variant(d->s);
        d->forced = 0;
        return GCONV_OK;
    }
    if (variant < GCONV_VARIANT_DIRECT_GENERIC || variant > GCONV_VARIANT_IGEMM_TF32) return GCONV_ERR_INVALID_ARG;
    if (!variant_supported(d->s, variant)) return GCONV_ERR_UNSUPPORTED;
    d->variant = variant;
    d->forced = 1;
    return GCONV_OK;
}

int gconv_pack_weights(gconv_desc_t d, const float* w_ochw, void* w_packed, void* stream) {
    if (d == nullptr || w_ochw == nullptr || w_packed == nullptr) return GCONV_ERR_NULL;
    if (!aligned16(w_ochw) || !aligned16(w_packed)) return GCONV_ERR_ALIGNMENT;
    int rc = ensure_device_state(d);
    if (rc != GCONV_OK) return rc;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    cudaError_t e;
    switch (d->variant) {
        case GCONV_VARIANT_DIRECT_TILED:
            e = tiled_pack(d->s, w_ochw, w_packed, st);
            break;
        case GCONV_VARIANT_IGEMM_TF32:
            e = igemm_pack(d->s, w_ochw, w_packed, st);
            break;
        case GCONV_VARIANT_DIRECT_GENERIC:
        default:
            e = generic_pack(d->s, w_ochw, w_packed, st);
            break;
    }
    return e == cudaSuccess ? GCONV_OK : fail_cuda(d, e);
}

int gconv_forward(gconv_desc_t d, const float* x, const void* w_packed, float* y, void* stream) {
    if (d == nullptr || x == nullptr || w_packed == nullptr || y == nullptr) return GCONV_ERR_NULL;
    if (!aligned16(x) || !aligned16(w_packed) || !aligned16(y)) return GCONV_ERR_ALIGNMENT;
    int rc = ensure_device_state(d);
    if (rc != GCONV_OK) return rc;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    cudaError_t e;
    switch (d->variant) {
        case GCONV_VARIANT_DIRECT_TILED:
            e = tiled_forward(d->s, x, w_packed, y, d->status_dev, d->sm_count, st);
            break;
        case GCONV_VARIANT_IGEMM_TF32: {
            const size_t need = igemm_scratch_bytes(d->s);
            if (need > d->scratch_bytes) {   // first forward of a layer that runs on a padded copy of x
                if (d->scratch != nullptr) cudaFree(d->scratch);
                d->scratch = nullptr;
                d->scratch_bytes = 0;
                e = cudaMalloc(&d->scratch, need);
                if (e != cudaSuccess) return fail_cuda(d, e);
                d->scratch_bytes = need;
            }
            e = igemm_forward(d->s, x, w_packed, y, d->status_dev, d->sm_count, st, d->scratch);
            break;
        }
        case GCONV_VARIANT_DIRECT_GENERIC:
        default:
            e = generic_forward(d->s, x, w_packed, y, d->status_dev, d->sm_count, st);
            break;
    }
    return e == cudaSuccess ? GCONV_OK : fail_cuda(d, e);
}

int gconv_forward_host(gconv_desc_t d, const float* x_host, const void* w_packed, float* y_host, float* x_stage,
                       float* y_stage, void* stream) {
    if (d == nullptr || x_host == nullptr || y_host == nullptr || x_stage == nullptr || y_stage == nullptr)
        return GCONV_ERR_NULL;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    const Shape& s = d->s;
    const size_t xb = sizeof(float) * (size_t)s.N * s.C_in * s.H * s.W;
    const size_t yb = sizeof(float) * (size_t)s.N * s.C_out * s.H_out * s.W_out;
    cudaError_t e = cudaMemcpyAsync(x_stage, x_host, xb, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return fail_cuda(d, e);
    int rc = gconv_forward(d, x_stage, w_packed, y_stage, stream);
    if (rc != GCONV_OK) return rc;
    e = cudaMemcpyAsync(y_host, y_stage, yb, cudaMemcpyDeviceToHost, st);
    if (e != cudaSuccess) return fail_cuda(d, e);
    return GCONV_OK;
}

int gconv_block_supported(gconv_desc_t d, int C2) { return (d != nullptr && igemm_block_supported(d->s, C2)) ? 1 : 0; }

size_t gconv_block_packed_bytes(gconv_desc_t d, int C2) {
    return (d != nullptr && igemm_block_supported(d->s, C2)) ? igemm_block_packed_bytes(d->s, C2) : 0;
}

int gconv_block_pack_weights(gconv_desc_t d, int C2, const float* w_ochw, const float* w2, void* w_packed, void* stream) {
    if (d == nullptr || w_ochw == nullptr || w2 == nullptr || w_packed == nullptr) return GCONV_ERR_NULL;
    if (!aligned16(w_ochw) || !aligned16(w2) || !aligned16(w_packed)) return GCONV_ERR_ALIGNMENT;
    if (!igemm_block_supported(d->s, C2)) return GCONV_ERR_UNSUPPORTED;
    int rc = ensure_device_state(d);
    if (rc != GCONV_OK) return rc;
    const cudaError_t e = igemm_block_pack(d->s, C2, w_ochw, w2, w_packed, reinterpret_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? GCONV_OK : fail_cuda(d, e);
}

int gconv_block_forward(gconv_desc_t d, int C2, const float* x, const void* w_packed, float* y2, void* stream) {
    if (d == nullptr || x == nullptr || w_packed == nullptr || y2 == nullptr) return GCONV_ERR_NULL;
    if (!aligned16(x) || !aligned16(w_packed) || !aligned16(y2)) return GCONV_ERR_ALIGNMENT;
    if (!igemm_block_supported(d->s, C2)) return GCONV_ERR_UNSUPPORTED;
    int rc = ensure_device_state(d);
    if (rc != GCONV_OK) return rc;
    const cudaError_t e = igemm_block_forward(d->s, C2, x, w_packed, y2, d->status_dev, d->sm_count, reinterpret_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? GCONV_OK : fail_cuda(d, e);
}

int gconv_forward_launches(gconv_desc_t d) {
    if (d == nullptr) return 0;
    return (d->variant == GCONV_VARIANT_IGEMM_TF32 && igemm_scratch_bytes(d->s) > 0) ? 2 : 1;
}

int gconv_last_status(gconv_desc_t d, void* stream) {
    if (d == nullptr) return GCONV_ERR_NULL;
    cudaError_t e = cudaStreamSynchronize(reinterpret_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return fail_cuda(d, e);
    if (d->status_dev == nullptr) return GCONV_OK;
    Status h;
    e = cudaMemcpy(&h, d->status_dev, sizeof(Status), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return fail_cuda(d, e);
    if (h.code != 0) {
        e = cudaMemset(d->status_dev, 0, sizeof(Status));
        if (e != cudaSuccess) return fail_cuda(d, e);
    }
    return h.code;
}

int gconv_last_cuda_error(gconv_desc_t d) { return d == nullptr ? 0 : d->last_cuda_error; }

const char* gconv_status_string(int status) {
    switch (status) {
        case GCONV_OK: return "ok";
        case GCONV_ERR_NULL: return "null pointer argument";
        case GCONV_ERR_INVALID_ARG: return "invalid shape argument";
        case GCONV_ERR_UNSUPPORTED: return "variant does not support this shape";
        case GCONV_ERR_ALIGNMENT: return "device pointer not 16-byte aligned";
        case GCONV_ERR_CUDA: return "CUDA call failed";
        case GCONV_ERR_PACK_MISMATCH: return "packed weights do not match the descriptor";
        case GCONV_ERR_TIMEOUT: return "bounded wait inside a kernel ran out";
        case GCONV_ERR_TOO_LARGE: return "layer larger than the static scratch (x and y must fit in 16 MiB)";
        default: return "unknown status";
    }
}

const char* gconv_variant_name(int variant) {
    switch (variant) {
        case GCONV_VARIANT_AUTO: return "auto";
        case GCONV_VARIANT_DIRECT_GENERIC: return "direct_generic";
        case GCONV_VARIANT_DIRECT_TILED: return "direct_tiled";
        case GCONV_VARIANT_IGEMM_TF32: return "igemm_tf32";
        default: return "unknown";
    }
}

}  // extern "C"
