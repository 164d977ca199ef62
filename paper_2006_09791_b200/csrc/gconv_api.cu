// Host side of libgconv: descriptor, validation, variant selection and the C ABI of include/gconv.h.
#include <atomic>
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

// Counts weight-packing calls of the whole process.  The tensor-core kernel reads packed weights before its
// programmatic dependency wait, which is only safe once the packing kernel is known to have completed: a descriptor
// whose last forward saw an older count launches its next forward as an ordinary (fully serialized) kernel.
std::atomic<unsigned long long> g_pack_epoch{1};

// Variant selector.  The paper leaves the per-layer choice (its tile sizes) to autotuning (Section III-C); here the
// measured timings of the forced variants reduce to a rule on the group width alone: the tensor-core variant wherever
// it supports the shape and a group has at least two channels (narrower groups are merged into block-diagonal ones),
// the FP32 stream/tiled kernels for depthwise and for 3x3 shapes it rejects, the generic kernel for the rest.  The
// choices that do depend on (Cg, Kg, H*W, N) -- tiling, filter tile, resident or streamed weights, launch shape --
// are made inside the tensor-core variant's configuration.
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

IgemmLaunchOpts launch_opts(gconv_desc* d) {
    IgemmLaunchOpts o;
    const unsigned long long epoch = g_pack_epoch.load(std::memory_order_relaxed);
    o.pdl = d->pack_epoch_seen == epoch;
    d->pack_epoch_seen = epoch;
    o.wait_us = (uint32_t)d->wait_us;
    o.dbg_skip = d->dbg_skip;
    return o;
}

}  // namespace

extern "C" {

int gconv_desc_create_2d(gconv_desc_t* out, int N, int C_in, int H, int W, int C_out, int KH, int KW, int stride_h,
                         int stride_w, int pad_h, int pad_w, int dilation_h, int dilation_w, int groups) {
    if (out == nullptr) return GCONV_ERR_NULL;
    *out = nullptr;
    if (N < 1 || C_in < 1 || H < 1 || W < 1 || C_out < 1 || KH < 1 || KW < 1) return GCONV_ERR_INVALID_ARG;
    if (stride_h < 1 || stride_w < 1 || pad_h < 0 || pad_w < 0 || dilation_h < 1 || dilation_w < 1 || groups < 1)
        return GCONV_ERR_INVALID_ARG;
    if (C_in % groups != 0 || C_out % groups != 0) return GCONV_ERR_INVALID_ARG;
    const long long span_h = (long long)H + 2LL * pad_h - (long long)dilation_h * (KH - 1) - 1;
    const long long span_w = (long long)W + 2LL * pad_w - (long long)dilation_w * (KW - 1) - 1;
    if (span_h < 0 || span_w < 0) return GCONV_ERR_INVALID_ARG;
    Shape s;
    s.N = N; s.C_in = C_in; s.H = H; s.W = W; s.C_out = C_out; s.KH = KH; s.KW = KW;
    s.stride = stride_h; s.pad = pad_h; s.dilation = dilation_h; s.groups = groups;
    s.stride_w = stride_w; s.pad_w = pad_w; s.dilation_w = dilation_w;
    s.Cg = C_in / groups;
    s.Kg = C_out / groups;
    s.H_out = (int)(span_h / stride_h) + 1;
    s.W_out = (int)(span_w / stride_w) + 1;
    const double lim = 1099511627776.0;  // 2^40 elements
    if ((double)N * C_in * H * W > lim || (double)N * C_out * s.H_out * s.W_out > lim ||
        (double)C_out * s.Cg * KH * KW > 2147483647.0 || (long long)H * W > 2147483647LL || pad_h > (1 << 20) ||
        pad_w > (1 << 20))
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
    d->last_detail = 0;
    d->workspace = nullptr;
    d->workspace_bytes = 0;
    d->pack_epoch_seen = 0;
    d->wait_us = 0;
    d->dbg_skip = -1;
    *out = d;
    return GCONV_OK;
}

int gconv_desc_create(gconv_desc_t* out, int N, int C_in, int H, int W, int C_out, int KH, int KW, int stride,
                      int pad, int dilation, int groups) {
    return gconv_desc_create_2d(out, N, C_in, H, W, C_out, KH, KW, stride, stride, pad, pad, dilation, dilation, groups);
}

int gconv_desc_destroy(gconv_desc_t d) {
    if (d == nullptr) return GCONV_OK;
    if (d->status_dev != nullptr) cudaFree(d->status_dev);
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
    g_pack_epoch.fetch_add(1, std::memory_order_relaxed);
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
            if (need > 0 && (d->workspace == nullptr || d->workspace_bytes < need)) return GCONV_ERR_WORKSPACE;
            e = igemm_forward(d->s, x, w_packed, y, d->status_dev, d->sm_count, st, need > 0 ? d->workspace : nullptr, launch_opts(d));
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
    g_pack_epoch.fetch_add(1, std::memory_order_relaxed);
    const cudaError_t e = igemm_block_pack(d->s, C2, w_ochw, w2, w_packed, reinterpret_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? GCONV_OK : fail_cuda(d, e);
}

int gconv_block_forward(gconv_desc_t d, int C2, const float* x, const void* w_packed, float* y2, void* stream) {
    if (d == nullptr || x == nullptr || w_packed == nullptr || y2 == nullptr) return GCONV_ERR_NULL;
    if (!aligned16(x) || !aligned16(w_packed) || !aligned16(y2)) return GCONV_ERR_ALIGNMENT;
    if (!igemm_block_supported(d->s, C2)) return GCONV_ERR_UNSUPPORTED;
    int rc = ensure_device_state(d);
    if (rc != GCONV_OK) return rc;
    const cudaError_t e = igemm_block_forward(d->s, C2, x, w_packed, y2, d->status_dev, d->sm_count, reinterpret_cast<cudaStream_t>(stream),
                                              launch_opts(d));
    return e == cudaSuccess ? GCONV_OK : fail_cuda(d, e);
}

size_t gconv_workspace_bytes(gconv_desc_t d) {
    if (d == nullptr) return 0;
    return d->variant == GCONV_VARIANT_IGEMM_TF32 ? igemm_scratch_bytes(d->s) : 0;
}

int gconv_desc_set_workspace(gconv_desc_t d, void* workspace, size_t bytes) {
    if (d == nullptr) return GCONV_ERR_NULL;
    if (workspace != nullptr && !aligned16(workspace)) return GCONV_ERR_ALIGNMENT;
    d->workspace = static_cast<float*>(workspace);
    d->workspace_bytes = workspace != nullptr ? bytes : 0;
    return GCONV_OK;
}

int gconv_desc_set_debug(gconv_desc_t d, int wait_limit_us, int skip_stage) {
    if (d == nullptr) return GCONV_ERR_NULL;
    d->wait_us = wait_limit_us > 0 ? wait_limit_us : 0;
    d->dbg_skip = skip_stage >= 0 ? skip_stage : -1;
    return GCONV_OK;
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
        d->last_detail = h.detail;
        e = cudaMemset(d->status_dev, 0, sizeof(Status));
        if (e != cudaSuccess) return fail_cuda(d, e);
    }
    return h.code;
}

int gconv_last_cuda_error(gconv_desc_t d) { return d == nullptr ? 0 : d->last_cuda_error; }

int gconv_last_status_detail(gconv_desc_t d) { return d == nullptr ? 0 : d->last_detail; }

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
        case GCONV_ERR_TOO_LARGE: return "layer larger than the static scratch (x, y and the workspace must fit in 16 MiB)";
        case GCONV_ERR_WORKSPACE: return "the layer needs a workspace (gconv_workspace_bytes) and none large enough is attached";
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
