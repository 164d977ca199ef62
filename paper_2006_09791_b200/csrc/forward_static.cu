// gconv_forward_host_static: grouped convolution on host buffers for callers that must not allocate.
//
// Some users of this library run where device allocation is off limits once they are up: a plugin
// inside an application whose memory pool owns the whole device, a service that pre-commits its
// memory at start and treats any later cudaMalloc as a fault, or a latency-critical loop that
// cannot afford the implicit device synchronisation an allocation brings.  gconv_forward
// allocates a small status block on its first call, and gconv_forward_host additionally needs two
// caller-allocated staging buffers (and, for a few layers, a caller-allocated workspace).  This
// entry point needs none of them: the device scratch it uses (a status block, staging room for x
// and y, and the workspace where the layer needs one) is a file-scope array in the library's
// device image.
//
// Consequences worth knowing:
//   * every GPU that loads the library carries the array (16 MiB + 256 B) until the process exits;
//   * layers whose x, y and workspace do not fit are rejected (GCONV_ERR_TOO_LARGE), nothing is enqueued;
//   * the call always synchronises its stream before it returns (so it cannot be part of a stream capture);
//   * all calls share the array, which keeps whatever the previous call left in it; the status
//     block is cleared at the start of every call and the staging regions are fully overwritten
//     before they are read, so stale contents never reach a result;
//   * two calls that overlap on the GPU (different streams, or threads) race on the array.
#include <mutex>

#include "gconv_internal.h"

using namespace gconv;

namespace {

constexpr size_t kStatusBytes = 256;
constexpr size_t kStageBytes = 16u * 1024u * 1024u;   // room for x and y together

// In host code this name is only a handle for the runtime; the device address comes from
// cudaGetSymbolAddress (a kernel given the host-side name would read the wrong memory or fault).
static __device__ __align__(256) unsigned char g_static_scratch[kStatusBytes + kStageBytes];

std::mutex g_setup_mutex;                        // first calls from several threads set a device up once
unsigned char* g_scratch_addr[64] = {nullptr};   // per device, filled on the first call made with that device current
int g_sm_count[64] = {0};

inline size_t round256(size_t v) { return (v + 255) & ~(size_t)255; }

}  // namespace

extern "C" int gconv_forward_host_static(gconv_desc_t d, const float* x_host, const void* w_packed, float* y_host,
                                         void* stream) {
    if (d == nullptr || x_host == nullptr || w_packed == nullptr || y_host == nullptr) return GCONV_ERR_NULL;
    if ((reinterpret_cast<uintptr_t>(w_packed) & 15u) != 0) return GCONV_ERR_ALIGNMENT;
    const Shape& s = d->s;
    const size_t xb = sizeof(float) * (size_t)s.N * s.C_in * s.H * s.W;
    const size_t yb = sizeof(float) * (size_t)s.N * s.C_out * s.H_out * s.W_out;
    // layers that the tensor-core variant runs on a zero-padded copy of x: the copy lives in the same array
    const size_t wsb = d->variant == GCONV_VARIANT_IGEMM_TF32 ? igemm_scratch_bytes(s) : 0;
    if (round256(xb) + round256(yb) + round256(wsb) > kStageBytes) return GCONV_ERR_TOO_LARGE;

    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess || dev < 0 || dev >= 64) {
        d->last_cuda_error = (int)(e != cudaSuccess ? e : cudaErrorInvalidDevice);
        (void)cudaGetLastError();
        return GCONV_ERR_CUDA;
    }
    unsigned char* base = nullptr;
    int sm_count = 0;
    {
        std::lock_guard<std::mutex> lock(g_setup_mutex);
        if (g_scratch_addr[dev] == nullptr) {
            // one-time set-up for this device: resolve the array's device address and the SM count
            unsigned char* p = nullptr;
            e = cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_static_scratch);
            if (e == cudaSuccess) e = cudaDeviceGetAttribute(&g_sm_count[dev], cudaDevAttrMultiProcessorCount, dev);
            if (e != cudaSuccess || p == nullptr) {
                d->last_cuda_error = (int)e;
                (void)cudaGetLastError();
                return GCONV_ERR_CUDA;
            }
            g_scratch_addr[dev] = p;
        }
        base = g_scratch_addr[dev];
        sm_count = g_sm_count[dev];
    }
    Status* status = reinterpret_cast<Status*>(base);
    float* x_stage = reinterpret_cast<float*>(base + kStatusBytes);
    float* y_stage = reinterpret_cast<float*>(base + kStatusBytes + round256(xb));
    float* ws = wsb > 0 ? reinterpret_cast<float*>(base + kStatusBytes + round256(xb) + round256(yb)) : nullptr;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);

    e = cudaMemsetAsync(status, 0, sizeof(Status), st);   // the status block must start at zero
    bool enqueued = false;       // something that reads or writes the caller's host buffers is in the stream
    if (e == cudaSuccess) {
        e = cudaMemcpyAsync(x_stage, x_host, xb, cudaMemcpyHostToDevice, st);
        enqueued = e == cudaSuccess;
    }
    if (e == cudaSuccess) {
        IgemmLaunchOpts opts;
        opts.pdl = false;        // the kernel follows a copy, not a kernel: nothing to overlap
        opts.wait_us = (uint32_t)d->wait_us;
        opts.dbg_skip = d->dbg_skip;
        switch (d->variant) {
            case GCONV_VARIANT_IGEMM_TF32:
                e = igemm_forward(s, x_stage, w_packed, y_stage, status, sm_count, st, ws, opts);
                break;
            case GCONV_VARIANT_DIRECT_TILED:
                e = tiled_forward(s, x_stage, w_packed, y_stage, status, sm_count, st);
                break;
            default:
                e = generic_forward(s, x_stage, w_packed, y_stage, status, sm_count, st);
                break;
        }
    }
    if (e == cudaSuccess) e = cudaMemcpyAsync(y_host, y_stage, yb, cudaMemcpyDeviceToHost, st);
    Status h;
    h.code = 0;
    if (e == cudaSuccess) e = cudaMemcpyAsync(&h, status, sizeof(Status), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) {
        // a copy that was already enqueued may still read x_host or write y_host: wait for it before returning
        if (enqueued) (void)cudaStreamSynchronize(st);
        d->last_cuda_error = (int)e;
        (void)cudaGetLastError();
        return GCONV_ERR_CUDA;
    }
    return h.code;   // GCONV_OK, or what a kernel recorded (pack mismatch, bounded wait ran out)
}
