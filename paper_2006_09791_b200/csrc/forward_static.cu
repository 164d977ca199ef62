// gconv_forward_host_static: grouped convolution on host buffers for callers that must not allocate.
//
// Some users of this library run where device allocation is off limits once they are up: a plugin
// inside an application whose memory pool owns the whole device, a service that pre-commits its
// memory at start and treats any later cudaMalloc as a fault, code that is called between
// cudaStreamBeginCapture and EndCapture (where cudaMalloc is illegal), or a latency-critical loop
// that cannot afford the implicit device synchronisation an allocation brings.  gconv_forward
// allocates a small status block on its first call, and gconv_forward_host additionally needs two
// caller-allocated staging buffers.  This entry point needs neither: the device scratch it uses (a
// status block plus staging room for x and y) is a file-scope array in the library's device image.
//
// Consequences worth knowing:
//   * every GPU that loads the library carries the array (16 MiB + 256 B) until the process exits;
//   * layers whose x and y do not fit are rejected (GCONV_ERR_TOO_LARGE), nothing is enqueued;
//   * all calls share the array, which keeps whatever the previous call left in it; the status
//     block is cleared at the start of every call and the staging regions are fully overwritten
//     before they are read, so stale contents never reach a result;
//   * two calls that overlap on the GPU (different streams, or threads) race on the array.
#include "gconv_internal.h"

using namespace gconv;

namespace {

constexpr size_t kStatusBytes = 256;
constexpr size_t kStageBytes = 16u * 1024u * 1024u;   // room for x and y together

// In host code this name is only a handle for the runtime; the device address comes from
// cudaGetSymbolAddress (a kernel given the host-side name would read the wrong memory or fault).
static __device__ __align__(256) unsigned char g_static_scratch[kStatusBytes + kStageBytes];

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
    if (round256(xb) + round256(yb) > kStageBytes) return GCONV_ERR_TOO_LARGE;
    // layers that the tensor-core variant runs on a padded copy of x need a second scratch buffer: not offered here
    if (d->variant == GCONV_VARIANT_IGEMM_TF32 && igemm_scratch_bytes(s) > 0) return GCONV_ERR_UNSUPPORTED;

    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess || dev < 0 || dev >= 64) {
        d->last_cuda_error = (int)(e != cudaSuccess ? e : cudaErrorInvalidDevice);
        (void)cudaGetLastError();
        return GCONV_ERR_CUDA;
    }
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
    unsigned char* base = g_scratch_addr[dev];
    Status* status = reinterpret_cast<Status*>(base);
    float* x_stage = reinterpret_cast<float*>(base + kStatusBytes);
    float* y_stage = reinterpret_cast<float*>(base + kStatusBytes + round256(xb));
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);

    e = cudaMemsetAsync(status, 0, sizeof(Status), st);   // the status block must start at zero
    if (e == cudaSuccess) e = cudaMemcpyAsync(x_stage, x_host, xb, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) {
        switch (d->variant) {
            case GCONV_VARIANT_IGEMM_TF32:
                e = igemm_forward(s, x_stage, w_packed, y_stage, status, g_sm_count[dev], st, nullptr);
                break;
            case GCONV_VARIANT_DIRECT_TILED:
                e = tiled_forward(s, x_stage, w_packed, y_stage, status, g_sm_count[dev], st);
                break;
            default:
                e = generic_forward(s, x_stage, w_packed, y_stage, status, g_sm_count[dev], st);
                break;
        }
    }
    if (e == cudaSuccess) e = cudaMemcpyAsync(y_host, y_stage, yb, cudaMemcpyDeviceToHost, st);
    Status h;
    h.code = 0;
    if (e == cudaSuccess) e = cudaMemcpyAsync(&h, status, sizeof(Status), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) {
        d->last_cuda_error = (int)e;
        (void)cudaGetLastError();
        return GCONV_ERR_CUDA;
    }
    return h.code;   // GCONV_OK, or what a kernel recorded (pack mismatch, bounded wait ran out)
}
