// DIRECT_TILED, depthwise kernel for small planes ("plane batches"): groups = C_in = C_out, 3x3 (pad 1) or 5x5 (pad 2),
// stride 1 or 2, planes 7, 14 or 28 pixels wide.
//
// Depthwise layers are a stream (9 or 25 MACs per output, 2.25 .. 6.25 FLOP per byte), and on small planes the stream
// kernel of direct_dw.cu is bound by instruction issue: with rows of 7 or 14 pixels its 16-byte loads degrade to scalar
// loads with a bounds check each.  Here the planes of NCHW are taken for what they are in memory, one contiguous run of
// floats: a CTA brings a batch of PB whole planes into shared memory with ONE bulk copy (no per-element address
// arithmetic, no bounds check, the next batch's copy in flight during this batch's math), every thread computes units
// of two output rows by up to seven adjacent columns from shared memory (an input row's window is read once for both
// output rows and all filter columns; the columns that fall into the padding are known at compile time and simply not
// read), the results go to a second
// shared-memory buffer and leave as ONE bulk store of the batch's output planes, which are contiguous as well.  This
// plays the role of Algorithm 1's input and output reshaping without a pass over HBM: x is read once, y written once.
// Sum order per output: (r, s) as in the convolution stage of Algorithm 1.
#include "gconv_internal.h"

namespace gconv {

namespace {

constexpr int kPlaneThreads = 224;                  // at most seven warps: a batch is 224 units on the stride-1 benchmark shapes
constexpr uint64_t kPlaneWaitNs = 1000000000ull;    // a wait for a bulk copy gives up after one second

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void bar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void bar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t bar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok;
}
__device__ __forceinline__ uint64_t timer_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait for a bulk copy: false when the time limit ran out.
__device__ __forceinline__ bool bar_wait(uint32_t bar, uint32_t parity) {
    if (bar_try_wait(bar, parity)) return true;
    uint64_t t0 = 0;
    for (uint32_t it = 0;; ++it) {
        if (bar_try_wait(bar, parity)) return true;
        if ((it & 63u) == 63u) {
            if (it == 63u) t0 = timer_ns();
            else if (timer_ns() - t0 > kPlaneWaitNs) return false;
        }
    }
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void bulk_store(void* dst, uint32_t src, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src), "r"(bytes) : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
// all but the newest `N` bulk stores of this thread have finished READING shared memory
template <int N>
__device__ __forceinline__ void bulk_store_wait_read() {
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}

template <int K, int S, int W>
struct PlaneGeom {
    static constexpr int PAD = K / 2;
    static constexpr int W_OUT = (W - 1) / S + 1;
    static constexpr int SW = W_OUT <= 8 ? W_OUT : 7;     // outputs per strip
    static constexpr int NS = W_OUT / SW;                 // strips per output row: 1, 2 or 4
    static constexpr int WN = (SW - 1) * S + K;           // input columns a strip reads
    static constexpr int RLIM = W + PAD - (NS - 1) * SW * S;   // window columns from here on are right of the image in a row's last strip
    // output rows per unit: two where an input row then serves both (stride 1), or where the planes are so small that
    // fewer, longer units win anyway (14x14 and 7x7 with stride 2: measured 13.5 against 17.2 us on 672 planes of 14x14, 5x5);
    // 28x28 planes with stride 2 need the threads more (17.6 against 27.3 us on 240 planes, 5x5)
    static constexpr int RPU = (S == 1 || W <= 14) ? 2 : 1;
    static constexpr int NR = K + (RPU - 1) * S;          // input rows a unit reads
    static_assert(W_OUT % SW == 0 && (NS & (NS - 1)) == 0, "rows are cut into equal strips");
};

// WHOLE (7x7 planes, stride 1): a thread computes a whole plane -- 49 inputs, the filter and 49 accumulators in
// registers, every index a compile-time constant, so the instruction stream is the FMAs plus one load and one store
// per pixel (the strip units above spend half of their instructions on windows, weights and addresses).
template <int K, int S, int W, bool WHOLE>
__global__ void __launch_bounds__(WHOLE ? 64 : kPlaneThreads)
dw_plane_kernel(const Shape s, const DwPlaneCfg c, const float* __restrict__ x, const uint32_t* __restrict__ packed,
                float* __restrict__ y, Status* status, uint32_t tag) {
    using G = PlaneGeom<K, S, W>;
    extern __shared__ __align__(128) float plane_smem[];
    __shared__ __align__(8) unsigned long long full[2];
    __shared__ int failed;
    const int tid = threadIdx.x;
    if (__ldg(packed) != tag) {                          // uniform across the grid
        if (tid == 0) record_status(status, GCONV_ERR_PACK_MISMATCH, (int)blockIdx.x);
        return;
    }
    const float* __restrict__ wpk = reinterpret_cast<const float*>(packed + kHeaderBytes / 4);
    const int H = s.H, H_out = s.H_out;
    const int HW = H * W, OHW = H_out * G::W_OUT;
    const uint32_t in_elems = (uint32_t)c.PB * (uint32_t)HW, out_elems = (uint32_t)c.PB * (uint32_t)OHW;
    float* const in_buf = plane_smem;                    // [2][PB * HW]
    float* const out_buf = plane_smem + 2 * in_elems;    // [2][PB * OHW]
    if (tid == 0) {
        bar_init(smem_addr(&full[0]), 1);
        bar_init(smem_addr(&full[1]), 1);
        failed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    // a whole batch goes through the bulk copies (sizes and addresses are multiples of 16 bytes: PB is a multiple of 4);
    // the last batch of the tensor may be short and is moved with plain loads and stores
    auto issue = [&](uint32_t b, uint32_t buf) {
        if ((uint64_t)(b + 1) * (uint64_t)c.PB > (uint64_t)c.planes) return;
        const uint32_t bar = smem_addr(&full[buf]);
        bar_expect_tx(bar, in_elems * 4u);
        bulk_load(smem_addr(in_buf + buf * in_elems), x + (size_t)b * in_elems, in_elems * 4u, bar);
    };
    uint32_t b = blockIdx.x, it = 0;
    if (tid == 0 && b < c.batches) issue(b, 0);
    for (; b < c.batches; b += gridDim.x, ++it) {
        const uint32_t buf = it & 1u;
        const uint32_t nb = b + gridDim.x;
        if (tid == 0) bulk_store_wait_read<1>();         // the store that read out_buf[buf] two batches ago is done with it
        __syncthreads();                                 // ... and every thread is done with the previous batch's input
        if (tid == 0 && nb < c.batches) issue(nb, buf ^ 1u);
        const uint32_t plane0 = b * (uint32_t)c.PB;
        const int np = (int)min((uint32_t)c.PB, c.planes - plane0);
        const bool whole = np == c.PB;
        float* const in = in_buf + buf * in_elems;
        float* const out = out_buf + buf * out_elems;
        if (whole) {
            // one thread polls; the others sleep in the barrier below instead of spending issue slots on the poll loop
            if (tid == 0 && !bar_wait(smem_addr(&full[buf]), (it >> 1) & 1u)) failed = 1;
            if (__syncthreads_or(failed)) {
                if (tid == 0) record_status(status, GCONV_ERR_TIMEOUT, 50 + (int)buf);
                break;
            }
        } else {
            const float* src = x + (size_t)plane0 * HW;
            for (int i = tid; i < np * HW; i += (int)blockDim.x) in[i] = __ldg(src + i);
            __syncthreads();
        }
        if constexpr (WHOLE) {
            for (int pl = tid; pl < np; pl += (int)blockDim.x) {
                uint32_t pq, ch;
                c.div_c.divmod(plane0 + (uint32_t)pl, pq, ch);
                const float* __restrict__ wk = wpk + (size_t)ch * (K * K);
                const float* __restrict__ ip = in + pl * (W * W);
                float xin[W * W], wr[K * K], acc[W * W];
#pragma unroll
                for (int i = 0; i < W * W; ++i) xin[i] = ip[i];
#pragma unroll
                for (int i = 0; i < K * K; ++i) wr[i] = __ldg(wk + i);
#pragma unroll
                for (int p = 0; p < W; ++p)
#pragma unroll
                    for (int q = 0; q < W; ++q) {
                        float a = 0.f;
#pragma unroll
                        for (int r = 0; r < K; ++r)
#pragma unroll
                            for (int t = 0; t < K; ++t) {
                                const int h = p + r - G::PAD, v = q + t - G::PAD;
                                if (h >= 0 && h < W && v >= 0 && v < W) a = fmaf(xin[h * W + v], wr[r * K + t], a);
                            }
                        acc[p * W + q] = a;
                    }
                float* __restrict__ op = out + pl * (W * W);
#pragma unroll
                for (int i = 0; i < W * W; ++i) op[i] = acc[i];
            }
        }
        const int units = WHOLE ? 0 : np * c.upp;
        for (int u = tid; u < units; u += (int)blockDim.x) {
            uint32_t pl, rem;
            c.div_upp.divmod((uint32_t)u, pl, rem);
            const int orow = (int)(rem / (uint32_t)G::NS) * G::RPU, st = (int)(rem % (uint32_t)G::NS);
            uint32_t pq, ch;
            c.div_c.divmod(plane0 + pl, pq, ch);
            const float* __restrict__ wk = wpk + (size_t)ch * (K * K);
            const float* __restrict__ ip = in + pl * (uint32_t)HW + (st * G::SW * S - G::PAD);
            const bool first = st == 0, last = st == G::NS - 1;
            float wr[K][K];
#pragma unroll
            for (int i = 0; i < K * K; ++i) wr[i / K][i % K] = __ldg(wk + i);
            float acc[G::RPU][G::SW];
#pragma unroll
            for (int i = 0; i < G::RPU; ++i)
#pragma unroll
                for (int q = 0; q < G::SW; ++q) acc[i][q] = 0.f;
            // input row rr of the unit is filter row rr - i*S of the unit's output row i
#pragma unroll
            for (int rr = 0; rr < G::NR; ++rr) {
                const int h = orow * S - G::PAD + rr;
                if (h >= 0 && h < H) {
                    const float* __restrict__ row = ip + h * W;
                    float win[G::WN];
#pragma unroll
                    for (int j = 0; j < G::WN; ++j) {
                        // columns left of the image exist only in a row's first strip, columns right of it only in its last
                        const bool in_image = (j >= G::PAD || !first) && (j < G::RLIM || !last);
                        win[j] = in_image ? row[j] : 0.f;
                    }
#pragma unroll
                    for (int i = 0; i < G::RPU; ++i) {
                        const int r = rr - i * S;
                        if (r >= 0 && r < K) {
#pragma unroll
                            for (int q = 0; q < G::SW; ++q)
#pragma unroll
                                for (int t = 0; t < K; ++t) acc[i][q] = fmaf(win[q * S + t], wr[r][t], acc[i][q]);
                        }
                    }
                }
            }
#pragma unroll
            for (int i = 0; i < G::RPU; ++i) {
                if (orow + i < H_out) {
                    float* __restrict__ op = out + pl * (uint32_t)OHW + (orow + i) * G::W_OUT + st * G::SW;
#pragma unroll
                    for (int q = 0; q < G::SW; ++q) op[q] = acc[i][q];
                }
            }
        }
        if (whole) {
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the bulk store reads shared memory through the async proxy
            __syncthreads();
            if (tid == 0) bulk_store(y + (size_t)plane0 * OHW, smem_addr(out), out_elems * 4u);
        } else {
            __syncthreads();
            float* dst = y + (size_t)plane0 * OHW;
            for (int i = tid; i < np * OHW; i += (int)blockDim.x) dst[i] = out[i];
        }
    }
    if (tid == 0) {
        asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // every bulk store of this CTA has completed (shared memory must
                                                                    // outlive the stores that read it; y is whole when the CTA exits)
        // after a wait that ran out a copy may still be in flight into this CTA's shared memory: give it the same limit again
        if (failed) {
            const uint32_t nb = b + gridDim.x;
            if (nb < c.batches) (void)bar_wait(smem_addr(&full[(it & 1u) ^ 1u]), ((it + 1) >> 1) & 1u);
            (void)bar_wait(smem_addr(&full[it & 1u]), (it >> 1) & 1u);
        }
    }
}

template <int K, int S, int W, bool WHOLE = false>
cudaError_t launch_plane(const Shape& s, const DwPlaneCfg& c, const float* x, const uint32_t* pk, float* y, Status* status,
                         uint32_t tag, cudaStream_t st) {
    auto kernel = dw_plane_kernel<K, S, W, WHOLE>;
    static bool attr_set[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 64 && !attr_set[dev]) {
        e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 64 * 1024);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    kernel<<<c.grid, c.threads, c.smem_bytes, st>>>(s, c, x, pk, y, status, tag);
    return cudaGetLastError();
}

}  // namespace

bool dw_plane_supported(const Shape& s) {
    if (!s.square() || !(s.Cg == 1 && s.Kg == 1) || s.dilation != 1 || !(s.stride == 1 || s.stride == 2)) return false;
    const bool k3 = s.KH == 3 && s.KW == 3 && s.pad == 1, k5 = s.KH == 5 && s.KW == 5 && s.pad == 2;
    if (!(k3 || k5)) return false;
    if (!(s.W == 7 || s.W == 14 || s.W == 28)) return false;
    const long long per_plane = (long long)s.H * s.W + (long long)s.H_out * s.W_out;
    if (per_plane * 4 * 8 > 50 * 1024) return false;              // a batch of four planes, in and out, twice
    return (unsigned long long)s.N * s.C_in < (1ull << 31) / 4;
}

// Planes per batch: a multiple of four (bulk copies move multiples of 16 bytes), as many as keep four CTAs on an SM,
// then fewer if that spreads the batches more evenly over the CTAs the grid holds.
DwPlaneCfg dw_plane_config(const Shape& s, int sm_count) {
    DwPlaneCfg c;
    const long long planes = (long long)s.N * s.C_in;
    const int per_plane = s.H * s.W + s.H_out * s.W_out;
    const int sw = s.W_out <= 8 ? s.W_out : 7;
    const int rpu = (s.stride == 1 || s.W <= 14) ? 2 : 1;
    const bool whole = s.W == 7 && s.H == 7 && s.stride == 1;     // a thread per plane
    c.upp = whole ? 1 : ((s.H_out + rpu - 1) / rpu) * (s.W_out / sw);   // a unit is one strip of one (stride 1: two) output rows, or a plane
    int pb_max = (50 * 1024) / (per_plane * 8);
    pb_max &= ~3;
    if (pb_max > 64) pb_max = 64;
    int best = 4;
    double best_eff = -1.0;
    auto threads_for = [&](int pb) {
        const int units = pb * c.upp;
        const int cap = whole ? 64 : kPlaneThreads;
        return units >= cap ? cap : ((units + 31) / 32) * 32;
    };
    auto ctas_per_sm = [&](int pb) {
        const size_t smem = (size_t)pb * per_plane * 8;
        int per_sm = (int)((220u * 1024u) / (smem + 1024u));
        const int by_threads = 2048 / threads_for(pb);
        return per_sm < by_threads ? per_sm : by_threads;
    };
    for (int pb = pb_max; pb >= 4; pb -= 4) {
        const long long batches = (planes + pb - 1) / pb;
        const long long slots = (long long)sm_count * ctas_per_sm(pb);
        const long long rounds = (batches + slots - 1) / slots;
        double eff = (double)batches / (double)(rounds * slots);
        const int units = pb * c.upp, t = threads_for(pb);        // a batch should fill its CTA's threads
        eff *= (double)units / (double)(((units + t - 1) / t) * t);
        if (eff > best_eff + 0.02) {
            best_eff = eff;
            best = pb;
        }
    }
    c.PB = best;
    c.planes = (uint32_t)planes;
    c.batches = (uint32_t)((planes + best - 1) / best);
    c.smem_bytes = (uint32_t)((size_t)best * per_plane * 8);
    c.threads = (uint32_t)threads_for(best);
    const long long slots = (long long)sm_count * ctas_per_sm(best);
    c.grid = (uint32_t)(c.batches < slots ? c.batches : slots);
    c.div_upp = make_fastdiv((uint32_t)c.upp);
    c.div_c = make_fastdiv((uint32_t)s.C_in);
    return c;
}

cudaError_t dw_plane_forward(const Shape& s, const float* x, const void* packed, float* y, Status* status, int sm_count,
                             cudaStream_t st) {
    const DwPlaneCfg c = dw_plane_config(s, sm_count);
    const uint32_t tag = pack_tag(s, GCONV_VARIANT_DIRECT_TILED);
    const uint32_t* pk = reinterpret_cast<const uint32_t*>(packed);
#define GCONV_PLANE_W(K, S) \
    do { \
        if (s.W == 7 && s.H == 7 && S == 1) return launch_plane<K, 1, 7, true>(s, c, x, pk, y, status, tag, st); \
        if (s.W == 7) return launch_plane<K, S, 7>(s, c, x, pk, y, status, tag, st); \
        if (s.W == 14) return launch_plane<K, S, 14>(s, c, x, pk, y, status, tag, st); \
        return launch_plane<K, S, 28>(s, c, x, pk, y, status, tag, st); \
    } while (0)
    if (s.KH == 3) {
        if (s.stride == 1) GCONV_PLANE_W(3, 1);
        else GCONV_PLANE_W(3, 2);
    } else {
        if (s.stride == 1) GCONV_PLANE_W(5, 1);
        else GCONV_PLANE_W(5, 2);
    }
#undef GCONV_PLANE_W
}

}  // namespace gconv
