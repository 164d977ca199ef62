// Variant IGEMM_TF32: per-group implicit GEMM on the 5th-generation tensor cores (tcgen05 + TMEM).
//
// Formulation.  For a 3x3, stride-1, pad-1 grouped convolution (Section II of the paper) write the
// image plane of a channel as a flat vector of H*W pixels, f = p*W + q.  Then
//
//     y[k, f] = D_0[k, f-1] * [q > 0]  +  D_1[k, f]  +  D_2[k, f+1] * [q < W-1],
//     D_s[k, f] = sum_{c<Cg} sum_{r<3} x[c, f + (r-1)*W] * w[k, c, r, s]        (x = 0 outside the plane),
//
// because a vertical tap is a shift by a whole row (W pixels, 16-byte aligned when W % 4 == 0) and
// reads outside [0, H*W) are exactly the rows above and below the image.  The three horizontal taps
// are NOT applied to the input: they become three accumulators per filter, combined in the
// epilogue with a one-lane shift.  So for a tile of 128 consecutive pixels the contraction is one
// dense GEMM  D[128 pixels, 3*Kt] += A_r[128 pixels, Cg] * B_r[Cg, 3*Kt]  summed over r = 0,1,2:
//   * A_r is the NCHW input itself, row-shifted: a TMA box of 32 pixels x CK channels lands in
//     shared memory as the canonical MN-major tcgen05 operand (pixels contiguous, 128-byte rows
//     swizzled in 32-byte atoms, which is the one MN-major layout TF32 operands may use),
//     zero-filled above/below the image by TMA's out-of-bounds fill.  No im2col copy exists anywhere.
//   * B_r comes from the pre-packed weights (kernel-reshaping stage of Algorithm 1): already
//     TF32-rounded and stored as the exact shared-memory image of a K-major core-matrix operand,
//     so one bulk copy per pipeline stage stages it.
//   * D lives in TMEM (3*Kt <= 192 fp32 columns, double buffered), the epilogue warps read it with
//     tcgen05.ld, apply the horizontal shifts with warp shuffles and write y directly in NCHW with
//     128-byte coalesced rows.
// Stride 2 (pad 1) keeps the even rows and columns of that stride-1 result: same operands, the
// epilogue stores only those lanes (and for W = 32 the odd rows are never loaded or multiplied).
// All groups and all images run in one persistent launch: the tile index enumerates
// (group, filter tile, pixel tile), one CTA per SM walks it.
//
// Warp roles: warp 0 = TMA producer, warp 1 = TMEM owner + single-thread MMA issuer,
// warps 2..5 = epilogue (TMEM lane quarter = warp_id % 4).  Every mbarrier wait is bounded: when a
// wait runs out the kernel records GCONV_ERR_TIMEOUT, all roles leave their loops, outstanding bulk
// copies are waited for (bounded), TMEM is freed and the kernel returns.
#include <cuda.h>

#include "gconv_internal.h"

namespace gconv {

namespace {

constexpr int kThreads = 192;
constexpr int kTmemCols = 512;
constexpr int kAccStride = 256;          // TMEM column offset between the two accumulator buffers
constexpr uint32_t kSpinLimit = 1u << 20;

struct __align__(8) SharedCtl {
    unsigned long long full[8];
    unsigned long long empty[8];
    unsigned long long tmem_full[2];
    unsigned long long tmem_empty[2];
    unsigned long long xchg_bar[2];
    uint32_t tmem_base;
    int abort_flag;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
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

// Bounded wait.  Returns false if the wait ran out or another role already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, Status* status,
                                          int where) {
    for (uint32_t it = 0; it < kSpinLimit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (it > 4096) __nanosleep(64);
    }
    *abort_flag = 1;
    record_status(status, GCONV_ERR_TIMEOUT, where);
    return false;
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void bulk_load_1d(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void umma_tf32(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(acc)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, float (&v)[8]) {
    uint32_t r0, r1, r2, r3, r4, r5, r6, r7;
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3), "=r"(r4), "=r"(r5), "=r"(r6), "=r"(r7)
                 : "r"(taddr));
    v[0] = __uint_as_float(r0); v[1] = __uint_as_float(r1); v[2] = __uint_as_float(r2); v[3] = __uint_as_float(r3);
    v[4] = __uint_as_float(r4); v[5] = __uint_as_float(r5); v[6] = __uint_as_float(r6); v[7] = __uint_as_float(r7);
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor (tcgen05): start address, leading/stride byte offsets in 16-byte
// units, descriptor version 1, swizzle mode in bits 61..63 (0 = none, 1 = 128-byte rows swizzled in
// 32-byte atoms, the only MN-major mode TF32 operands accept, 2 = 128-byte with 16-byte atoms).
__device__ __forceinline__ uint64_t make_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint32_t layout) {
    const uint32_t lo = ((addr >> 4) & 0x3FFFu) | (((lbo_bytes >> 4) & 0x3FFFu) << 16);
    const uint32_t hi = ((sbo_bytes >> 4) & 0x3FFFu) | (1u << 14) | (layout << 29);
    return ((uint64_t)hi << 32) | lo;
}


__global__ void __launch_bounds__(kThreads, 1)
igemm_tf32_kernel(const __grid_constant__ CUtensorMap xmap, const Shape s, const IgemmCfg c,
                  const uint32_t* __restrict__ packed, float* __restrict__ y, Status* status, uint32_t tag) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    __shared__ SharedCtl ctl;
    __shared__ float xchg[2][4][2][64];

    if (packed[0] != tag) {
        if (threadIdx.x == 0) record_status(status, GCONV_ERR_PACK_MISMATCH, (int)blockIdx.x);
        return;
    }
    const uint8_t* __restrict__ wblocks = reinterpret_cast<const uint8_t*>(packed) + kHeaderBytes;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t smem_base = smem_u32(smem);
    volatile int* abort_flag = &ctl.abort_flag;

    if (threadIdx.x == 0) {
        for (int i = 0; i < c.stages; ++i) {
            mbar_init(smem_u32(&ctl.full[i]), 1);
            mbar_init(smem_u32(&ctl.empty[i]), 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&ctl.tmem_full[i]), 1);
            mbar_init(smem_u32(&ctl.tmem_empty[i]), 4);
            mbar_init(smem_u32(&ctl.xchg_bar[i]), 4);
        }
        ctl.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl.tmem_base)),
                     "r"(kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctl.tmem_base;

    const int kstages = 3 * c.chunks;                 // pipeline stages per tile: (r, channel chunk)
    const uint32_t a_bytes = 4u * (uint32_t)c.CK * 128u;
    const uint32_t b_bytes = (uint32_t)c.Np * (uint32_t)c.CK * 4u;
    const int HW = s.H * s.W;
    const size_t OHW = (size_t)s.H_out * s.W_out;

    if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < c.num_tiles && ok; tile += gridDim.x) {
                const int mt = tile % c.MT;
                const int rest = tile / c.MT;
                const int nt = rest % c.NT;
                const int g = rest / c.NT;
                int seg_n[4], seg_f[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (c.seg_mode) {
                        const int sg = mt * 4 + j;
                        int n = sg / c.SPI;
                        seg_f[j] = (sg - n * c.SPI) * c.seg_fstep;
                        seg_n[j] = n < s.N ? n : s.N;   // past the last image: fully out of bounds, zero fill
                    } else {
                        const int n = mt / c.RB;
                        seg_n[j] = n;
                        seg_f[j] = (mt - n * c.RB) * c.R * s.W + 32 * j;
                    }
                }
                const uint8_t* wtile = wblocks + (size_t)(g * c.NT + nt) * (size_t)kstages * b_bytes;
                for (int ks = 0; ks < kstages; ++ks, ++it) {
                    const int stage = it % c.stages;
                    const uint32_t ph = (it / c.stages) & 1;
                    if (!mbar_wait(smem_u32(&ctl.empty[stage]), ph ^ 1, abort_flag, status, 100 + stage)) { ok = false; break; }
                    const int r = ks / c.chunks;
                    const int ch = ks - r * c.chunks;
                    const uint32_t full = smem_u32(&ctl.full[stage]);
                    const uint32_t a_dst = smem_base + (uint32_t)stage * c.stage_bytes;
                    mbar_arrive_expect_tx(full, a_bytes + b_bytes);
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        tma_load_3d(a_dst + (uint32_t)j * (uint32_t)c.CK * 128u, &xmap, seg_f[j] + (r - 1) * s.W,
                                    g * s.Cg + ch * c.CK, seg_n[j], full);
                    bulk_load_1d(a_dst + a_bytes, wtile + (size_t)ks * b_bytes, b_bytes, full);
                }
            }
            if (!ok) {
                // drain: wait (bounded) for the copies of every stage that may still be in flight
                for (int i = 0; i < c.stages && i < (int)it; ++i) {
                    const uint32_t j = it - 1 - i;
                    const uint32_t bar = smem_u32(&ctl.full[j % c.stages]);
                    for (uint32_t spin = 0; spin < kSpinLimit; ++spin)
                        if (mbar_try_wait(bar, (j / c.stages) & 1)) break;
                }
            }
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer
        if (lane == 0) {
            const uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | (1u << 15) | ((uint32_t)(c.Np >> 3) << 17) |
                                   ((128u >> 4) << 24);
            const uint32_t a_lbo = (uint32_t)c.CK * 128u;          // next 32-pixel block
            const uint32_t b_lbo = (uint32_t)(c.Np >> 3) * 128u;   // next 4-channel core matrix along K
            const uint32_t b_kstep = 2u * b_lbo;                   // 8 channels
            uint32_t it = 0, tcount = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < c.num_tiles && ok; tile += gridDim.x, ++tcount) {
                const uint32_t buf = tcount & 1;
                if (!mbar_wait(smem_u32(&ctl.tmem_empty[buf]), ((tcount >> 1) & 1) ^ 1, abort_flag, status, 200 + buf)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * kAccStride;
                for (int ks = 0; ks < kstages; ++ks, ++it) {
                    const int stage = it % c.stages;
                    if (!mbar_wait(smem_u32(&ctl.full[stage]), (it / c.stages) & 1, abort_flag, status, 300 + stage)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_addr = smem_base + (uint32_t)stage * c.stage_bytes;
                    const uint32_t b_addr = a_addr + a_bytes;
                    for (int k8 = 0; k8 < c.CK / 8; ++k8) {
                        const uint64_t adesc = make_desc(a_addr + (uint32_t)k8 * 1024u, a_lbo, 512u, 1u);
                        const uint64_t bdesc = make_desc(b_addr + (uint32_t)k8 * b_kstep, b_lbo, 128u, 0u);
                        umma_tf32(d_tmem, adesc, bdesc, idesc, (ks | k8) != 0 ? 1u : 0u);
                    }
                    umma_commit(smem_u32(&ctl.empty[stage]));
                }
                if (ok) umma_commit(smem_u32(&ctl.tmem_full[buf]));
            }
        }
    } else {
        // ---------------------------------------------------------------- epilogue warps
        const int wq = warp & 3;                       // TMEM lane quarter this warp may read
        const int l = wq * 32 + lane;                  // pixel lane inside the tile
        const int Kt = c.Kt;
        uint32_t tcount = 0;
        for (int tile = blockIdx.x; tile < c.num_tiles; tile += gridDim.x, ++tcount) {
            const int mt = tile % c.MT;
            const int rest = tile / c.MT;
            const int nt = rest % c.NT;
            const int g = rest / c.NT;
            int n, f;
            bool valid;
            if (c.seg_mode) {
                const int sg = mt * 4 + wq;
                n = sg / c.SPI;
                f = (sg - n * c.SPI) * c.seg_fstep + lane;
                valid = n < s.N;
            } else {
                n = mt / c.RB;
                f = (mt - n * c.RB) * c.R * s.W + l;
                valid = (l < c.R * s.W) && (f < HW);
            }
            const int prow = f / s.W;
            const int q = f - prow * s.W;
            const bool use_left = q > 0;
            const bool use_right = q < s.W - 1;
            int fo = f;                                  // position in the output plane
            if (s.stride == 2) {                         // stride 2 keeps the even rows and columns of the stride-1 result
                valid = valid && ((prow & 1) == 0) && ((q & 1) == 0);
                fo = (prow >> 1) * s.W_out + (q >> 1);
            }
            const uint32_t buf = tcount & 1;
            if (!mbar_wait(smem_u32(&ctl.tmem_full[buf]), (tcount >> 1) & 1, abort_flag, status, 400 + buf)) break;
            tc_fence_after();
            const uint32_t t0 = tmem_base + buf * kAccStride + ((uint32_t)(wq * 32) << 16);
            float* yk = y + ((size_t)n * s.C_out + (size_t)g * s.Kg + (size_t)nt * Kt) * OHW + fo;
            for (int k0 = 0; k0 < Kt; k0 += 8) {
                float d0[8], d1[8], d2[8];
                tmem_ld8(t0 + (uint32_t)k0, d0);
                tmem_ld8(t0 + (uint32_t)(Kt + k0), d1);
                tmem_ld8(t0 + (uint32_t)(2 * Kt + k0), d2);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const float up = __shfl_up_sync(0xffffffffu, d0[i], 1);
                    const float dn = __shfl_down_sync(0xffffffffu, d2[i], 1);
                    float v = d1[i];
                    if (use_left && lane > 0) v += up;
                    if (use_right && lane < 31) v += dn;
                    if (c.need_xchg) {
                        if (lane == 31) xchg[buf][wq][0][k0 + i] = d0[i];
                        if (lane == 0) xchg[buf][wq][1][k0 + i] = d2[i];
                    }
                    if (valid) yk[(size_t)(k0 + i) * OHW] = v;
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctl.tmem_empty[buf]));
            if (c.need_xchg) {
                // rows that straddle a warp boundary: add the neighbour warp's edge lane once all four
                // epilogue warps have published theirs (bounded mbarrier wait, never a named barrier)
                if (lane == 0) mbar_arrive(smem_u32(&ctl.xchg_bar[buf]));
                if (!mbar_wait(smem_u32(&ctl.xchg_bar[buf]), (tcount >> 1) & 1, abort_flag, status, 500 + buf)) break;
                if (valid && lane == 0 && wq > 0 && use_left)
                    for (int k = 0; k < Kt; ++k) yk[(size_t)k * OHW] += xchg[buf][wq - 1][0][k];
                if (valid && lane == 31 && wq < 3 && use_right)
                    for (int k = 0; k < Kt; ++k) yk[(size_t)k * OHW] += xchg[buf][wq + 1][1][k];
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

// Weight pre-pack for this variant.  Output block (g, nt, r, chunk) is the shared-memory image of
// the K-major, unswizzled B operand of one pipeline stage: [k8][k2][n/8][n%8][4 channels], where
// column n = s*Kt + k holds filter nt*Kt + k at horizontal tap s (columns >= 3*Kt are zero) and
// values are rounded to TF32 (round to nearest, ties away from zero).
__global__ void igemm_pack_kernel(Shape s, IgemmCfg c, const float* __restrict__ w, uint32_t* __restrict__ packed, uint32_t tag) {
    const size_t total = (size_t)s.groups * c.NT * 3 * c.chunks * c.Np * c.CK;
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i == 0) {
        packed[0] = tag;
        for (int j = 1; j < kHeaderBytes / 4; ++j) packed[j] = 0;
    }
    uint32_t* dst = packed + kHeaderBytes / 4;
    for (; i < total; i += (size_t)gridDim.x * blockDim.x) {
        size_t t = i;
        const int e = (int)(t % 4); t /= 4;        // channel within the 16-byte core-matrix row
        const int n8 = (int)(t % 8); t /= 8;       // row within the core matrix
        const int nb = (int)(t % (c.Np / 8)); t /= (c.Np / 8);
        const int k2 = (int)(t % 2); t /= 2;
        const int k8 = (int)(t % (c.CK / 8)); t /= (c.CK / 8);
        const int ch = (int)(t % c.chunks); t /= c.chunks;
        const int r = (int)(t % 3); t /= 3;
        const int nt = (int)(t % c.NT);
        const int g = (int)(t / c.NT);
        const int ncol = nb * 8 + n8;
        const int cc = ch * c.CK + k8 * 8 + k2 * 4 + e;
        uint32_t bits = 0;
        if (ncol < 3 * c.Kt) {
            const int ss = ncol / c.Kt;
            const int k = ncol - ss * c.Kt;
            const float v = w[(((size_t)(g * s.Kg + nt * c.Kt + k)) * s.Cg + cc) * 9 + r * 3 + ss];
            asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(bits) : "f"(v));
        }
        dst[i] = bits;
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (fn == nullptr) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

}  // namespace

bool igemm_supported(const Shape& s) {
    if (!(s.KH == 3 && s.KW == 3 && (s.stride == 1 || s.stride == 2) && s.pad == 1 && s.dilation == 1)) return false;
    if (s.Cg % 8 != 0 || s.Kg % 8 != 0) return false;
    if (s.W % 4 != 0 || s.W > 128) return false;
    if ((long long)s.H * s.W < 32) return false;
    if (s.C_in > 65535 * 8) return false;
    return true;
}

IgemmCfg igemm_config(const Shape& s, int sm_count) {
    IgemmCfg c;
    c.CK = (s.Cg % 32 == 0) ? 32 : (s.Cg % 16 == 0 ? 16 : 8);
    c.chunks = s.Cg / c.CK;
    int kt = s.Kg <= 64 ? s.Kg : 64;
    while (s.Kg % kt != 0 || kt % 8 != 0) kt -= 8;   // largest multiple of 8 dividing Kg, at most 64
    c.Kt = kt;
    c.NT = s.Kg / kt;
    c.Np = (3 * kt + 15) & ~15;
    const int HW = s.H * s.W;
    c.seg_mode = (32 % s.W == 0) && (HW % 32 == 0);
    c.seg_fstep = 32;
    if (c.seg_mode) {
        c.SPI = HW / 32;
        if (s.stride == 2 && s.W == 32) {   // a segment is one row: visit the even rows only
            c.seg_fstep = 64;
            c.SPI = (s.H + 1) / 2;
        }
        c.R = 0;
        c.RB = 0;
        c.MT = (int)(((long long)s.N * c.SPI + 3) / 4);
        c.need_xchg = 0;
    } else {
        c.SPI = 0;
        c.R = 128 / s.W;
        c.RB = (s.H + c.R - 1) / c.R;
        c.MT = s.N * c.RB;
        c.need_xchg = 1;
    }
    c.num_tiles = s.groups * c.NT * c.MT;
    const uint32_t a_bytes = 4u * c.CK * 128u, b_bytes = (uint32_t)c.Np * c.CK * 4u;
    c.stage_bytes = (a_bytes + b_bytes + 1023u) & ~1023u;
    int st = (int)((160u * 1024u) / c.stage_bytes);
    if (st > 8) st = 8;
    if (st < 2) st = 2;
    c.stages = st;
    c.smem_bytes = (size_t)c.stages * c.stage_bytes + 1024;
    c.grid = c.num_tiles < sm_count ? c.num_tiles : sm_count;
    return c;
}

size_t igemm_packed_bytes(const Shape& s) {
    const IgemmCfg c = igemm_config(s, 148);
    return kHeaderBytes + sizeof(float) * (size_t)s.groups * c.NT * 3 * c.chunks * c.Np * c.CK;
}

cudaError_t igemm_pack(const Shape& s, const float* w, void* packed, cudaStream_t st) {
    const IgemmCfg c = igemm_config(s, 148);
    const size_t total = (size_t)s.groups * c.NT * 3 * c.chunks * c.Np * c.CK;
    int blocks = (int)((total + 255) / 256 < 2368 ? (total + 255) / 256 : 2368);
    igemm_pack_kernel<<<blocks, 256, 0, st>>>(s, c, w, reinterpret_cast<uint32_t*>(packed), pack_tag(s, GCONV_VARIANT_IGEMM_TF32));
    return cudaGetLastError();
}

cudaError_t igemm_forward(const Shape& s, const float* x, const void* packed, float* y, Status* status, int sm_count,
                          cudaStream_t st) {
    const IgemmCfg c = igemm_config(s, sm_count);
    EncodeTiledFn encode = get_encode_fn();
    if (encode == nullptr) return cudaErrorNotSupported;
    CUtensorMap xmap;
    const cuuint64_t HW = (cuuint64_t)s.H * s.W;
    const cuuint64_t dims[3] = {HW, (cuuint64_t)s.C_in, (cuuint64_t)s.N};
    const cuuint64_t strides[2] = {HW * 4, HW * 4 * (cuuint64_t)s.C_in};
    const cuuint32_t box[3] = {32, (cuuint32_t)c.CK, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    const CUresult r = encode(&xmap, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float*>(x), dims, strides, box, estr,
                              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
    static bool attr_set[64] = {false};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64 || !attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(igemm_tf32_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) attr_set[dev] = true;
    }
    igemm_tf32_kernel<<<c.grid, kThreads, c.smem_bytes, st>>>(xmap, s, c, reinterpret_cast<const uint32_t*>(packed), y, status,
                                                              pack_tag(s, GCONV_VARIANT_IGEMM_TF32));
    return cudaGetLastError();
}


}  // namespace gconv
