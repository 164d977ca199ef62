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
//   * D lives in TMEM (3*Kt <= 192 fp32 columns, a ring of 2 to 4 accumulators), the epilogue warps read it with
//     tcgen05.ld, apply the horizontal shifts with warp shuffles and write y directly in NCHW with
//     128-byte coalesced rows.
// Stride 2 (pad 1) keeps the even rows and columns of that stride-1 result: same operands, the
// epilogue stores only those lanes; for widths 16..62 a tile is four OUTPUT rows and the odd input rows are never
// multiplied (their stage holds nine input rows, a tap is the view of every other one).
// All groups and all images run in one persistent launch: the tile index enumerates
// (group, filter tile, pixel tile).  Two launch shapes: one CTA per SM with all 21 warps ("heavy"), or two CTAs per SM
// of 11 warps each ("light": small filter banks, two accumulators in 256 TMEM columns, half the shared memory).
// The kernel body is written once against the run-time configuration and compiled in a few "families" whose mode
// fields are compile-time constants (see Family below); the host picks the instantiation.
//
// Warp roles: warp 0 = TMA producer, warps 1, 10 (and 19, 20 when four accumulators fit) = single-thread MMA issuers
// taking tiles in turn, each with its own accumulator buffer (warp 1 owns the TMEM allocation),
// warps 2..9 and 11..18 = two epilogue groups for alternate tiles (TMEM lane quarter = warp_id % 4); the light shape
// launches warps 0..10 only.
// Every mbarrier wait is bounded: when a
// wait runs out the kernel records GCONV_ERR_TIMEOUT, all roles leave their loops, outstanding bulk
// copies are waited for (bounded), TMEM is freed and the kernel returns.
#include <cuda.h>
#include <string.h>

#include "gconv_internal.h"

namespace gconv {

namespace {

constexpr int kEpiWarps = 8;             // warps of one epilogue group: two per TMEM lane quarter, each takes half of the filters
constexpr int kMmaWarp2 = 2 + kEpiWarps;     // second MMA-issuing warp (the first is warp 1)
constexpr int kEpi2First = kMmaWarp2 + 1;    // first warp of the second epilogue group
constexpr int kMmaWarp3 = kEpi2First + kEpiWarps;   // third and fourth MMA-issuing warps (used when four accumulators fit)
constexpr int kThreads = 32 * (kMmaWarp3 + 2);
constexpr int kSoftWarps = 4;        // copy warps of the gather producer, one per segment of a tile: warps kEpi2First ... in the light shape;
                                     // the heavy shape has twice as many (two per segment, half of a stage's channels each)
constexpr int kTmemCols = 512;
constexpr int kMaxAcc = 4;               // accumulator buffers in TMEM (ring), as many as fit 512 columns
// Decisions that shape the packed weights use this SM count, not the device's, so that packing and forward agree.
constexpr int kLayoutSMs = 148;
constexpr uint32_t kPrefetchUses = 2;   // stage fills (from the CTA's first on) whose input idle epilogue warps ask L2 for before the dependency wait
                                        // (measured on the 90-launch stack: none 0.660 ms, one 0.610, two 0.597, three 0.602, four 0.611, eight 0.619)
constexpr uint32_t kDefaultWaitUs = 1000000u;   // a wait gives up after one second unless the descriptor says otherwise
constexpr int kMaxDynSmem = 226 * 1024;   // 227 KB per CTA minus the static control block (under 1 KB)

struct __align__(8) SharedCtl {
    unsigned long long full[8];
    unsigned long long empty[8];
    unsigned long long tmem_full[kMaxAcc];
    unsigned long long tmem_empty[kMaxAcc];
    unsigned long long xchg_bar[kMaxAcc];
    unsigned long long b_full[2];   // resident weights of a (group, filter tile) have landed
    unsigned long long b_free[2];   // every MMA that read that weight buffer has completed
    // fused grouped + pointwise block: the grouped result of a tile goes through shared memory (a2, one buffer per
    // epilogue group) into a second MMA that accumulates the pointwise output of the pixel tile over all groups (d2)
    unsigned long long a2_full[2], a2_free[2], d2_full[2], d2_free[2], w2_full;
    unsigned long long raw_full[4], raw_empty[4];   // gather producer: ring of raw input buffers (bulk copies in, copy warps out)
    uint32_t tmem_base;
    int abort_flag;      // set by the first role whose wait ran out; every other role then leaves at its next wait
    uint32_t wait_us;    // time limit of one wait, in microseconds (read as abort_flag[1] by the wait helpers)
};
static_assert(offsetof(SharedCtl, wait_us) == offsetof(SharedCtl, abort_flag) + sizeof(int), "wait helpers read the limit behind the flag");

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

// Non-blocking probe (try_wait may suspend the thread for a hardware time limit while the phase is incomplete).
__device__ __forceinline__ uint32_t mbar_test_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok;
}

__device__ __forceinline__ uint64_t global_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

// Bounded wait: gives up after the CTA's time limit (one second by default).  Returns false if the wait ran out or
// another role already gave up; the first role to run out records GCONV_ERR_TIMEOUT with `where` as the detail.
//
// The polls follow each other as closely as they can.  Some waiters only OBSERVE a barrier that others drive (an MMA warp
// walking the other warp's stages, see there): a parity wait is only meaningful one phase at a time, so such a waiter must
// never be away from the barrier for as long as two phase flips take (a refill is a microsecond or more away).  The clock
// (a read of the global timer is slow) is therefore looked at only once every 128 polls.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, Status* status,
                                          int where) {
    if (mbar_try_wait(bar, parity)) return true;
    uint64_t limit_ns = 0, t0 = 0;
    for (uint32_t it = 0;; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if ((it & 127u) == 127u) {
            if (it == 127u) {
                limit_ns = 1000ull * (uint64_t)(uint32_t)abort_flag[1];
                t0 = global_ns();
            } else if (global_ns() - t0 > limit_ns) {
                break;
            }
        }
        if (it > 4096) __nanosleep(64);
    }
    *abort_flag = 1;
    record_status(status, GCONV_ERR_TIMEOUT, where);
    return false;
}

// Drain wait, used only after a role gave up: waits (same time limit) for a phase whose copies may still be in flight.
// Returns false if it ran out as well.
__device__ __forceinline__ bool mbar_drain(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    const uint64_t limit_ns = 1000ull * (uint64_t)(uint32_t)abort_flag[1];
    const uint64_t t0 = global_ns();
    while (!mbar_test_wait(bar, parity)) {
        if (global_ns() - t0 > limit_ns) return false;
        __nanosleep(64);
    }
    return true;
}

// The same wait for a converged warp: every lane gets the same answer, so the warp never splits
// around the warp-level primitives that follow.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, volatile int* abort_flag, Status* status,
                                               int where) {
    return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag, status, where) ? 1 : 0) != 0;
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, int c3, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, int c3, int c4,
                                            uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4), "r"(bar)
        : "memory");
}
// L2 prefetch of the same boxes (a cache hint: nothing is written, no barrier is involved)
__device__ __forceinline__ void tma_prefetch_3d(const CUtensorMap* map, int c0, int c1, int c2) {
    asm volatile("cp.async.bulk.prefetch.tensor.3d.L2.global.tile [%0, {%1, %2, %3}];" ::"l"(map), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
__device__ __forceinline__ void tma_prefetch_4d(const CUtensorMap* map, int c0, int c1, int c2, int c3) {
    asm volatile("cp.async.bulk.prefetch.tensor.4d.L2.global.tile [%0, {%1, %2, %3, %4}];" ::"l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
                 : "memory");
}
__device__ __forceinline__ void tma_prefetch_5d(const CUtensorMap* map, int c0, int c1, int c2, int c3, int c4) {
    asm volatile("cp.async.bulk.prefetch.tensor.5d.L2.global.tile [%0, {%1, %2, %3, %4, %5}];" ::"l"(map), "r"(c0), "r"(c1), "r"(c2),
                 "r"(c3), "r"(c4)
                 : "memory");
}
__device__ __forceinline__ void bulk_load_1d(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// One MMA: D[128 x N] (+)= A[128 x 8] * B[8 x N], TF32 in, FP32 accumulate in TMEM.  Each shared-memory descriptor is
// given as its two 32-bit halves: between MMAs only the low words change.
__device__ __forceinline__ void umma_tf32_split(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
                                                uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
        "mov.b64 da, {%1, %2};\n\t"
        "mov.b64 db, {%3, %4};\n\t"
        "setp.ne.b32 p, %6, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], da, db, %5, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(acc)
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


// tile index -> (gn = group * NT + filter tile, mt = pixel tile).  With resident weights the pixel tile runs
// fastest (a CTA keeps its weights across consecutive tiles); with streamed weights the filter tile runs fastest, so
// the NT tiles that read the same input block run at the same time and the re-reads hit L2 instead of HBM.
__device__ __forceinline__ void tile_coords(const IgemmCfg& c, uint32_t tile, uint32_t& gn, uint32_t& mt) {
    if (c.fuse) {                     // fused block: group fastest, a CTA takes all groups of a pixel tile in turn
        c.div_ngn.divmod(tile, mt, gn);
    } else if (c.nt_fast) {
        uint32_t gm, nt, g;
        c.div_nt.divmod(tile, gm, nt);
        c.div_mt.divmod(gm, g, mt);
        gn = g * (uint32_t)c.NT + nt;
    } else {
        c.div_mt.divmod(tile, gn, mt);
    }
}

// Gather tilings (c.soft).  A segment is `rps` whole output rows side by side in 32 lanes.  With at least three segments
// per image a tile is four consecutive segments of ONE image (TPI tiles per image, the last one possibly short) and its
// raw buffer holds one part: the input rows those segments need.  Smaller planes put IPT = 4 / SPI whole images into a
// tile, one part (whole plane) per image.
__device__ __forceinline__ void gath_segment(const IgemmCfg& c, uint32_t mt, int wq, int& n, int& i, int& part) {
    if (c.IPT == 1) {
        uint32_t nn, t;
        c.div_spi.divmod(mt, nn, t);              // div_spi divides by the tiles per image
        n = (int)nn;
        i = (int)t * 4 + wq;
        part = 0;
    } else {
        part = c.SPI == 2 ? (wq >> 1) : wq;
        i = c.SPI == 2 ? (wq & 1) : 0;
        n = (int)mt * c.IPT + part;
    }
}
// Part `part` of tile mt's raw buffer: the image it is read from and the flat pixel (a multiple of 4) it starts at.
__device__ __forceinline__ void gath_part(const Shape& s, const IgemmCfg& c, uint32_t mt, int part, int& n, int& fa) {
    fa = 0;
    if (c.IPT == 1) {
        uint32_t nn, t;
        c.div_spi.divmod(mt, nn, t);
        n = (int)nn;
        if (!c.raw_whole) {
            const int p0 = (int)t * 4 * c.rps;    // first output row of the tile
            int h_lo = c.soft == 2 ? 2 * p0 - 1 : p0 - s.dilation;
            if (h_lo < 0) h_lo = 0;
            fa = (h_lo * s.W) & ~3;
        }
    } else {
        n = (int)mt * c.IPT + part;
    }
}

// Families: sets of configuration fields fixed at compile time (-1 = left to the run-time configuration).  The kernel
// body is written once against the run-time configuration; a family instantiation overwrites the listed fields of a
// local copy with constants, and the compiler drops every path they rule out.  The role code is a single warp (often a
// single thread) walking branchy set-up code a handful of times per launch, so on short layers the shorter
// instruction stream matters: the 8x8 layers of the WRN stack run 20 % faster on their family than on family 0.
struct Family {
    int rowbox, seg_mode, nr, need_xchg, b_res, egroups, s2h, lbo_segs, stride, CK, chunks, Kt, Np, NT, nacc, issuers, padded,
        nt_fast, wseg, nseg, SR, fast4, tapb, fuse, ball, soft, pw, pair;   // (pair: 0 where a row leaves it out)
};
constexpr int kFamilies = 31;
__host__ __device__ constexpr Family family(int f) {
    //                 rowbox seg nr xchg bres egr s2h lbo str CK  ch  Kt  Np  NT acc iss pad ntf wseg nseg SR f4 tapb fuse ball soft pw
    return f == 1 ? Family{0,   1,  1,  0,   1,  1,  0,  1,  1, 32,  1, 32,  96,  1,  2,  2, -1,  0,  0,   4,  0, -1,  0,  0,  0,  0,  0}     // 16x16 / 8x8 planes, narrow groups
         : f == 2 ? Family{0,   1,  3,  0,   1,  1,  0,  1,  1, 32,  1, 32,  96,  1,  2,  2,  0,  0,  1,   6,  0,  2,  0,  0,  0,  0,  0}     // 32-wide planes with halo stages
         : f == 3 ? Family{1,   0,  3,  0,   1,  1,  0,  1,  1, 16,  2, 32,  96,  1,  2,  2, -1,  0,  2,   8,  2,  1,  0,  0,  0,  0,  0}     // row boxes of two segments, narrow groups, 16-channel stages
         : f == 4 ? Family{1,   0,  3,  0,   0,  2,  1,  2,  2, 32, -1, 64, 192, -1,  2,  2, -1, -1,  1,   9,  1,  1,  0,  0,  0,  0,  0}     // stride-2 row tiles, 64-filter tiles, streamed weights
         : f == 5 ? Family{1,   0,  3,  0,   1,  1,  1,  2,  2, 32,  1, 32,  96,  1,  2,  2, -1,  0,  1,   9, -1,  1,  0,  0,  0,  0,  0}     // stride-2 row tiles, narrow groups
         : f == 6 ? Family{1,   0,  3,  0,   0,  2,  0,  1,  1, 32, -1, 64, 192, -1,  2,  2, -1, -1, -1,  -1, -1,  1,  0,  0,  0,  0,  0}     // row boxes, 64-filter tiles, streamed weights
         : f == 7 ? Family{1,   0,  3,  0,   1,  2,  0,  1,  1, 32, -1, 64, 192,  1,  2,  2, -1,  0, -1,  -1, -1,  1,  0,  0,  0,  0,  0}     // row boxes, 64-filter tiles, one resident bank
         : f == 8 ? Family{0,   1,  1,  0,   0,  2,  0,  1,  1, 32, -1, 64, 192, -1,  2,  2, -1, -1,  0,   4,  0, -1,  0,  0,  0,  0,  0}     // 16x16 / 8x8 planes, 64-filter tiles, streamed weights
         : f == 9 ? Family{1,   0,  3,  0,   1,  1,  0,  1,  1, 16,  2, 32,  96,  1,  2,  2, -1,  0,  1,   6,  1,  1,  0,  0,  0,  0,  0}     // row boxes of one segment, narrow groups, 16-channel stages
         : f == 10 ? Family{0,  1,  3,  0,   1,  1,  0,  1,  1, 32,  1, 32,  96,  1,  2,  2, -1,  0,  4,  12,  0,  0,  1,  0,  0,  0,  0}     // 16x16 / 8x8 planes, narrow groups, tap blocks
         : f == 11 ? Family{0,  1,  3,  0,   1,  2,  0,  1,  1, 32,  1, 32,  96,  1,  2,  2,  0,  0,  1,   6,  0,  2,  0,  1,  0,  0,  0}     // fused block, 32-wide planes with halo stages
         : f == 12 ? Family{0,  1,  1,  0,   2,  2,  0,  1,  1, 32,  1, 32,  96,  1,  2,  2,  0,  0,  0,   4,  0, -1,  0,  1, -1,  0,  0}     // fused block, 16x16 / 8x8 planes, two resident banks (switching, or one per group)
         : f == 13 ? Family{0,  1,  3,  0,   1,  1,  0,  1,  1, 32,  1, 32,  96,  1,  2,  1,  0,  0,  1,   6,  0,  2,  0,  1,  0,  0,  0}     // fused block, 32-wide planes, two CTAs per SM
         : f == 14 ? Family{1,  0,  3,  0,   2,  2,  0,  1,  1, 32,  1, 32,  96,  1,  2,  2, -1,  0, -1,  -1, -1,  1,  0,  1, -1,  0,  0}     // fused block, row boxes, two resident banks
         : f == 15 ? Family{0,  0,  3,  0,   1,  1,  0,  1,  1, 16, -1, -1,  -1, -1,  2,  2,  0,  0,  4,  12,  0, -1,  0,  0,  0,  1,  0}     // gather producer, stride 1 (14x14, 7x7, ... planes), narrow groups, 16-channel stages
         : f == 16 ? Family{0,  0,  3,  0,   1,  1,  0,  1,  2, 16, -1, -1,  -1, -1,  2,  2,  0,  0,  8,  24,  0, -1,  0,  0,  0,  2,  0}     // gather producer, stride 2 (even/odd column blocks), narrow groups, 16-channel stages
         : f == 17 ? Family{0, 1, 1, 0, 1, 1, 0, 1, -1, 32, -1, -1, -1, -1, 2, 2, 0, 0, 0, 4, 0, -1, 0, 0, 0, 0, 1}     // pointwise, segment tilings, two CTAs per SM
         : f == 18 ? Family{1, 0, 1, 0, -1, -1, 0, 1, -1, 32, -1, -1, -1, -1, -1, -1, 0, -1, 0, 4, -1, 1, 0, 0, 0, 0, 1}     // pointwise, row boxes
         : f == 19 ? Family{0, 1, 1, 0, -1, -1, 0, 1, -1, 32, -1, -1, -1, -1, -1, -1, 0, -1, 0, 4, 0, -1, 0, 0, 0, 0, 1}     // pointwise, segment tilings, one CTA per SM
         : f == 20 ? Family{1,   0,  3,  0,   1,  1,  1,  2,  2, 16,  1, 32,  96,  1,  2,  2, -1,  0,  1,   9, -1,  1,  0,  0,  0,  0,  0}     // stride-2 row tiles, 16-channel merged groups (channel-doubling transitions)
         : f == 21 ? Family{1,   0,  3,  0,   0,  2,  0,  1,  1, 16, -1, 64, 192, -1,  1,  1, -1, -1, -1,  -1, -1,  1,  0,  0,  0,  0,  0,  1}     // row boxes, 64-filter tiles, streamed weights shared by a pair of pixel tiles
         : f == 22 ? Family{1,   0,  3,  0,   1,  2,  1,  2,  2, 32, -1, 64, 192, -1,  2,  2, -1,  0,  1,   9, -1,  1,  0,  0,  0,  0,  0,  0}     // stride-2 row tiles, 64-filter tiles, one resident bank
         : f == 23 ? Family{1,   0,  3,  0,   1,  2,  0,  1,  1, 16, -1, 64, 192,  1,  2,  2, -1,  0, -1,  -1, -1,  1,  0,  0,  0,  0,  0,  0}     // row boxes, 64-filter tiles, one large resident bank, 16-channel stages
         : f == 24 ? Family{1,   0,  3,  0,   1,  2,  1,  2,  2, 16, -1, 64, 192, -1,  2,  2, -1,  0,  1,   9, -1,  1,  0,  0,  0,  0,  0,  0}     // stride-2 row tiles, one resident 64-filter bank, 16-channel stages
         : f == 25 ? Family{1,   0,  3,  0,   0,  2,  1,  2,  2, 16, -1, 64, 192, -1,  2,  2, -1, -1,  1,   9, -1,  1,  0,  0,  0,  0,  0,  0}     // stride-2 row tiles, 64-filter tiles, streamed weights, 16-channel stages
         : f == 26 ? Family{0,   0,  3,  0,   1,  1,  0,  1,  1,  8, -1, -1,  -1, -1,  2,  2,  0,  0,  4,  12,  0, -1,  0,  0,  0,  1,  0,  0}     // gather producer, stride 1, 8-channel stages
         : f == 27 ? Family{0,   0,  3,  0,   1,  1,  0,  1,  2,  8, -1, -1,  -1, -1,  2,  2,  0,  0,  8,  24,  0, -1,  0,  0,  0,  2,  0,  0}     // gather producer, stride 2, 8-channel stages
         : f == 28 ? Family{0,   0,  3,  0,  -1,  2,  0,  1,  1, 16, -1, 64, 192, -1,  2,  2,  0, -1,  4,  12,  0, -1,  0,  0,  0,  1,  0,  0}     // gather producer, stride 1, wide groups (one CTA per SM, 29 warps)
         : f == 29 ? Family{0,   0,  3,  0,   0,  2,  0,  1,  2,  8, -1, 64, 192, -1,  1,  1,  0, -1,  8,  24,  0, -1,  0,  0,  0,  2,  0,  1}     // gather producer, stride 2, wide groups, 8-channel stages, streamed weights shared by a pair of pixel tiles
         : f == 30 ? Family{0,   0,  3,  0,   0,  2,  0,  1,  1, 16, -1, 64, 192, -1,  1,  1,  0, -1,  4,  12,  0, -1,  0,  0,  0,  1,  0,  1}     // gather producer, stride 1, wide groups, streamed weights shared by a pair of pixel tiles
                  : Family{-1, -1, -1, -1,  -1, -1, -1, -1, -1, -1, -1, -1,  -1, -1, -1, -1, -1, -1, -1,  -1, -1, -1, -1, -1, -1, -1, -1, -1};
}
#define GCONV_FAMILY_FIELDS(X) \
    X(rowbox) X(seg_mode) X(nr) X(need_xchg) X(b_res) X(egroups) X(s2h) X(lbo_segs) X(CK) X(chunks) X(Kt) X(Np) X(NT) X(nacc) X(issuers) \
    X(padded) X(nt_fast) X(wseg) X(nseg) X(SR) X(fast4) X(tapb) X(fuse) X(ball) X(soft) X(pw) X(pair)

static bool family_matches(int f, const Shape& s, const IgemmCfg& c) {
    const Family fam = family(f);
#define GCONV_CHK(field) if (fam.field >= 0 && c.field != fam.field) return false;
    GCONV_FAMILY_FIELDS(GCONV_CHK)
#undef GCONV_CHK
    if (fam.stride >= 0 && s.stride != fam.stride) return false;
    return s.dilation == 1;          // every family fixes dilation 1; dilated layers run the generic instantiation
}

__device__ __forceinline__ void
igemm_tf32_body(const CUtensorMap& xmap, const CUtensorMap& xmap4, const Shape& s, const IgemmCfg& c,
                const uint32_t* __restrict__ packed, float* __restrict__ y, Status* status, uint32_t tag,
                const float* __restrict__ x) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    __shared__ SharedCtl ctl;
    static_assert(sizeof(SharedCtl) <= 1024, "control block must leave 226 KB of dynamic shared memory");

    // Programmatic dependent launch: let the next kernel in the stream be scheduled as SMs free up, and run this
    // kernel's own set-up (barriers, TMEM) while the previous kernel drains.  Before griddepcontrol.wait has
    // returned (the previous kernel's writes complete and visible) the only global memory read is the packed weights
    // (their tag here, the first resident bank in the producer).  Only the dependency wait guarantees that an earlier
    // kernel's writes are visible, so the host launches the first forward after ANY weight packing of the process
    // without programmatic serialization (a full stream dependency); by every later launch the weights are older than
    // a completed kernel boundary.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const uint32_t tag_seen = __ldg(packed);
    const uint8_t* __restrict__ wblocks = reinterpret_cast<const uint8_t*>(packed) + kHeaderBytes;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t smem_base = smem_u32(smem);
    volatile int* abort_flag = &ctl.abort_flag;
    float (*xchg)[4][2][64] = reinterpret_cast<float (*)[4][2][64]>(smem + c.xchg_off);   // edge-lane exchange (flat row tiles only)

    // Set-up.  The producer warp initialises every barrier itself and goes straight on to its copies: it needs neither the
    // tensor-memory address nor anybody else's work, and on a short layer its first copy is the head of the critical path.
    // It only ARRIVES on the set-up barrier (named barrier 1); the other warps wait there for the barriers and for warp 1's
    // tensor-memory allocation.
    if (warp == 0) {
        // The barriers are consecutive 8-byte words at the head of the control block; lane j initialises numbers j and
        // j + 32 with a count picked by selects (no divergent branches: this warp is alone on the critical path here).
        // Barriers a configuration does not use are initialised too; nobody touches them.
        constexpr int kBarriers = (int)(offsetof(SharedCtl, tmem_base) / 8);
        static_assert(offsetof(SharedCtl, full) == 0 && kBarriers <= 64, "barriers first, at most two per lane");
        const uint32_t n_copy = (uint32_t)kSoftWarps * (uint32_t)c.egroups;                 // copy warps of the gather producer
        const uint32_t n_full = c.soft ? n_copy + (c.b_res ? 0u : 1u) : 1u;                 // copy warps (+ the streamed weights' arm)
        const uint32_t n_tmem_empty = c.pair ? 2u * kEpiWarps : (uint32_t)kEpiWarps;         // pair tiles: both groups drain the buffer
#pragma unroll
        for (int round = 0; round < 2; ++round) {
            const int t = lane + 32 * round;
            const int w8 = t * 8;                       // byte offset of barrier t
            uint32_t n = 1u;
            n = (w8 >= (int)offsetof(SharedCtl, full) && w8 < (int)offsetof(SharedCtl, empty)) ? n_full : n;
            n = (w8 >= (int)offsetof(SharedCtl, empty) && w8 < (int)offsetof(SharedCtl, tmem_full)) ? (uint32_t)c.issuers : n;   // the consumer's MMAs and every observer
            n = (w8 >= (int)offsetof(SharedCtl, tmem_empty) && w8 < (int)offsetof(SharedCtl, xchg_bar)) ? n_tmem_empty : n;
            n = (w8 >= (int)offsetof(SharedCtl, xchg_bar) && w8 < (int)offsetof(SharedCtl, b_full)) ? (uint32_t)kEpiWarps : n;
            n = (w8 >= (int)offsetof(SharedCtl, b_free) && w8 < (int)offsetof(SharedCtl, a2_full)) ? (uint32_t)c.issuers : n;
            n = (w8 >= (int)offsetof(SharedCtl, a2_full) && w8 < (int)offsetof(SharedCtl, a2_free)) ? (uint32_t)kEpiWarps : n;
            n = (w8 >= (int)offsetof(SharedCtl, d2_free) && w8 < (int)offsetof(SharedCtl, w2_full)) ? (uint32_t)kEpiWarps : n;
            n = (w8 >= (int)offsetof(SharedCtl, raw_empty) && w8 < (int)offsetof(SharedCtl, tmem_base)) ? n_copy : n;
            if (t < kBarriers) mbar_init(smem_u32(&ctl) + (uint32_t)w8, n);
        }
        if (lane == 0) {
            ctl.abort_flag = 0;
            ctl.wait_us = c.wait_us;
        }
        // the bulk copies complete on these barriers through the async proxy and may be issued a few instructions from
        // here: the initialisations have to be visible to that proxy, not only to the other threads
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        asm volatile("barrier.arrive 1, %0;" ::"r"((uint32_t)blockDim.x) : "memory");
    } else {
        if (warp == 1) {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl.tmem_base)),
                         "r"((uint32_t)c.tmem_cols)
                         : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
        tc_fence_before();
        asm volatile("barrier.sync 1, %0;" ::"r"((uint32_t)blockDim.x) : "memory");
        tc_fence_after();
    }
    const uint32_t tmem_base = warp == 0 ? 0u : ctl.tmem_base;   // (the producer never touches tensor memory)
    const bool tag_ok = (tag_seen == tag);   // uniform across the CTA
    // Tiles of this CTA: every gridDim.x-th tile, or -- with resident weights and several (group, filter tile) pairs --
    // the CTAs split into one set per pair, each set striding over that pair's pixel tiles: no CTA ever switches
    // weights, and the CTAs of a set still read neighbouring pixels at the same time.
    int tile_first = (int)blockIdx.x, tile_end = c.num_tiles, tile_step = (int)gridDim.x;
    if (c.fuse) tile_first = (int)blockIdx.x * c.n_gn;    // tile = pixel tile * n_gn + group; see tile_next
    // next tile of this CTA: every gridDim.x-th tile, or (fused block) the next group of the pixel tile and, after
    // its last group, the first group of the pixel tile gridDim.x further on
    auto tile_next = [&](int tile) -> int {
        if (!c.fuse) return tile + tile_step;
        uint32_t mt, gn;
        c.div_ngn.divmod((uint32_t)tile, mt, gn);
        return (int)gn + 1 == c.n_gn ? tile + 1 + ((int)gridDim.x - 1) * c.n_gn : tile + 1;
    };
    if (c.cps > 0) {
        const int set = (int)blockIdx.x / c.cps;
        tile_first = set * c.MT + ((int)blockIdx.x - set * c.cps);
        tile_end = (set + 1) * c.MT;
        tile_step = c.cps;
    }

    // Pipeline geometry.  A stage holds the input segments of one channel chunk: either the four
    // segments of one vertical tap (nr = 1, stages run chunk-major, tap-minor), or the tile plus its
    // row halo (nr = 3: the three taps are views of the same stage, shifted by whole segments).
    const int vt = c.pw ? 1 : 3;                 // vertical taps (a pointwise layer has one tap, no neighbours)
    const int kstages = (vt / c.nr) * c.chunks;
    const uint32_t seg_bytes = (uint32_t)c.CK * 128u;
    const uint32_t a_bytes = (uint32_t)c.nseg * seg_bytes;
    const uint32_t a_all = c.pair ? 2u * a_bytes : a_bytes;   // pair tiles: the second tile's input sits behind the first's
    const uint32_t blk_bytes = (uint32_t)c.Np * (uint32_t)c.CK * 4u;   // weights of one (chunk, tap)
    const uint32_t b_tile_bytes = (uint32_t)vt * (uint32_t)c.chunks * blk_bytes;   // weights of one (group, filter tile)
    const uint32_t bres_base = smem_base;                                // two resident weight buffers (if b_res)
    const uint32_t stage_base = smem_base + (uint32_t)c.b_res * c.bres_stride;   // b_res = number of resident weight buffers
    const int HW = s.H * s.W;
    const int rstep = s.W * s.dilation;          // flat-pixel distance between vertical taps
    const size_t OHW = (size_t)s.H_out * s.W_out;

    bool run_epilogue = false;
    if (!tag_ok) {
        // wrong weights: no role runs, y stays untouched; fall through to the common exit (TMEM is freed there)
        asm volatile("griddepcontrol.wait;" ::: "memory");
        if (threadIdx.x == 0) record_status(status, GCONV_ERR_PACK_MISMATCH, (int)blockIdx.x);
    } else if (warp == 0 || (warp >= 2 && warp < 2 + kEpiWarps && !c.soft)) {
        // ---------------------------------------------------------------- TMA producer (warp 0)
        // The whole warp walks the tiles; lane j issues the copy of segment j, lane 0 arms the barriers.
        // Warp 2, an epilogue warp with nothing to do yet, runs the same tile walk once as a prefetch pass (see below) and
        // then goes on to its epilogue role.
        const bool producer = warp == 0;
        uint32_t it = 0, switches = 0;
        int stage = 0;
        uint32_t ph = 0;                                   // phase parity of the current pass over the stage ring
        int cur_gn = -1;
        bool ok = true;
        if (lane == 0) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(&xmap) : "memory");
            if (c.fast4 || c.rowbox) asm volatile("prefetch.tensormap [%0];" ::"l"(&xmap4) : "memory");
        }
        if (producer && c.b_res && tile_first < tile_end) {
            // The first tile's resident weights do not depend on the previous kernel: fetch them before waiting for it.
            uint32_t gn, mt;
            tile_coords(c, (uint32_t)tile_first, gn, mt);
            const uint8_t* wtile = wblocks + (size_t)gn * b_tile_bytes;
            const uint32_t bar = smem_u32(&ctl.b_full[0]);
            if (lane == 0) mbar_arrive_expect_tx(bar, b_tile_bytes);
            __syncwarp();
            for (uint32_t blk = lane; blk < (uint32_t)vt * (uint32_t)c.chunks; blk += 32)
                bulk_load_1d(bres_base + blk * blk_bytes, wtile + (size_t)blk * blk_bytes, blk_bytes, bar);
            cur_gn = (int)gn;
            switches = 1;
            if (c.ball) {
                // every (group, filter tile) has a resident buffer of its own: fetch the second bank too, nothing ever switches
                const uint32_t bar1 = smem_u32(&ctl.b_full[1]);
                if (lane == 0) mbar_arrive_expect_tx(bar1, b_tile_bytes);
                __syncwarp();
                for (uint32_t blk = lane; blk < (uint32_t)vt * (uint32_t)c.chunks; blk += 32)
                    bulk_load_1d(bres_base + c.bres_stride + blk * blk_bytes, wblocks + (size_t)b_tile_bytes + (size_t)blk * blk_bytes, blk_bytes, bar1);
                switches = 2;
            }
        }
        if (producer && c.fuse) {
            // the pointwise weights of every group stay resident (they come from the packing kernel too)
            const uint32_t bar = smem_u32(&ctl.w2_full);
            const uint32_t w2_blk = (uint32_t)c.Kt * (uint32_t)c.C2 * 4u;
            if (lane == 0) mbar_arrive_expect_tx(bar, w2_blk * (uint32_t)c.n_gn);
            __syncwarp();
            for (int blk = lane; blk < c.n_gn; blk += 32)
                bulk_load_1d(smem_base + c.w2_off + (uint32_t)blk * w2_blk,
                             reinterpret_cast<const uint8_t*>(packed) + c.w2_goff + (size_t)blk * w2_blk, w2_blk, bar);
        }
        // Two walks over the tiles.  The prefetch walk (warp 2, before its own dependency wait) only asks L2 to fetch the
        // input box of the first stage: a cache hint, nothing is consumed, and L2 is the point of coherence, so it stays
        // correct if the previous kernel is still writing those lines (then they are in L2 already).  The CTA usually
        // sits in the wait while the previous kernel's last CTAs finish; the first copy after the wait then comes from L2
        // instead of starting a DRAM round trip.  The walk used to run on the producer warp ahead of the real one and cost
        // it 1 500 cycles (a single warp walking branchy code retires an instruction every five to ten cycles) before the
        // first real copy; now the epilogue warps of the first group share it (warp 2 + j takes fill j).  Asking for more
        // than two fills competes with the previous kernel's own traffic and loses again (kPrefetchUses).  The real walk
        // is the producer's.
        // One tile's stages: the real copies (arming the stage barriers), or -- pf -- only L2 prefetches of the first
        // pf_limit of them (no barrier).  (Asking L2 for the CTA's next tile while the current one is in flight was
        // measured too: 2 % slower on the stack.)
        // The dependency wait sits directly in front of the producer's first input copy: tile coordinates, barrier and
        // buffer addresses of that copy are worked out while the previous kernel is still running, so that what follows
        // the release of the wait is the copy itself (the producer is one warp walking this code alone: the set-up of a
        // stage is some hundred instructions, about 600 cycles, in front of every kernel's first load otherwise).
        bool dep_pending = true;
        auto visit = [&](const int tile, const bool pf, const uint32_t pf_limit, uint32_t& it, int& stage, uint32_t& ph) {
            uint32_t gn, mt;
            tile_coords(c, (uint32_t)tile, gn, mt);      // gn = (group, filter tile) index
            uint32_t gq = gn, ntq = 0;
            if (c.NT > 1) c.div_nt.divmod(gn, gq, ntq);
            const int g = (int)gq;
            const uint8_t* wtile = wblocks + (size_t)gn * b_tile_bytes;
            const bool switch_b = !pf && c.b_res && !c.ball && (int)gn != cur_gn;
            if (c.soft) {
                // Gather producer: this warp brings the resident weights of a new (group, filter tile) and, per stage, the
                // raw input of the tile's parts into the raw ring (tiled boxes of flat pixels x channels, or one bulk copy
                // of whole planes where the plane is not a multiple of 16 bytes) plus -- with streamed weights -- the
                // stage's weight blocks.  The copy warps turn raw buffers into operand stages.
                if (switch_b) {
                    const uint32_t bb = c.b_res == 2 ? (switches & 1) : 0u, use = c.b_res == 2 ? (switches >> 1) : switches;
                    if (!mbar_wait_warp(smem_u32(&ctl.b_free[bb]), (use & 1) ^ 1, abort_flag, status, 600 + bb)) { ok = false; return; }
                    const uint32_t bar = smem_u32(&ctl.b_full[bb]);
                    if (lane == 0) mbar_arrive_expect_tx(bar, b_tile_bytes);
                    __syncwarp();
                    for (uint32_t blk = lane; blk < (uint32_t)vt * (uint32_t)c.chunks; blk += 32)
                        bulk_load_1d(bres_base + bb * c.bres_stride + blk * blk_bytes, wtile + (size_t)blk * blk_bytes, blk_bytes, bar);
                    cur_gn = (int)gn;
                    ++switches;
                }
                const uint32_t piece_bytes = (uint32_t)c.CK * (uint32_t)c.boxpx * 4u;
                const uint32_t part_bytes = (uint32_t)c.pieces * piece_bytes;
                // pair tiles: a stage (and a raw buffer) holds two pixel tiles, 2 mt and 2 mt + 1, one behind the other
                const int npt = c.pair ? 2 : 1;
                const uint32_t mt0 = (uint32_t)npt * mt;
                for (int ks = 0; ks < kstages; ++ks, ++it) {
                    const uint32_t rs = it % (uint32_t)c.raw_stages, ruse = it / (uint32_t)c.raw_stages;
                    if (ruse > 0 && !mbar_wait_warp(smem_u32(&ctl.raw_empty[rs]), (ruse - 1) & 1u, abort_flag, status, 150 + (int)rs)) { ok = false; break; }
                    const uint32_t rbar = smem_u32(&ctl.raw_full[rs]);
                    const uint32_t rdst = smem_base + c.raw_off + rs * c.raw_bytes;
                    const int chan = g * c.Cg + ks * c.CK;
                    if (dep_pending) {
                        asm volatile("griddepcontrol.wait;" ::: "memory");   // the input may be the previous kernel's output
                        dep_pending = false;
                    }
                    if (c.raw_bulk) {
                        // whole planes of CK consecutive channels are one contiguous run of the input tensor
                        uint32_t live = 0;
                        for (int pt = 0; pt < npt * c.IPT; ++pt) {
                            int n, fa;
                            gath_part(s, c, mt0 + (uint32_t)(pt / c.IPT), pt % c.IPT, n, fa);
                            live += n < s.N ? 1u : 0u;
                        }
                        if (lane == 0) mbar_arrive_expect_tx(rbar, live * part_bytes);
                        __syncwarp();
                        if (lane < npt * c.IPT) {
                            int n, fa;
                            gath_part(s, c, mt0 + (uint32_t)(lane / c.IPT), lane % c.IPT, n, fa);
                            if (n < s.N)
                                bulk_load_1d(rdst + (uint32_t)lane * part_bytes, x + ((size_t)n * s.C_in + (size_t)chan) * (size_t)HW, part_bytes, rbar);
                        }
                    } else {
                        if (lane == 0) mbar_arrive_expect_tx(rbar, (uint32_t)(npt * c.IPT) * part_bytes);   // out-of-range boxes arrive as zeros
                        __syncwarp();
                        if (lane < npt * c.IPT * c.pieces) {
                            const int pt = lane / c.pieces, pc = lane - pt * c.pieces;   // pt counts the parts of both tiles
                            int n, fa;
                            gath_part(s, c, mt0 + (uint32_t)(pt / c.IPT), pt % c.IPT, n, fa);
                            tma_load_3d(rdst + (uint32_t)pt * part_bytes + (uint32_t)pc * piece_bytes, &xmap4, fa + pc * c.boxpx, chan, n, rbar);
                        }
                    }
                    if (!c.b_res) {
                        if (it >= (uint32_t)c.stages && !mbar_wait_warp(smem_u32(&ctl.empty[stage]), ph ^ 1, abort_flag, status, 100 + stage)) { ok = false; break; }
                        const uint32_t nb = (uint32_t)c.nr * blk_bytes;
                        const uint32_t full = smem_u32(&ctl.full[stage]);
                        if (lane == 0) {
                            mbar_arrive_expect_tx(full, nb);
                            bulk_load_1d(stage_base + (uint32_t)stage * c.stage_bytes + a_all, wtile + (size_t)ks * nb, nb, full);
                        }
                    }
                    if (++stage == c.stages) { stage = 0; ph ^= 1; }
                }
                return;
            }
            // Whole-tile copies: a row-box tile is always one 5-D box; a flat tile whose segments are one contiguous run
            // is one 4-D box for every tap whose run stays inside the image plane.  Everything else (tiles that straddle
            // images, and the plane's first/last tiles, whose out-of-plane part must be zero-filled) is copied segment
            // by segment, lane j issuing segment j with its own (image, first pixel).
            const bool whole = c.rowbox || c.fast4;
            int tile_n = 0, tile_f0 = 0, rb_row0 = 0, rb_seg = 0;
            int tile_n1 = 0, rb_row1 = 0, rb_seg1 = 0;   // pair tiles: the second pixel tile of the pair (row boxes, stride 1)
            if (c.pair) {
                mt *= 2u;
                uint32_t n, i;
                c.div_spi.divmod(mt + 1u, n, i);         // past the last tile: the image index is out of range, the box reads as zeros
                tile_n1 = (int)n;
                rb_row1 = (int)i * c.R - 1;
            }
            if (whole) {
                uint32_t n, i;
                c.div_spi.divmod(c.seg_mode ? mt * 4u : mt, n, i);
                tile_n = (int)n;
                if (c.rowbox && c.s2h) {                 // stride 2: four output rows of one row segment, input rows 2p - 1 .. 2p + 7
                    const int pb = c.SR == 2 ? (int)(i >> 1) : (int)i;
                    rb_seg = c.SR == 2 ? (int)(i & 1u) : 0;
                    rb_row0 = 8 * pb - 1;
                } else if (c.rowbox) rb_row0 = (int)i * c.R - (c.pw ? 0 : 1);    // the row above the tile's first row (pointwise: the first row)
                else tile_f0 = c.seg_mode ? (int)i * 32 : (int)i * c.R * s.W;    // first flat pixel of the tile
            }
            int my_n = 0, my_f = 0;
            bool have_lane_coords = false;
            int ch = 0, r = (c.nr == 3 || c.pw) ? 1 : 0;   // r = 1: the centre tap (row offset 0)
            for (int ks = 0; ks < kstages; ++ks, ++it) {
                if (pf && it >= pf_limit) break;
                if (pf && (it & (uint32_t)(kEpiWarps - 1)) != (uint32_t)(warp - 2)) {   // the prefetch walk is shared: warp 2 + j takes fills j, j + 8, ...
                    if (c.nr == 3 || c.pw) { ++ch; } else if (++r == 3) { r = 0; ++ch; }
                    continue;
                }
                // the first pass over the ring finds every stage free
                if (!pf && it >= (uint32_t)c.stages && !mbar_wait_warp(smem_u32(&ctl.empty[stage]), ph ^ 1, abort_flag, status, 100 + stage)) { ok = false; break; }
                const uint32_t full = smem_u32(&ctl.full[stage]);
                const uint32_t a_dst = stage_base + (uint32_t)stage * c.stage_bytes;
                const uint32_t nb = c.b_res ? 0u : (uint32_t)c.nr * blk_bytes;
                const int chan = g * c.Cg + ch * c.CK;
                // Failure-path test hook (gconv_desc_set_debug): CTA 0 leaves out one stage fill entirely -- no copy is
                // issued and the barrier is not armed -- so the consumer's bounded wait on that stage runs out.
                const bool skip_fill = !pf && (int)it == c.dbg_skip && blockIdx.x == 0;
                const int lo = tile_f0 + (r - 1) * rstep - c.wseg * 32;
                const bool box = c.rowbox || c.fast4 == 2 || (c.fast4 == 1 && lo >= 0 && lo + c.nseg * 32 <= HW);
                if (!pf && dep_pending) {
                    asm volatile("griddepcontrol.wait;" ::: "memory");   // the input may be the previous kernel's output
                    dep_pending = false;
                }
                if (skip_fill) {
                    // nothing
                } else if (lane == 0 && pf) {
                    if (box) {
                        if (c.rowbox) tma_prefetch_5d(&xmap4, 0, chan, rb_seg, rb_row0, tile_n);
                        else if (c.fast4 == 2) tma_prefetch_4d(&xmap4, 0, chan, lo >> 5, tile_n);
                        else tma_prefetch_4d(&xmap4, lo, chan, 0, tile_n);
                    }
                } else if (lane == 0) {
                    mbar_arrive_expect_tx(full, a_all + nb);
                    if (box) {
                        if (c.rowbox) {
                            tma_load_5d(a_dst, &xmap4, 0, chan, rb_seg, rb_row0, tile_n, full);   // rows above/below and columns past W: zero fill
                            if (c.pair) tma_load_5d(a_dst + a_bytes, &xmap4, 0, chan, rb_seg1, rb_row1, tile_n1, full);
                        }
                        else if (c.fast4 == 2) tma_load_4d(a_dst, &xmap4, 0, chan, lo >> 5, tile_n, full);   // segments outside the plane read as zeros
                        else tma_load_4d(a_dst, &xmap4, lo, chan, 0, tile_n, full);
                    }
                    if (nb) bulk_load_1d(a_dst + a_all, wtile + (size_t)ks * nb, nb, full);
                }
                if (!box && !skip_fill) {
                    if (!have_lane_coords) {
                        uint32_t n, i;
                        if (c.tapb) {                      // lane = 4 * tap + segment: the tap's own row shift, any image
                            c.div_spi.divmod(mt * 4u + (uint32_t)(lane & 3), n, i);
                            my_n = (int)n < s.N ? (int)n : s.N;
                            my_f = (int)i * 32 + ((lane >> 2) - 1) * s.W;
                        } else if (c.nr == 3) {            // tile plus halo: contiguous segments of one image
                            c.div_spi.divmod(c.seg_mode ? mt * 4u : mt, n, i);
                            my_n = (int)n;
                            my_f = (c.seg_mode ? (int)i * 32 : (int)i * c.R * s.W) + (lane - c.wseg) * 32;
                        } else if (c.seg_mode) {
                            c.div_spi.divmod(mt * 4u + (uint32_t)(lane & 3), n, i);
                            my_n = (int)n < s.N ? (int)n : s.N;   // past the last image: fully out of bounds, zero fill
                            my_f = (int)i * c.seg_fstep;
                        } else {
                            c.div_spi.divmod(mt, n, i);
                            my_n = (int)n;
                            my_f = (int)i * c.R * s.W + 32 * (lane & 3);
                        }
                        have_lane_coords = true;
                    }
                    __syncwarp();                          // the barrier is armed before any lane's copy can complete on it
                    if (lane < c.nseg) {
                        if (pf) tma_prefetch_3d(&xmap, my_f + (r - 1) * rstep, chan, my_n);
                        else tma_load_3d(a_dst + (uint32_t)lane * seg_bytes, &xmap, my_f + (r - 1) * rstep, chan, my_n, full);
                    }
                }
                if (ks == 0 && switch_b) {
                    // New (group, filter tile): its weights go to the free resident buffer.  Issued after the tile's
                    // first input copy, which has the longer way to come (HBM); the weights are usually in L2.
                    const uint32_t bb = c.b_res == 2 ? (switches & 1) : 0u, use = c.b_res == 2 ? (switches >> 1) : switches;
                    if (!mbar_wait_warp(smem_u32(&ctl.b_free[bb]), (use & 1) ^ 1, abort_flag, status, 600 + bb)) { ok = false; break; }
                    const uint32_t bar = smem_u32(&ctl.b_full[bb]);
                    if (lane == 0) mbar_arrive_expect_tx(bar, b_tile_bytes);
                    __syncwarp();
                    for (uint32_t blk = lane; blk < (uint32_t)vt * (uint32_t)c.chunks; blk += 32)
                        bulk_load_1d(bres_base + bb * c.bres_stride + blk * blk_bytes, wtile + (size_t)blk * blk_bytes, blk_bytes, bar);
                    cur_gn = (int)gn;
                    ++switches;
                }
                if (c.nr == 3 || c.pw) { ++ch; } else if (++r == 3) { r = 0; ++ch; }
                if (++stage == c.stages) { stage = 0; ph ^= 1; }
            }
        };
        if (!producer) {
            for (int tile = tile_first; tile < tile_end && it < kPrefetchUses; tile = tile_next(tile)) visit(tile, true, kPrefetchUses, it, stage, ph);
            run_epilogue = true;
        } else {
            for (int tile = tile_first; tile < tile_end && ok; tile = tile_next(tile)) visit(tile, false, 0u, it, stage, ph);
        }
        if (producer && !ok && lane == 0) {
            // drain: wait (bounded) for the copies of every stage that may still be in flight, so that no bulk copy
            // lands in this CTA's shared memory after it has exited; a drain that runs out too is recorded in the
            // status detail (1000 + stage, 1100 + weight buffer) beside the code of the wait that gave up first
            // (gather producer: the copies in flight are the raw buffers'; its stage barriers complete by arrivals)
            for (int i = 0; c.soft && i < c.raw_stages && i < (int)it; ++i) {
                const uint32_t j = it - 1 - i;
                if (!mbar_drain(smem_u32(&ctl.raw_full[j % c.raw_stages]), (j / c.raw_stages) & 1, abort_flag)) status->detail = 1200 + (int)(j % c.raw_stages);
            }
            for (int i = 0; !c.soft && i < c.stages && i < (int)it; ++i) {
                const uint32_t j = it - 1 - i;
                if ((int)j == c.dbg_skip && blockIdx.x == 0) continue;   // the test hook issued nothing for this fill
                if (!mbar_drain(smem_u32(&ctl.full[j % c.stages]), (j / c.stages) & 1, abort_flag)) status->detail = 1000 + (int)(j % c.stages);
            }
            for (uint32_t i = 0; i < (uint32_t)c.b_res && i < switches; ++i) {
                const uint32_t j = switches - 1 - i;
                const uint32_t bb = c.b_res == 2 ? (j & 1) : 0u;
                const uint32_t par = (c.b_res == 2 ? (j >> 1) : j) & 1;
                if (!mbar_drain(smem_u32(&ctl.b_full[bb]), par, abort_flag)) status->detail = 1100 + (int)bb;
            }
        }
    } else if (c.fuse && warp == (c.egroups == 2 ? kMmaWarp3 : kMmaWarp2)) {
        // ---------------------------------------------------------------- pointwise MMA issuer (fused block)
        // D2[128 pixels, C2] += A2[128 pixels, Kt] * W2[group][Kt, C2] for every group of the pixel tile in turn; A2 is the
        // grouped result the epilogue warps wrote to shared memory in the MN-major operand layout.
        if (lane == 0) {
            bool ok = mbar_wait(smem_u32(&ctl.w2_full), 0, abort_flag, status, 900);
            const uint32_t idesc2 = (1u << 4) | (2u << 7) | (2u << 10) | (1u << 15) | ((uint32_t)(c.C2 >> 3) << 17) | ((128u >> 4) << 24);
            const uint32_t a2_blk = (uint32_t)c.Kt * 128u;                      // one 32-pixel block of A2
            const uint64_t a2_desc0 = make_desc(0, a2_blk, 512u, 1u);
            const uint32_t b2_lbo = (uint32_t)(c.C2 >> 3) * 128u;
            const uint64_t b2_desc0 = make_desc(0, b2_lbo, 128u, 0u);
            const uint32_t a2_hi = (uint32_t)(a2_desc0 >> 32), a2_lo0 = (uint32_t)a2_desc0;
            const uint32_t b2_hi = (uint32_t)(b2_desc0 >> 32), b2_lo0 = (uint32_t)b2_desc0;
            const uint32_t w2_blk = (uint32_t)c.Kt * (uint32_t)c.C2 * 4u;
            uint32_t uses[2] = {0u, 0u}, ptiles = 0, e = 0;
            for (int tile = tile_first; tile < tile_end && ok; tile = tile_next(tile), e ^= (c.egroups == 2 ? 1u : 0u)) {   // A2 buffer = epilogue group
                uint32_t gn, mt;
                tile_coords(c, (uint32_t)tile, gn, mt);
                if (!mbar_wait(smem_u32(&ctl.a2_full[e]), uses[e] & 1u, abort_flag, status, 910 + (int)e)) break;
                // the pixel tile's accumulator: two of them take alternate pixel tiles when TMEM has the room
                const uint32_t db = c.d2_bufs == 2 ? (ptiles & 1u) : 0u, du = c.d2_bufs == 2 ? (ptiles >> 1) : ptiles;
                const uint32_t d2 = tmem_base + (uint32_t)c.d2_col + db * (uint32_t)c.C2;
                if (gn == 0 && du > 0 && !mbar_wait(smem_u32(&ctl.d2_free[db]), (du - 1) & 1u, abort_flag, status, 920)) break;
                tc_fence_after();
                uint32_t al = a2_lo0 + ((smem_base + c.a2_off + e * 4u * a2_blk) >> 4);
                uint32_t bl = b2_lo0 + ((smem_base + c.w2_off + gn * w2_blk) >> 4);
                for (int k8 = 0; k8 < c.Kt / 8; ++k8, al += 64u, bl += (2u * b2_lbo) >> 4)
                    umma_tf32_split(d2, al, a2_hi, bl, b2_hi, idesc2, (gn != 0 || k8 != 0) ? 1u : 0u);
                umma_commit(smem_u32(&ctl.a2_free[e]));
                ++uses[e];
                if ((int)gn + 1 == c.n_gn) {
                    umma_commit(smem_u32(&ctl.d2_full[db]));
                    ++ptiles;
                }
            }
        }
    } else if (c.soft && warp >= (c.egroups == 1 ? kEpi2First : kMmaWarp3 + 2)) {
        // ---------------------------------------------------------------- gather producer (copy warps)
        // Planes the tiled bulk copies cannot bring as operand rows (row length not a multiple of 16 bytes: 14, 7, ...
        // wide) and small stride-2 planes.  A tile is four segments; a segment is `rps` whole OUTPUT rows laid side by
        // side in its 32 lanes (lane = row-in-segment * W_out + column), so a pixel's horizontal neighbours are the
        // neighbouring lanes and nothing is padded.  Warp 0 lands the raw input rows of the tile in the raw ring; copy
        // warp j builds segment j of every operand block of the stage from them, shared memory to shared memory, in
        // exactly the image the tensor core expects (32-pixel blocks, 128-byte row per channel, 32-byte chunks
        // XOR-swizzled by the channel):
        //   stride 1: three blocks, one per vertical tap r: A_r[lane] = x[p + (r-1)*dil, q]
        //   stride 2: six blocks, per vertical tap the even and the odd input column of the output pixel:
        //             A_rE[lane] = x[2p + r - 1, 2q],  A_rO[lane] = x[2p + r - 1, 2q + 1]
        // rows and columns outside the plane, lanes past the segment's rows and images past the batch are written as
        // zeros.  Then fence.proxy.async, one arrival per copy warp on the stage barrier, one on the raw buffer's.
        // copy warp j builds segment j & 3; in the heavy shape warps 4..7 take the second half of the stage's channels
        const int gw = warp - (c.egroups == 1 ? kEpi2First : kMmaWarp3 + 2);
        // (pair tiles: warps 4..7 build the stage's second pixel tile instead, all channels)
        const int pw = gw & 3;
        const int tp = c.pair ? (gw >> 2) : 0;                          // which tile of the pair
        const int kcount = (c.egroups == 2 && !c.pair) ? c.CK / 2 : c.CK;   // channels of the stage this warp copies
        const uint32_t kbase = c.pair ? 0u : (uint32_t)(gw >> 2) * (uint32_t)kcount;  // (a multiple of 4: the swizzle term k & 3 is unchanged)
        const bool g2 = c.soft == 2;
        // lanes take two adjacent pixels (8-byte accesses) when pixel pairs never straddle a row: the two half-warps
        // then take alternate channels
        const bool pairs = !g2 && (s.W & 1) == 0;
        const int u = pairs ? (lane & 15) : lane;
        const int kfirst = pairs ? (lane >> 4) : 0;
        const int l0 = pairs ? 2 * u : lane;                 // first output lane this thread fills
        uint32_t rr_, q_;
        c.div_w.divmod((uint32_t)l0, rr_, q_);
        const int rr = (int)rr_, q = (int)q_;
        const uint32_t unit_chunk = pairs ? (uint32_t)(u >> 2) : (uint32_t)(u >> 3);
        const uint32_t unit_in = pairs ? (uint32_t)(u & 3) * 8u : (uint32_t)(u & 7) * 4u;
        const uint32_t piece_bytes = (uint32_t)c.CK * (uint32_t)c.boxpx * 4u;
        const uint32_t part_bytes = (uint32_t)c.pieces * piece_bytes;
        const int dil = s.dilation;
        uint32_t it = 0;
        uint32_t rs = 0, ruse = 0;                           // raw ring position of the current fill and its pass over the ring
        int stage = 0;
        uint32_t ph = 0;
        bool ok = true;
        for (int tile = tile_first; tile < tile_end && ok; tile = tile_next(tile)) {
            uint32_t gn, mt;
            tile_coords(c, (uint32_t)tile, gn, mt);
            // this warp's segment: image, segment of the image, part of the raw buffer it reads
            if (c.pair) mt = 2u * mt + (uint32_t)tp;
            int n, i, pt;
            gath_segment(c, mt, pw, n, i, pt);
            int npart, fa;
            gath_part(s, c, mt, pt, npart, fa);
            const int p = i * c.rps + rr;                    // output row of this lane
            const bool lane_ok = n < s.N && i < c.SPI && rr < c.rps && p < s.H_out;
            // the raw-buffer offsets of this lane's three tap rows do not depend on the channel stage
            uint32_t tap_idx[3], tap_in[3];
            bool tap_v[3];
#pragma unroll
            for (int r = 0; r < 3; ++r) {
                const int h = g2 ? 2 * p + r - 1 : p + (r - 1) * dil;
                tap_v[r] = lane_ok && h >= 0 && h < s.H;
                tap_idx[r] = 0;
                tap_in[r] = 0;
                if (tap_v[r]) {
                    uint32_t pc, in;
                    c.div_boxpx.divmod((uint32_t)(h * s.W + (g2 ? 2 * q : q) - fa), pc, in);
                    tap_idx[r] = pc * (uint32_t)c.CK * (uint32_t)c.boxpx + in;
                    tap_in[r] = in;
                }
            }
            for (int ks = 0; ks < kstages; ++ks, ++it) {
                if (!mbar_wait_warp(smem_u32(&ctl.raw_full[rs]), ruse & 1u, abort_flag, status, 160 + (int)rs)) { ok = false; break; }
                if (it >= (uint32_t)c.stages && !mbar_wait_warp(smem_u32(&ctl.empty[stage]), ph ^ 1, abort_flag, status, 100 + stage)) { ok = false; break; }
                // Plain shared-memory pointers; a lane with nothing to read loads from the start of its part and stores zeros
                // (no divergent branches).  Per element the work is one address add, the load, a select and a store with a
                // constant offset: the swizzled destination of channel k is base[k & 3] + k * 128 bytes, and the four (two)
                // bases are computed once per block.  A copy warp is alone with this code on its scheduler, so every
                // instruction saved shortens the stage's critical path directly.
                const float* __restrict__ rawp = reinterpret_cast<const float*>(smem + c.raw_off + rs * c.raw_bytes + (uint32_t)(tp * c.IPT + pt) * part_bytes);
                float* __restrict__ stg = reinterpret_cast<float*>(smem + (uint32_t)c.b_res * c.bres_stride + (uint32_t)stage * c.stage_bytes + (uint32_t)tp * a_bytes);
                const uint32_t seg_f = seg_bytes >> 2;       // floats per 32-pixel block
                const uint32_t bpx = (uint32_t)c.boxpx;
                // (a pointwise layer has the centre tap only: one block, and with stride 2 only the even columns)
                if (!g2) {
#pragma unroll
                    for (int r = 0; r < 3; ++r) {
                        if (c.pw && r != 1) continue;
                        const bool v = tap_v[r];
                        const uint32_t idx = tap_idx[r];
                        float* __restrict__ dp = stg + (uint32_t)((c.pw ? 0 : r) * 4 + pw) * seg_f + (unit_in >> 2);
                        if (pairs) {
                            // half-warp hw takes channels k = 2 j + hw: k & 3 is hw or hw + 2
                            const float* __restrict__ sp = rawp + idx + ((uint32_t)kfirst + kbase) * bpx;
                            float* __restrict__ d0 = dp + ((uint32_t)kfirst + kbase) * 32u + ((unit_chunk ^ (uint32_t)kfirst) << 3);
                            float* __restrict__ d1 = dp + ((uint32_t)kfirst + kbase) * 32u + ((unit_chunk ^ (uint32_t)(kfirst + 2)) << 3);
                            const uint32_t bp2 = 2u * bpx;
#pragma unroll
                            for (int j0 = 0; j0 < kcount / 2; j0 += 8) {
                                float2 t[8];
#pragma unroll
                                for (int j = 0; j < 8; ++j)
                                    if (j0 + j < kcount / 2) t[j] = *reinterpret_cast<const float2*>(sp + (uint32_t)(j0 + j) * bp2);
#pragma unroll
                                for (int j = 0; j < 8; ++j)
                                    if (j0 + j < kcount / 2)
                                        *reinterpret_cast<float2*>((((j0 + j) & 1) ? d1 : d0) + (j0 + j) * 64) = v ? t[j] : make_float2(0.f, 0.f);
                            }
                        } else {
                            const float* __restrict__ sp = rawp + idx + kbase * bpx;
                            float* __restrict__ d[4];
#pragma unroll
                            for (int m = 0; m < 4; ++m) d[m] = dp + kbase * 32u + ((unit_chunk ^ (uint32_t)m) << 3);
#pragma unroll
                            for (int k0 = 0; k0 < kcount; k0 += 8) {
                                float t[8];
#pragma unroll
                                for (int j = 0; j < 8; ++j) t[j] = sp[(uint32_t)(k0 + j) * bpx];
#pragma unroll
                                for (int j = 0; j < 8; ++j) d[(k0 + j) & 3][(k0 + j) * 32] = v ? t[j] : 0.f;
                            }
                        }
                    }
                } else {
                    const bool w_even = (s.W & 1) == 0;      // the (even, odd) column pair of an output pixel is 8-byte aligned
                    const bool odd_ok = 2 * q + 1 < s.W;
#pragma unroll
                    for (int r = 0; r < 3; ++r) {
                        if (c.pw && r != 1) continue;
                        const bool v = tap_v[r];
                        const uint32_t idx = tap_idx[r], in_piece = tap_in[r];
                        const float* __restrict__ sp = rawp + idx + kbase * bpx;
                        float* __restrict__ dE = stg + (uint32_t)((c.pw ? 0 : r) * 8 + pw) * seg_f + (unit_in >> 2);
                        float* __restrict__ d[4];
#pragma unroll
                        for (int m = 0; m < 4; ++m) d[m] = dE + kbase * 32u + ((unit_chunk ^ (uint32_t)m) << 3);
                        const uint32_t oblk = 4u * seg_f;    // the odd-column block sits four segments behind the even one
                        // the odd column sits one float behind the even one -- or, on odd widths, where rows start at odd flat
                        // pixels, at the head of the next piece of the raw part when the even column is a piece's last pixel
                        const bool has_odd = v && odd_ok;
                        const uint32_t oo = !has_odd ? 0u : ((!w_even && in_piece + 1u == bpx) ? (uint32_t)c.CK * bpx - in_piece : 1u);
#pragma unroll
                        for (int k0 = 0; k0 < kcount; k0 += 8) {
                            float e[8], o[8];
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                const float* a = sp + (uint32_t)(k0 + j) * bpx;
                                if (w_even) {
                                    const float2 t = *reinterpret_cast<const float2*>(a);
                                    e[j] = t.x;
                                    o[j] = t.y;
                                } else {
                                    e[j] = a[0];
                                    o[j] = a[oo];
                                }
                            }
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                float* de = d[(k0 + j) & 3] + (k0 + j) * 32;
                                de[0] = v ? e[j] : 0.f;
                                if (!c.pw) de[oblk] = has_odd ? o[j] : 0.f;
                            }
                        }
                    }
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(smem_u32(&ctl.full[stage]));
                    mbar_arrive(smem_u32(&ctl.raw_empty[rs]));
                }
                if (++stage == c.stages) { stage = 0; ph ^= 1; }
                if (++rs == (uint32_t)c.raw_stages) { rs = 0; ++ruse; }
            }
        }
    } else if (warp == 1 || warp == kMmaWarp2 || warp >= kMmaWarp3) {
        // ---------------------------------------------------------------- MMA issuers
        // Two warps issue alternate tiles (each owns one TMEM buffer), so the barrier waits and descriptor
        // set-up of one tile hide behind the other warp's MMAs.  Both walk every tile to keep the stage ring
        // and the weight-buffer switches in step.
        const uint32_t mslot = warp == 1 ? 0u : (warp == kMmaWarp2 ? 1u : 2u + (uint32_t)(warp - kMmaWarp3));
        if (lane == 0 && mslot < (uint32_t)c.issuers) {
            const uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | (1u << 15) | ((uint32_t)(c.Np >> 3) << 17) |
                                   ((128u >> 4) << 24);
            // stride-2 gather stages: the even-column block meets the centre tap (N = Kt), the odd-column block the left and
            // right taps (N = 2 Kt); the packed columns are ordered (centre, left, right) for this
            const uint32_t idesc_e = (idesc & ~(0x3Fu << 17)) | ((uint32_t)(c.Kt >> 3) << 17);
            const uint32_t idesc_o = (idesc & ~(0x3Fu << 17)) | ((uint32_t)(c.Kt >> 2) << 17);
            const uint32_t b_lbo = (uint32_t)(c.Np >> 3) * 128u;   // next 4-channel core matrix along K
            const uint32_t b_kstep = 2u * b_lbo;                   // 8 channels
            // descriptors differ only in the start-address field of the low word
            const uint64_t a_desc0 = make_desc(0, (uint32_t)c.lbo_segs * seg_bytes, 512u, 1u);   // 32-pixel blocks of M: every segment, or every other one
            const uint64_t b_desc0 = make_desc(0, b_lbo, 128u, 0u);
            const uint32_t a_hi = (uint32_t)(a_desc0 >> 32), a_lo0 = (uint32_t)a_desc0;   // low word: address (16-byte units) | LBO << 16
            const uint32_t b_hi = (uint32_t)(b_desc0 >> 32), b_lo0 = (uint32_t)b_desc0;
            const int k8n = c.CK / 8;
            // 16-byte-unit offsets that do not depend on the tile: the A view of a tap inside a halo stage, the weight
            // block of a tap, one 8-channel step of B.  Shared-memory addresses stay below 2^18, so adding them to a
            // low word never carries into the LBO field.
            const uint32_t view16 = (uint32_t)(c.nr == 3 ? c.wseg : 0) * (seg_bytes >> 4);
            const uint32_t blk16 = blk_bytes >> 4;
            const uint32_t bk16 = b_kstep >> 4;
            const uint32_t b_in_stage16 = a_all >> 4;
            const uint32_t a_pair16 = a_bytes >> 4;   // pair tiles: the second tile's input inside the stage
            uint32_t tcount = 0, switches = 0;
            int stage = 0;
            uint32_t ph = 0;
            uint32_t buf = 0, bph = 0;      // accumulator ring position of the current tile and its pass parity
            uint32_t turn = 0;              // which issuing warp's turn the current tile is
            int cur_gn = -1;
            uint32_t bres_addr = 0;
            bool ok = true;
            for (int tile = tile_first; tile < tile_end && ok;
                 tile = tile_next(tile), ++tcount, buf = (buf + 1 == (uint32_t)c.nacc ? 0u : buf + 1), bph ^= (buf == 0 ? 1u : 0u),
                     turn = (turn + 1 == (uint32_t)c.issuers ? 0u : turn + 1)) {
                uint32_t gn, mt;
                tile_coords(c, (uint32_t)tile, gn, mt);
                const bool mine = turn == mslot;
                if (c.ball) {
                    // bank gn lives in buffer gn for the whole launch; the first use waits for its one fill
                    if (switches < 2u && (int)gn != cur_gn) {
                        if (!mbar_wait(smem_u32(&ctl.b_full[gn]), 0, abort_flag, status, 710)) break;
                        ++switches;
                    }
                    bres_addr = bres_base + gn * c.bres_stride;
                    cur_gn = (int)gn;
                } else if (c.b_res && (int)gn != cur_gn) {
                    // the previous weight buffer is free once every MMA this warp issued so far has completed
                    // (the barrier counts both issuing warps)
                    const uint32_t bb = c.b_res == 2 ? (switches & 1) : 0u, use = c.b_res == 2 ? (switches >> 1) : switches;
                    if (switches > 0) umma_commit(smem_u32(&ctl.b_free[c.b_res == 2 ? ((switches - 1) & 1) : 0u]));
                    // Both warps observe every fill of a weight buffer, in order, even when the tiles that
                    // use it are the other warp's: a parity wait is only meaningful one phase at a time.
                    if (!mbar_wait(smem_u32(&ctl.b_full[bb]), use & 1, abort_flag, status, 700)) break;
                    bres_addr = bres_base + bb * c.bres_stride;
                    cur_gn = (int)gn;
                    ++switches;
                }
                if (!mine) {
                    // The other warp's tile: observe its stages' phases in order (no MMAs) so that this warp's own parity
                    // waits never alias a phase it has not seen -- and tell the producer so: a stage is refilled only when
                    // its consumer's MMAs have completed AND every other issuing warp has seen the fill.  Without that
                    // arrival a warp held up on one stage (its copy arriving late, say from DRAM while the others hit L2)
                    // could miss two flips of another stage and wait for ever on a phase that has long passed.
                    for (int ks = 0; ks < kstages && ok; ++ks) {
                        if (!mbar_wait(smem_u32(&ctl.full[stage]), ph, abort_flag, status, 800 + stage)) ok = false;
                        else mbar_arrive(smem_u32(&ctl.empty[stage]));
                        if (++stage == c.stages) { stage = 0; ph ^= 1; }
                    }
                    continue;
                }
                if (!mbar_wait(smem_u32(&ctl.tmem_empty[buf]), bph ^ 1, abort_flag, status, 200 + buf)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * (uint32_t)c.Np;
                uint32_t acc = 0;
                for (int ks = 0; ks < kstages; ++ks) {
                    // (the descriptors of the stage are worked out before the wait: what follows the arrival of the data is the MMAs)
                    const uint32_t a16 = (stage_base + (uint32_t)stage * c.stage_bytes) >> 4;
                    // weights of this stage: (chunk, tap) blocks of the resident bank, or the blocks staged behind A
                    const uint32_t b16 = c.b_res ? (bres_addr >> 4) + (uint32_t)(c.nr == 3 ? ks * 3 : ks) * blk16 : a16 + b_in_stage16;
                    uint32_t alo = a_lo0 + a16, blo = b_lo0 + b16;
                    if (!mbar_wait(smem_u32(&ctl.full[stage]), ph, abort_flag, status, 300 + stage)) { ok = false; break; }
                    tc_fence_after();
                    // tap r of a halo stage is the view that starts r rows (wseg segments per row) further in
                    for (int rr = 0; rr < c.nr; ++rr, alo += view16, blo += blk16) {
                        uint32_t al = alo, bl = blo;
#pragma unroll 4
                        for (int k8 = 0; k8 < k8n; ++k8, al += 64u, bl += bk16) {
                            if (c.soft == 2 && !c.pw) {
                                umma_tf32_split(d_tmem, al, a_hi, bl, b_hi, idesc_e, acc);
                                umma_tf32_split(d_tmem + (uint32_t)c.Kt, al + 4u * (seg_bytes >> 4), a_hi, bl + (uint32_t)c.Kt, b_hi, idesc_o, acc);
                                if (c.pair) {                  // same weights, second tile
                                    umma_tf32_split(d_tmem + (uint32_t)c.Np, al + a_pair16, a_hi, bl, b_hi, idesc_e, acc);
                                    umma_tf32_split(d_tmem + (uint32_t)(c.Np + c.Kt), al + a_pair16 + 4u * (seg_bytes >> 4), a_hi, bl + (uint32_t)c.Kt, b_hi, idesc_o, acc);
                                }
                            } else {
                                umma_tf32_split(d_tmem, al, a_hi, bl, b_hi, idesc, acc);
                                if (c.pair) umma_tf32_split(d_tmem + (uint32_t)c.Np, al + a_pair16, a_hi, bl, b_hi, idesc, acc);   // same weights, second tile
                            }
                            acc = 1;
                        }
                    }
                    umma_commit(smem_u32(&ctl.empty[stage]));
                    if (++stage == c.stages) { stage = 0; ph ^= 1; }
                }
                if (ok) umma_commit(smem_u32(&ctl.tmem_full[buf]));
            }
        }
    } else {
        run_epilogue = true;
    }
    if (run_epilogue) {
        // ---------------------------------------------------------------- epilogue warps
        // Two groups of eight warps take alternate tiles, so one tile's TMEM reads, shuffles and stores overlap
        // the next tile's.  With an even number of accumulators a buffer always belongs to the same group.
        asm volatile("griddepcontrol.wait;" ::: "memory");   // y may still be read (or written) by the previous kernel
        const int wq = warp & 3;                       // TMEM lane quarter this warp may read
        const uint32_t egroup = warp >= kEpi2First ? 1u : 0u;
        const int half = ((warp - (egroup ? kEpi2First : 2)) >> 2);   // which half of the tile's filters this warp stores
        const int l = wq * 32 + lane;                  // pixel lane inside the tile
        const int Kt = c.Kt;
        const int kh = (Kt / 2 + 7) & ~7;              // filters of the first half (multiple of 8)
        const int kbeg = half == 0 ? 0 : kh;
        const int kend = half == 0 ? kh : Kt;
        uint32_t buf = 0, bph = 0, tpar = 0;
        uint32_t a2_uses = 0, ptiles = 0, d2_seen = 0;   // fused block: uses of this group's A2 buffer, pixel tiles finished,
                                                         // phases of d2_full this group has observed
        // Fused block, second epilogue: the pointwise result of pixel tile p (accumulator p % d2_bufs) goes to y2.  With two
        // accumulators it is deferred until the group has handed its next grouped result to the tensor core, so the
        // group never idles through the pointwise MMAs' latency; pend_* remember the deferred tile.
        bool pend = false, pend_valid = false;
        uint32_t pend_p = 0;
        float* pend_y2 = nullptr;
        const int c2h = ((c.C2 / 2) + 7) & ~7;
        const int c2beg = half == 0 ? 0 : c2h, c2end = half == 0 ? c2h : c.C2;
        auto epilogue2 = [&](uint32_t db, uint32_t parity, float* y2, bool v) -> bool {
            if (!mbar_wait_warp(smem_u32(&ctl.d2_full[db]), parity, abort_flag, status, 940)) return false;
            tc_fence_after();
            const uint32_t d2 = tmem_base + (uint32_t)c.d2_col + db * (uint32_t)c.C2 + ((uint32_t)(wq * 32) << 16);
            for (int k0 = c2beg; k0 < c2end; k0 += 8) {
                float d[8];
                tmem_ld8(d2 + (uint32_t)k0, d);
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    if (v) *y2 = d[j];
                    y2 += OHW;
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctl.d2_free[db]));
            return true;
        };
        for (int tile = tile_first; tile < tile_end;
             tile = tile_next(tile), tpar ^= 1u, buf = (buf + 1 == (uint32_t)c.nacc ? 0u : buf + 1), bph ^= (buf == 0 ? 1u : 0u)) {
            uint32_t gn, mt;
            if (c.egroups == 2 && tpar != egroup && !c.pair) {           // the other group's tile
                if (c.fuse) {
                    tile_coords(c, (uint32_t)tile, gn, mt);
                    if ((int)gn + 1 == c.n_gn) ++ptiles;
                }
                continue;
            }
            tile_coords(c, (uint32_t)tile, gn, mt);
            if (c.pair) mt = 2u * mt + egroup;               // pair tiles: group e drains the pair's tile e (accumulator e of the buffer)
            uint32_t n, i;
            int f = 0;
            bool valid;
            bool g_left = false, g_right = false;
            int g_fo = 0;
            if (c.soft) {
                // gather tilings: quarter wq is one segment, lane = row-in-segment * W_out + column
                int gn_, gi_, gp_;
                gath_segment(c, mt, wq, gn_, gi_, gp_);
                n = (uint32_t)gn_;
                uint32_t rr, q;
                c.div_w.divmod((uint32_t)lane, rr, q);
                const int p = gi_ * c.rps + (int)rr;
                valid = gn_ < s.N && gi_ < c.SPI && (int)rr < c.rps && p < s.H_out;
                g_fo = p * s.W_out + (int)q;
                const int dl = c.soft == 2 ? 1 : s.dilation;
                g_left = (int)q >= dl;
                g_right = c.soft == 2 ? false : (int)q + dl < s.W_out;
            } else if (c.rowbox) {
                // quarter wq is segment h = wq % SR of row p0 + wq / SR; the last segment of a two-segment row is
                // shifted left to end at column W, and each column is stored by the segment that holds both of its
                // horizontal neighbours
                // (stride 2: quarter wq is output row 4*pb + wq of the tile's one segment, i.e. input row twice that)
                c.div_spi.divmod(mt, n, i);
                int h, row;
                if (c.s2h) {
                    const int pb = c.SR == 2 ? (int)(i >> 1) : (int)i;
                    h = c.SR == 2 ? (int)(i & 1u) : 0;
                    row = 2 * (4 * pb + wq);
                } else {
                    h = c.SR == 2 ? (wq & 1) : 0;
                    row = (int)i * c.R + (c.SR == 2 ? (wq >> 1) : wq);
                }
                const int col = (h ? s.W - 32 : 0) + lane;
                valid = row < s.H && col < s.W && (c.SR == 1 || (h == 0 ? col <= 30 : col >= 31));
                if (c.pair) valid = valid && (int)n < s.N;   // an odd tile count leaves the last pair's second tile empty
                f = row * s.W + (col < s.W ? col : s.W - 1);
            } else if (c.seg_mode) {
                c.div_spi.divmod(mt * 4u + (uint32_t)wq, n, i);
                f = (int)i * c.seg_fstep + lane;
                valid = (int)n < s.N;
            } else {
                c.div_spi.divmod(mt, n, i);
                f = (int)i * c.R * s.W + l;
                valid = (l < c.R * s.W) && (f < HW);
            }
            uint32_t prow = 0, q = 0;
            if (!c.soft) c.div_w.divmod((uint32_t)f, prow, q);
            const int dil = c.soft == 2 ? 1 : s.dilation;   // horizontal taps sit dil columns away (dil > 1: segment and gather tilings only)
            const bool use_left = c.soft ? g_left : (int)q >= dil;
            const bool use_right = c.soft ? g_right : (int)q + dil < s.W;
            // s.H x s.W is the (possibly padded) plane the kernel computes on; only the first Hv x Wv pixels exist in y
            if (!c.soft) valid = valid && (int)prow < c.Hv && (int)q < c.Wv;
            int fo = c.soft ? g_fo : (int)prow * s.W_out + (int)q;       // position in the output plane
            if (!c.soft && (c.sub_h | c.sub_w)) {        // a stride of 2 keeps the even rows (columns) of the stride-1 result
                valid = valid && ((prow & (uint32_t)c.sub_h) == 0) && ((q & (uint32_t)c.sub_w) == 0);
                fo = (int)(prow >> c.sub_h) * s.W_out + (int)(q >> c.sub_w);
            }
            const bool add_up = use_left && lane >= dil;
            const bool add_dn = use_right && lane + dil < 32;
            // (addresses first, then the wait for the accumulator: what follows the MMAs' completion is the reads and the stores)
            const uint32_t t0 = tmem_base + (c.pair ? egroup : buf) * (uint32_t)c.Np + ((uint32_t)(wq * 32) << 16);
            // output channel of filter 0 of this tile: gn*Kt == g*Kg_eff + nt*Kt
            float* yk = y + ((size_t)n * s.C_out + (size_t)gn * Kt + (size_t)kbeg) * OHW + fo;
            if (!mbar_wait_warp(smem_u32(&ctl.tmem_full[buf]), bph, abort_flag, status, 400 + buf)) break;
            tc_fence_after();
            // fused block: this lane's slot in the A2 operand (32-pixel block wq, 128-byte row per channel, 32-byte
            // chunks swizzled by the channel index), once the pointwise MMAs of the buffer's previous use are done
            uint8_t* a2p = smem + c.a2_off + (size_t)egroup * 4u * (size_t)Kt * 128u + (size_t)wq * (size_t)Kt * 128u + (size_t)(lane & 7) * 4u;
            if (c.fuse && a2_uses > 0 && !mbar_wait_warp(smem_u32(&ctl.a2_free[egroup]), (a2_uses - 1) & 1u, abort_flag, status, 930)) break;
            if (c.need_xchg) {
                // Rows may straddle a warp boundary: publish this warp's edge lanes (lane 31's left-tap
                // and lane 0's right-tap accumulators) so the neighbouring quarter can add them, then wait
                // (bounded mbarrier wait, never a named barrier) until all epilogue warps have published.
                for (int k0 = kbeg; k0 < kend; k0 += 8) {
                    float d0[8], d2[8];
                    tmem_ld8(t0 + (uint32_t)k0, d0);
                    tmem_ld8(t0 + (uint32_t)(2 * Kt + k0), d2);
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        if (lane == 31) xchg[buf][wq][0][k0 + j] = d0[j];
                        if (lane == 0) xchg[buf][wq][1][k0 + j] = d2[j];
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&ctl.xchg_bar[buf]));
                if (!mbar_wait_warp(smem_u32(&ctl.xchg_bar[buf]), bph, abort_flag, status, 500 + buf)) break;
            }
            const bool edge_up = c.need_xchg && lane == 0 && wq > 0 && use_left;     // left neighbour is in the previous quarter
            const bool edge_dn = c.need_xchg && lane == 31 && wq < 3 && use_right;   // right neighbour is in the next quarter
            if (c.pair) {
                // Pair tiles have one accumulator buffer, so the next pair's MMAs wait for this epilogue: read and combine
                // the warp's 32 filters into registers first, hand the buffer back, and only then store.
                float v[32];
#pragma unroll
                for (int kk = 0; kk < 32; kk += 8) {
                    float d0[8], d1[8], d2[8];
                    tmem_ld8(t0 + (uint32_t)(kbeg + kk), d0);
                    tmem_ld8(t0 + (uint32_t)(Kt + kbeg + kk), d1);
                    tmem_ld8(t0 + (uint32_t)(2 * Kt + kbeg + kk), d2);
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        float t;
                        if (c.soft == 2) {                     // columns (centre, left, right): d0 = centre, d1 = left, d2 = right (own lane)
                            const float up = __shfl_up_sync(0xffffffffu, d1[j], 1u);
                            t = d0[j] + d2[j];
                            if (add_up) t += up;
                        } else {
                            t = d1[j];
                            const float up = __shfl_up_sync(0xffffffffu, d0[j], 1u);
                            const float dn = __shfl_down_sync(0xffffffffu, d2[j], 1u);
                            if (add_up) t += up;
                            if (add_dn) t += dn;
                        }
                        v[kk + j] = t;
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&ctl.tmem_empty[buf]));
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    if (valid) *yk = v[j];
                    yk += OHW;
                }
                continue;
            }
            for (int k0 = kbeg; k0 < kend; k0 += 8) {
                float d0[8], d1[8], d2[8];
                if (c.pw) {                                // one accumulator per filter, nothing to combine
                    tmem_ld8(t0 + (uint32_t)k0, d1);
                } else if (c.soft == 2) {                  // columns (centre, left, right): the right tap already sits in its own lane (c.pw is handled above)
                    tmem_ld8(t0 + (uint32_t)k0, d1);
                    tmem_ld8(t0 + (uint32_t)(Kt + k0), d0);
                    tmem_ld8(t0 + (uint32_t)(2 * Kt + k0), d2);
                } else {
                    tmem_ld8(t0 + (uint32_t)k0, d0);
                    tmem_ld8(t0 + (uint32_t)(Kt + k0), d1);
                    tmem_ld8(t0 + (uint32_t)(2 * Kt + k0), d2);
                }
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    float v = d1[j];
                    if (c.soft == 2 && !c.pw) {
                        const float up = __shfl_up_sync(0xffffffffu, d0[j], 1u);
                        v += d2[j];
                        if (add_up) v += up;
                    } else if (!c.pw) {
                        const float up = __shfl_up_sync(0xffffffffu, d0[j], (unsigned)dil);
                        const float dn = __shfl_down_sync(0xffffffffu, d2[j], (unsigned)dil);
                        if (add_up) v += up;
                        if (add_dn) v += dn;
                    }
                    if (edge_up) v += xchg[buf][wq - 1][0][k0 + j];
                    if (edge_dn) v += xchg[buf][wq + 1][1][k0 + j];
                    if (c.fuse) {
                        const int k = k0 + j;
                        *reinterpret_cast<float*>(a2p + (size_t)k * 128u + (size_t)((((uint32_t)lane >> 3) ^ ((uint32_t)k & 3u)) << 5)) = v;
                    } else {
                        if (valid) *yk = v;
                        yk += OHW;
                    }
                }
            }
            if (c.fuse) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the tensor core reads A2 through the async proxy
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctl.tmem_empty[buf]));
            if (c.fuse) {
                if (lane == 0) mbar_arrive(smem_u32(&ctl.a2_full[egroup]));
                ++a2_uses;
                float* y2_tile = y + ((size_t)n * c.C2 + (size_t)c2beg) * OHW + fo;
                const bool last_gn = (int)gn + 1 == c.n_gn;   // the pixel tile's pointwise result is complete once the MMAs just requested are done
                if (c.d2_bufs == 2) {
                    // each accumulator's phases are seen in order by one group: group p % 2 when n_gn is odd, else the second
                    if (pend) {
                        if (!epilogue2(pend_p & 1u, (pend_p >> 1) & 1u, pend_y2, pend_valid)) break;
                        pend = false;
                    }
                    if (last_gn) {
                        pend = true;
                        pend_p = ptiles;
                        pend_y2 = y2_tile;
                        pend_valid = valid;
                        ++ptiles;
                    }
                } else if (last_gn) {
                    // one accumulator, both groups wait on the same barrier: a parity wait is only meaningful one phase at
                    // a time, so first observe, in order, the phases of the pixel tiles the other group finished
                    bool ok2 = true;
                    for (; d2_seen < ptiles && ok2; ++d2_seen)
                        ok2 = mbar_wait_warp(smem_u32(&ctl.d2_full[0]), d2_seen & 1u, abort_flag, status, 941);
                    if (!ok2 || !epilogue2(0u, d2_seen & 1u, y2_tile, valid)) break;
                    ++d2_seen;
                    ++ptiles;
                }
            }
        }
        if (c.fuse && pend && !*abort_flag) epilogue2(pend_p & 1u, (pend_p >> 1) & 1u, pend_y2, pend_valid);
    }

    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)c.tmem_cols) : "memory");
    }
}

// (the narrow-group gather families run two 480-thread CTAs per SM: at most 68 registers per thread; the wide-group ones run
// one CTA of 928 threads: at most 70)
template <int F>
__global__ void __launch_bounds__(family(F).soft >= 1 ? (family(F).egroups == 2 ? 32 * (kMmaWarp3 + 2 + 2 * kSoftWarps) : 32 * (kEpi2First + kSoftWarps)) : kThreads,
                                  family(F).soft >= 1 && family(F).egroups == 1 ? 2 : 1)
igemm_tf32_kernel(const __grid_constant__ CUtensorMap xmap, const __grid_constant__ CUtensorMap xmap4, const Shape s_in,
                  const IgemmCfg c_in, const uint32_t* __restrict__ packed, float* __restrict__ y, Status* status, uint32_t tag,
                  const float* __restrict__ x) {
    if constexpr (F == 0) {
        IgemmCfg c = c_in;
        c.pair = 0;     // pair tiles always run on their own instantiation (the host refuses anything else)
        igemm_tf32_body(xmap, xmap4, s_in, c, packed, y, status, tag, x);
    } else {
        constexpr Family fam = family(F);
        IgemmCfg c = c_in;
        Shape s = s_in;
#define GCONV_FIX(field) if constexpr (fam.field >= 0) c.field = fam.field;
        GCONV_FAMILY_FIELDS(GCONV_FIX)
#undef GCONV_FIX
        if constexpr (fam.stride >= 0) s.stride = fam.stride;
        if constexpr (fam.stride == 2) c.sub_h = c.sub_w = 1;     // (a stride-1 instantiation also runs the layers with a stride of 2 on one axis)
        s.dilation = 1;
        igemm_tf32_body(xmap, xmap4, s, c, packed, y, status, tag, x);
    }
}

// Weight pre-pack for this variant.  Output block (group, filter tile, chunk, r) is the shared-memory
// image of the K-major, unswizzled B operand of one (channel chunk, vertical tap):
// [k8][k2][n/8][n%8][4 channels], where column n = s*Kt + k holds filter k of the tile at horizontal
// tap s (columns >= 3*Kt are zero) and values are rounded to TF32 (round to nearest, ties away).
// When `merge` > 1 that many adjacent groups are presented to the kernel as one group with a
// block-diagonal filter bank: entries that would mix channels of different groups are zero.
__global__ void igemm_pack_kernel(Shape s, IgemmCfg c, const float* __restrict__ w, uint32_t* __restrict__ packed, uint32_t tag) {
    const int vt = c.pw ? 1 : 3, ht = c.pw ? 1 : 3;   // vertical and horizontal taps
    const size_t total = (size_t)c.groups * c.NT * vt * c.chunks * c.Np * c.CK;
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
        const int r = (int)(t % vt); t /= vt;
        const int ch = (int)(t % c.chunks); t /= c.chunks;
        const int nt = (int)(t % c.NT);
        const int g = (int)(t / c.NT);             // merged group
        const int ncol = nb * 8 + n8;
        const int ce = ch * c.CK + k8 * 8 + k2 * 4 + e;   // channel within the merged group
        uint32_t bits = 0;
        if (ncol < ht * c.Kt) {
            const int cb = ncol / c.Kt;
            const int ss = c.soft == 2 ? (cb == 0 ? 1 : (cb == 1 ? 0 : 2)) : cb;   // stride-2 gather: columns ordered (centre, left, right)
            const int ke = nt * c.Kt + (ncol - cb * c.Kt);  // filter within the merged group
            const int gi = ke / s.Kg;                        // which original group of the merge
            if (ce / s.Cg == gi) {
                const int ko = (g * c.merge + gi) * s.Kg + (ke - gi * s.Kg);
                // a pointwise (1x1) filter is the centre tap of a 3x3 filter whose other taps are zero
                const size_t wi = ((size_t)ko) * s.Cg + (ce - gi * s.Cg);
                const float v = c.pw ? w[wi] : (s.KH == 1 ? ((r == 1 && ss == 1) ? w[wi] : 0.f) : w[wi * 9 + r * 3 + ss]);
                asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(bits) : "f"(v));
            }
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

// Widths that are not a multiple of 4 cannot be addressed by TMA (row shifts must be 16-byte aligned), so such
// layers run on a zero-padded copy of x: rows padded to a multiple of 4 columns (and, when that width divides 32,
// the row count padded until the plane is a whole number of 32-pixel segments).  The zero columns and rows are
// exactly the convolution's right and bottom padding; outputs that fall in them are never stored.
struct IgemmGeom {
    int Hp, Wp;
    bool padded;
};
// A pointwise convolution (1x1, pad 0) runs as the 3x3, pad 1 convolution whose only non-zero tap is the centre one
// (same output size for either stride); the packing kernel writes the zeros.
// With stride 1 a pointwise layer has no use for rows at all -- every output pixel reads the input pixel at the same flat
// position -- so the plane is re-cut into rows the tilings like: 32 wide when H*W is a multiple of 128 (segment tiling,
// every lane used, whole tiles per image); a width TMA cannot address becomes the widest multiple of 4 up to 32 that
// divides H*W (14x14 becomes 7x28: no padded copy).
static Shape as_3x3(const Shape& s) {
    Shape t = s;
    // One stride per axis (the paper's S_h, S_w) with a stride of 2 on one axis only: every tiling computes the stride-1 layer
    // and the epilogue stores its even rows or columns (IgemmCfg::sub_h, sub_w), as stride 2 does on planes without row tiles.
    if (s.stride != s.stride_w) t.stride = t.stride_w = 1;
    if (s.KH == 1 && s.KW == 1) {
        t.KH = 3;
        t.KW = 3;
        t.pad = 1;
        t.dilation = 1;
        if (s.stride == 1) {
            const long long hw = (long long)s.H * s.W;
            int w = 0;
            if (s.W % 4 == 0) {
                if (hw % 128 == 0) w = 32;           // whole tiles per image: one box copy per stage
            } else {
                for (int cand = 32; cand >= 4 && w == 0; cand -= 4)
                    if (hw % cand == 0) w = cand;
            }
            if (w != 0 && hw / w < (1 << 30)) {
                t.W = t.W_out = w;
                t.H = t.H_out = (int)(hw / w);
            }
        }
    }
    return t;
}

static IgemmGeom igemm_geom(const Shape& s) {
    IgemmGeom g;
    g.Wp = (s.W + 3) & ~3;
    g.Hp = s.H;
    g.padded = g.Wp != s.W;
    if (g.padded && 32 % g.Wp == 0)
        while ((g.Hp * g.Wp) % 32 != 0) ++g.Hp;
    return g;
}

namespace {
// Zero-padded copy of x for widths TMA cannot address: every plane becomes Hp x Wp (Wp a multiple of 4), one thread
// per group of four output columns.  IDX is the index type: 32-bit whenever the padded tensor has fewer than 2^32
// column groups (the common case: the divisions are then cheap multiply-shift ones).
template <typename IDX>
__global__ void igemm_pad_kernel(const float* __restrict__ x, float* __restrict__ xp, size_t planes, int H, int W, int Hp, int Wp,
                                 FastDiv div_plane, FastDiv div_row) {
    // the convolution kernel that follows may be scheduled now: its set-up overlaps this copy, and it reads the padded
    // planes only after its own griddepcontrol.wait (this grid complete and visible)
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const size_t per_plane = (size_t)Hp * (Wp / 4);
    const size_t total = planes * per_plane;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        size_t plane;
        int h, w4;
        if constexpr (sizeof(IDX) == 4) {
            uint32_t pl, rem, hh, q;
            div_plane.divmod((uint32_t)i, pl, rem);
            div_row.divmod(rem, hh, q);
            plane = pl;
            h = (int)hh;
            w4 = (int)q * 4;
        } else {
            plane = i / per_plane;
            const int rem = (int)(i - plane * per_plane);
            h = rem / (Wp / 4);
            w4 = (rem - h * (Wp / 4)) * 4;
        }
        float v[4] = {0.f, 0.f, 0.f, 0.f};
        if (h < H) {
            const float* src = x + (plane * H + h) * (size_t)W;
            if ((W & 1) == 0) {                    // even width: rows start on 8-byte boundaries
                if (w4 < W) { const float2 a = __ldg(reinterpret_cast<const float2*>(src + w4)); v[0] = a.x; v[1] = a.y; }
                if (w4 + 2 < W) { const float2 b = __ldg(reinterpret_cast<const float2*>(src + w4 + 2)); v[2] = b.x; v[3] = b.y; }
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    if (w4 + j < W) v[j] = __ldg(src + w4 + j);
            }
        }
        *reinterpret_cast<float4*>(xp + (plane * Hp + h) * (size_t)Wp + w4) = make_float4(v[0], v[1], v[2], v[3]);
    }
}
}  // namespace

static int igemm_merge(const Shape& s) {
    int m = 1;
    // Stride 2: stop at 32 filters per merged group, so that channel-doubling transition layers (Kg = 2 Cg) keep one
    // resident 32-filter bank and the two-CTA launch shape instead of streaming 64-filter banks (measured: 64 -> 128
    // channels at 56x56, 32 groups, 35.5 -> 17.0 us).
    const int kcap = s.stride == 2 ? 32 : 64;
    while (m * 2 <= s.groups && s.groups % (m * 2) == 0 && s.Cg * m * 2 <= 32 && s.Kg * m * 2 <= kcap) m *= 2;
    return m;
}

bool igemm_supported(const Shape& s_any) {
    if (!s_any.square()) {
        // Per axis only the stride may differ: 3x3, pad 1, dilation 1, strides of 1 and 2, on planes the tiled copies address
        // (the gather producer and the padded copy build on one stride for both axes).
        if (s_any.pad_w != s_any.pad || s_any.dilation_w != s_any.dilation || s_any.dilation != 1 || s_any.pad != 1) return false;
        if (s_any.KH != 3 || s_any.KW != 3 || s_any.W % 4 != 0) return false;
        if (!((s_any.stride == 1 && s_any.stride_w == 2) || (s_any.stride == 2 && s_any.stride_w == 1))) return false;
    }
    if (s_any.KH == 1 && s_any.KW == 1 && !(s_any.pad == 0 && s_any.dilation == 1)) return false;
    const Shape s = as_3x3(s_any);
    if (!(s.KH == 3 && s.KW == 3 && (s.stride == 1 || s.stride == 2) && s.dilation >= 1 && s.pad == s.dilation)) return false;
    if (s.dilation > 1 && (s.stride != 1 || s.dilation > 16)) return false;
    const int m = igemm_merge(s);
    if ((s.Cg * m) % 8 != 0 || (s.Kg * m) % 8 != 0) return false;
    const IgemmGeom ge = igemm_geom(s);
    if (ge.Wp > 128) return false;
    if ((long long)ge.Hp * ge.Wp < 32) return false;
    if (s.C_in > 65535 * 8) return false;
    const IgemmCfg c = igemm_config(s, 148);
    // Dilation: vertical taps are whole-row shifts for any tiling, but the horizontal neighbours dil columns away must
    // lie in the same 32-pixel segment: segment tilings only (rows that divide 32 pixels).
    if (s.dilation > 1 && !(c.soft == 1 || (c.seg_mode && !c.rowbox && c.nr == 1 && !c.tapb))) return false;
    return c.smem_bytes <= (size_t)kMaxDynSmem;   // the smallest pipeline (two stages) must fit
}

size_t igemm_scratch_bytes(const Shape& s_any) {
    const Shape s = as_3x3(s_any);
    const IgemmGeom ge = igemm_geom(s);
    if (!ge.padded || igemm_config(s_any, kLayoutSMs).soft) return 0;   // the gather producer reads the real rows: no padded copy
    return sizeof(float) * (size_t)s.N * s.C_in * ge.Hp * ge.Wp;
}


// Gather producer (see the copy warps in the kernel): planes whose rows the tiled bulk copies cannot deliver as operand
// rows (width not a multiple of 4, up to 32) with stride 1, and stride-2 layers on such planes.  Narrow (merged) groups in
// the two-CTA launch shape.  Fills every field of the configuration; returns false when the shape is not taken.
static bool gather_config(IgemmCfg& out, const Shape& st, int sm_count) {
    IgemmCfg c = out;                    // committed only when the shape is taken
    const int mode = st.stride == 2 ? 2 : 1;
    if (st.KH != 3 || st.W % 4 == 0 || st.W_out > 32 || st.W_out < 1) return false;
    const int vt = c.pw ? 1 : 3;                                         // vertical taps (a pointwise layer has the centre one only)
    // Two launch shapes, as for the other producers: narrow (merged) groups run two CTAs per SM with a small resident bank;
    // wide groups (more than 32 channels) run one CTA per SM with 29 warps (eight copy warps behind the two epilogue
    // groups, two per segment), 16-channel stages and the bank resident (up to 144 KB) or streamed with the stages.
    // (groups of up to 32 channels with 64-filter tiles -- two accumulators do not fit 256 columns -- take the one-CTA shape
    // too when its instantiations allow; otherwise 32-filter tiles in the two-CTA shape, which gathers every tile twice)
    const bool heavy_ok = !c.pw && c.Cg % 16 == 0 && c.Kt == 64 && st.dilation == 1;      // (what the one-CTA instantiations fix)
    const bool heavy = c.Cg > 32 || (2 * c.Np > 256 && heavy_ok);
    if (heavy && !heavy_ok) return false;
    if (!heavy && !c.pw && 2 * c.Np > 256 && c.Kg % 32 == 0) {           // two accumulators must fit 256 columns: 32-filter tiles
        c.Kt = 32;
        c.NT = c.Kg / 32;
        c.Np = 96;
    }
    if (2 * c.Np > (heavy ? 512 : 256)) return false;
    if (mode == 2 && (st.dilation != 1 || c.Kt % 16 != 0)) return false;
    const uint32_t b_tile = (uint32_t)vt * (uint32_t)c.Cg * (uint32_t)c.Np * 4u;
    if (!heavy && b_tile > 40u * 1024u) return false;
    c.soft = mode;
    c.padded = 0;
    c.Hv = st.H;
    c.Wv = st.W;
    c.CK = c.Cg % 16 == 0 ? 16 : 8;
    if (heavy && mode == 2) c.CK = 8;            // two pixel tiles of six blocks each share a stage with the streamed weights (pair tiles, below)
    c.chunks = c.Cg / c.CK;
    const int Wo = st.W_out, Ho = st.H_out, HW = st.H * st.W;
    c.rps = 32 / Wo;
    c.SPI = (Ho + c.rps - 1) / c.rps;
    int tpi = 1;
    if (c.SPI >= 3) {
        c.IPT = 1;
        tpi = (c.SPI + 3) / 4;
        c.MT = st.N * tpi;
    } else {
        c.IPT = 4 / c.SPI;
        c.MT = (st.N + c.IPT - 1) / c.IPT;
    }
    c.MTr = c.MT;
    // raw parts: the input rows a tile needs, as flat pixels from a multiple of 4 on
    c.raw_bulk = HW % 4 != 0 ? 1 : 0;
    int px;
    if (c.raw_bulk) {
        c.raw_whole = 1;
        c.pieces = 1;
        c.boxpx = HW;
        px = HW;
    } else {
        const int rows = st.stride * (4 * c.rps - 1) + 2 * st.dilation + 1;
        px = rows * st.W + 3;
        c.raw_whole = (c.IPT > 1 || px >= HW) ? 1 : 0;
        if (c.raw_whole) px = HW;
        c.pieces = (px + 255) / 256;
        c.boxpx = (((px + c.pieces - 1) / c.pieces) + 3) & ~3;
    }
    if (c.IPT * c.pieces > 32) return false;
    c.div_boxpx = make_fastdiv((uint32_t)c.boxpx);
    c.raw_bytes = (uint32_t)c.IPT * (uint32_t)c.pieces * (uint32_t)c.CK * (uint32_t)c.boxpx * 4u;
    c.raw_bytes = (c.raw_bytes + 127u) & ~127u;
    c.seg_mode = 0;
    c.seg_fstep = 32;
    c.R = c.RB = 0;
    c.need_xchg = 0;
    c.rowbox = c.SR = 0;
    c.s2h = 0;
    c.lbo_segs = 1;
    c.nr = vt;
    c.wseg = c.pw ? 0 : (mode == 1 ? 4 : 8);
    c.nseg = c.pw ? 4 : (mode == 1 ? 12 : 24);
    c.tapb = 0;
    c.fast4 = 0;
    c.pair = 0;
    c.nacc = 2;
    c.issuers = 2;
    c.egroups = heavy ? 2 : 1;
    c.threads = heavy ? 32 * (kMmaWarp3 + 2 + 2 * kSoftWarps) : 32 * (kEpi2First + kSoftWarps);
    c.tmem_cols = heavy ? 512 : 256;
    c.div_spi = make_fastdiv((uint32_t)tpi);
    c.div_w = make_fastdiv((uint32_t)Wo);
    c.div_nt = make_fastdiv((uint32_t)c.NT);
    c.bres_stride = (b_tile + 1023u) & ~1023u;
    const uint32_t a_stage = ((uint32_t)c.nseg * (uint32_t)c.CK * 128u + 1023u) & ~1023u;
    // two CTAs per SM: (228 KB - 2 x 2 KB of static and reserved shared memory) / 2, minus the alignment slack; one CTA: 226 KB
    const uint32_t total = heavy ? (uint32_t)kMaxDynSmem - 1024u : 112u * 1024u - 1024u;
    // the bank stays resident when it leaves room for two stages and two raw buffers, and (a large bank) when a CTA reuses
    // it over at least two pixel tiles; otherwise its blocks stream with the stages
    c.b_res = 1;
    if (heavy && (b_tile > 144u * 1024u || c.bres_stride + 2u * a_stage + 2u * c.raw_bytes > total || c.MT < 2 * sm_count)) c.b_res = 0;
    c.nt_fast = (!c.b_res && c.NT > 1) ? 1 : 0;
    // Pair tiles: streamed weight blocks cross L2 -> shared memory once per pixel tile, and on wide groups that traffic, not
    // the tensor core, is the bound.  A stage then holds the operand blocks of TWO pixel tiles and one set of weight blocks;
    // every weight block feeds two MMAs (two accumulators side by side, one buffer), the eight copy warps build one tile each
    // per four, and the two epilogue groups drain the two accumulators at the same time.
    if (heavy && mode == 2) c.b_res = 0;         // (its stages leave no room for a resident bank)
    if (heavy && !c.b_res && c.MT >= 2 && 2u * a_stage + (uint32_t)c.nr * (uint32_t)c.Np * (uint32_t)c.CK * 4u <= 100u * 1024u) {
        c.pair = 1;
        c.MT = (c.MTr + 1) / 2;
        c.nacc = 1;
        c.issuers = 1;
        c.raw_bytes *= 2u;
    }
    c.num_tiles = c.groups * c.NT * c.MT;
    c.div_mt = make_fastdiv((uint32_t)c.MT);
    c.stage_bytes = ((c.pair ? 2u : 1u) * a_stage + (c.b_res ? 0u : (uint32_t)c.nr * (uint32_t)c.Np * (uint32_t)c.CK * 4u) + 1023u) & ~1023u;
    const uint32_t bank = c.b_res ? c.bres_stride : 0u;
    // the bank, then stages and raw buffers in turn (at most four and four) while they fit; a single stage and a single raw
    // buffer as the last resort
    if (bank + c.stage_bytes + c.raw_bytes > total) return false;
    c.stages = 1;
    c.raw_stages = 1;
    const int max_ring = heavy ? 4 : 3;
    for (;;) {
        const uint32_t used = bank + (uint32_t)c.stages * c.stage_bytes + (uint32_t)c.raw_stages * c.raw_bytes;
        if (c.raw_stages <= c.stages && c.raw_stages < max_ring && used + c.raw_bytes <= total) { ++c.raw_stages; continue; }
        if (c.stages < max_ring && used + c.stage_bytes <= total) { ++c.stages; continue; }
        break;
    }
    if (heavy && (c.stages < 2 || (mode == 2 && !c.pair))) return false;
    c.raw_off = bank + (uint32_t)c.stages * c.stage_bytes;
    c.xchg_off = c.raw_off + (uint32_t)c.raw_stages * c.raw_bytes;
    c.smem_bytes = (size_t)c.xchg_off + 1024;
    const int ctas = heavy ? sm_count : 2 * sm_count;
    c.grid = c.num_tiles < ctas ? c.num_tiles : ctas;
    c.cps = 0;
    c.fuse = 0;
    c.ball = 0;
    c.C2 = 0;
    c.n_gn = c.groups * c.NT;
    c.div_ngn = make_fastdiv((uint32_t)c.n_gn);
    c.d2_col = c.nacc * c.Np;
    c.d2_bufs = 1;
    c.w2_off = c.a2_off = 0;
    c.w2_goff = 0;
    if (c.b_res && c.n_gn > 1 && c.grid >= c.n_gn) {
        c.cps = c.grid / c.n_gn;                     // CTAs per (group, filter tile): no CTA ever switches weights
        if (c.cps > c.MT) c.cps = c.MT;
        c.grid = c.cps * c.n_gn;
    }
    out = c;
    return true;
}

static IgemmCfg igemm_config_c2(const Shape& s_any, int sm_count, int C2) {
    const Shape s_true = as_3x3(s_any);
    IgemmCfg c;
    c.wait_us = kDefaultWaitUs;
    c.dbg_skip = -1;
    // Pointwise: one vertical tap (a third of the stages and MMAs), one accumulator per filter (N = Kt), filter tiles of
    // up to 128.  Stride 2 computes every pixel and stores the even ones (no stride-2 row tiles: those are built around
    // nine staged rows).
    c.sub_h = s_any.stride == 2 ? 1 : 0;
    c.sub_w = s_any.stride_w == 2 ? 1 : 0;
    c.pw = (s_any.KH == 1 && s_any.KW == 1 && C2 == 0) ? 1 : 0;
    const int vt = c.pw ? 1 : 3;
    const bool fuse = C2 > 0;          // fused grouped + pointwise block: heavy shape, streamed or resident grouped weights
    const IgemmGeom ge = igemm_geom(s_true);
    Shape s = s_true;          // the plane the kernel computes on
    s.H = ge.Hp;
    s.W = ge.Wp;
    c.Hv = s_true.H;
    c.Wv = s_true.W;
    c.padded = ge.padded ? 1 : 0;
    c.merge = igemm_merge(s);
    c.groups = s.groups / c.merge;
    c.Cg = s.Cg * c.merge;
    c.Kg = s.Kg * c.merge;
    c.CK = (c.Cg % 32 == 0) ? 32 : (c.Cg % 16 == 0 ? 16 : 8);
    c.chunks = c.Cg / c.CK;
    const int kt_max = c.pw ? 128 : 64;
    int kt = c.Kg <= kt_max ? c.Kg : kt_max;
    while (c.Kg % kt != 0 || kt % 8 != 0) kt -= 8;   // largest multiple of 8 dividing Kg, at most 64 (pointwise: 128)
    if (c.pw) {
        // small planes: narrower filter tiles until there is a tile per SM (each re-reads its pixels from L2)
        const long long px_tiles = ((long long)s.N * s.H * s.W + 127) / 128;
        while (kt >= 64 && kt % 16 == 0 && (long long)c.groups * (c.Kg / kt) * px_tiles < (long long)kLayoutSMs) kt /= 2;
    }
    c.Kt = kt;
    c.NT = c.Kg / kt;
    c.Np = (vt * kt + 15) & ~15;
    c.soft = 0;
    c.rps = c.IPT = c.boxpx = c.pieces = c.raw_whole = c.raw_bulk = c.raw_stages = 0;
    c.raw_off = c.raw_bytes = 0;
    c.div_boxpx = make_fastdiv(1);
    if (!fuse && gather_config(c, s_true, sm_count)) return c;
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
    // Row boxes: for widths that do not divide 32 a tile can instead be RT whole rows of SR 32-pixel segments each
    // (the second segment of a row shifted left to end at column W).  Every vertical tap is then a whole number of
    // segments away, so one staged block (tile + a row above and below, one 5-D TMA box) serves all three taps, and
    // each segment contains the horizontal neighbours of the columns it stores (no exchange between warps).  Used
    // when it wastes at most a quarter more lanes than the flat tiling.
    c.rowbox = 0;
    c.SR = 0;
    if (!c.seg_mode && s.W <= 62) {
        const int sr = s.W <= 32 ? 1 : 2;
        const double util_box = (double)s.W / (32.0 * sr), util_flat = (double)((128 / s.W) * s.W) / 128.0;
        if (util_box >= 0.8 * util_flat) {
            c.rowbox = 1;
            c.SR = sr;
            c.R = 4 / sr;                                // rows per tile
            c.RB = (s.H + c.R - 1) / c.R;
            c.MT = s.N * c.RB;
            c.need_xchg = 0;
        }
    }
    // Stride 2 on widths 17..62: a tile is four output rows of one 32-column segment.  Its stage holds the nine input
    // rows 2p-1 .. 2p+7 of that segment; the rows a vertical tap needs are every other one, so tap r is the view that
    // starts at staged row r with its 32-pixel blocks two rows apart.  Odd input rows are never multiplied or stored
    // (the odd columns still are: TMA cannot skip elements of the innermost dimension).
    c.s2h = 0;
    c.lbo_segs = 1;
    if (s.stride == 2 && s.W > 8 && s.W <= 62 && !c.pw) {
        c.s2h = 1;
        c.lbo_segs = 2;
        c.seg_mode = 0;
        c.seg_fstep = 32;
        c.SPI = 0;
        c.rowbox = 1;
        c.SR = s.W <= 32 ? 1 : 2;
        c.R = 4;
        c.RB = ((s.H_out + 3) / 4) * c.SR;               // tiles per image
        c.MT = s.N * c.RB;
        c.need_xchg = 0;
    }
    // Row halo: when a row is a whole number of 32-pixel segments the three vertical taps are views of
    // one staged block (tile + one row above and below), so the input crosses L2 -> shared memory once.
    c.nr = 1;
    c.nseg = 4;
    c.wseg = 0;
    if (c.rowbox && c.s2h) {
        c.nr = 3;
        c.wseg = 1;
        c.nseg = 9;
    } else if (c.rowbox && c.pw) {
        c.nr = 1;                                        // the tile's own rows, no halo
    } else if (c.rowbox) {
        c.nr = 3;
        c.wseg = c.SR;
        c.nseg = 4 + 2 * c.SR;
    } else if (!c.pw && s.stride == 1 && s.dilation == 1 && s.W % 32 == 0 && s.W <= 64 && (c.seg_mode ? (c.SPI % 4 == 0) : true)) {
        c.nr = 3;
        c.wseg = s.W / 32;
        c.nseg = 4 + 2 * c.wseg;
    }
    // Tap blocks: small planes whose rows are shorter than a segment (16x16, 8x8) cannot take the taps as views of one
    // halo block, but narrow groups can still stage all three taps of a tile in ONE stage -- three blocks of four
    // segments, each loaded with its own row shift -- so a tile costs one barrier round trip instead of three.  Only
    // where a tile straddles images anyway (8x8): 16x16 planes keep their one-box-per-tap copies, which are faster.
    c.tapb = 0;
    if (!fuse && !c.pw && c.seg_mode && c.SPI % 4 != 0 && c.nr == 1 && s.stride == 1 && s.dilation == 1 && c.CK == 32 && c.chunks == 1 && c.NT == 1 && 2 * c.Np <= 256 &&
        3u * (uint32_t)c.Cg * (uint32_t)c.Np * 4u <= 40u * 1024u) {
        c.tapb = 1;
        c.nr = 3;
        c.wseg = 4;
        c.nseg = 12;
    }
    if (c.pw) c.need_xchg = 0;                          // no horizontal neighbours to exchange
    c.fast4 = 0;
    c.nacc = 4 * c.Np <= 512 ? 4 : 2;                 // even, so a buffer always meets the same issuing warp and epilogue group
    c.issuers = c.nacc;                                // MMA-issuing warps: one per accumulator buffer
    // Row boxes with narrow groups (the two-CTA shape below): stages of 16 channels.  Twice as many stages of half the
    // size let a tile's first MMAs start when half of its input has arrived and hand shared memory back to the copies
    // in smaller pieces: 3-7 % on 56x56 and 28x28 planes (256 channels @56x56 N = 32 g = 8: 44.2 -> 42.8 us,
    // 64 @56x56 N = 64 g = 4: 23.7 -> 22.2 us, 128 @28x28 N = 64 g = 8: 14.3 -> 13.4 us).  Planes 32 pixels wide
    // (halo stages of whole segments) measured the same either way and keep 32 channels.
    if (!fuse && !c.pw && c.rowbox && !c.s2h && c.nr == 3 && s.stride == 1 && s.dilation == 1 && c.CK == 32 && c.NT == 1 &&
        2 * c.Np <= 256 && (uint32_t)vt * (uint32_t)c.Cg * (uint32_t)c.Np * 4u <= 40u * 1024u) {
        c.CK = 16;
        c.chunks = c.Cg / 16;
    }
    // Pair tiles: a filter bank too large to stay resident streams through every CTA's shared memory once per pixel
    // tile, and that traffic (L2 -> shared memory), not the tensor core, bounds the wide layers.  A stage then holds the
    // input of TWO pixel tiles and one set of weight blocks; every weight block feeds two MMAs (one per tile, two
    // accumulators side by side in TMEM), so the weights cross once per 256 pixels.  Stages shrink to 16 channels so
    // that three of them fit; the two epilogue groups drain the two accumulators at the same time.  The decision uses
    // only the shape (the packed layout depends on CK).
    c.pair = 0;
    c.MTr = c.MT;
    if (!fuse && !c.pw && c.rowbox && !c.s2h && c.nr == 3 && s.stride == 1 && s.dilation == 1 && c.Kt == 64 && c.Cg % 16 == 0 &&
        (uint32_t)vt * (uint32_t)c.Cg * (uint32_t)c.Np * 4u > 144u * 1024u && (long long)c.groups * c.NT * c.MT >= 4LL * kLayoutSMs) {
        c.pair = 1;
        c.CK = 16;
        c.chunks = c.Cg / 16;
        c.MT = (c.MTr + 1) / 2;
        c.nacc = 1;
        c.issuers = 1;
    }
    // One large resident bank (40 .. 144 KB) on row boxes leaves little room for input stages, and two 32-channel
    // stages keep the copies only one stage ahead of the MMAs (tensor pipe active 56 %).  Stages of 16 channels and
    // the whole 226 KB give five or six of them: the copies run four stages ahead.
    bool deep_ring = false;
    {
        const uint32_t b_any = (uint32_t)vt * (uint32_t)c.Cg * (uint32_t)c.Np * 4u;
        const bool s1 = !c.s2h && s.stride == 1 && b_any <= 144u * 1024u && c.MT >= 2 * kLayoutSMs;
        const bool s2 = c.s2h && s.stride == 2 && c.MT >= kLayoutSMs && c.Cg >= 64;   // stride-2 row tiles, resident or streamed banks (one 32-channel chunk: slower)
        if (!c.pair && !fuse && !c.pw && c.rowbox && c.nr == 3 && s.dilation == 1 && c.CK == 32 && b_any > 40u * 1024u && (s1 || s2)) {
            deep_ring = true;
            c.CK = 16;
            c.chunks = c.Cg / 16;
        }
    }
    c.num_tiles = c.groups * c.NT * c.MT;
    c.div_mt = make_fastdiv((uint32_t)c.MT);
    c.div_spi = make_fastdiv((uint32_t)(c.seg_mode ? c.SPI : c.RB));
    c.div_w = make_fastdiv((uint32_t)s.W);
    c.div_nt = make_fastdiv((uint32_t)c.NT);
    const uint32_t blk = (uint32_t)c.Np * c.CK * 4u;
    const uint32_t b_tile = (uint32_t)vt * c.chunks * blk;
    const uint32_t a_bytes = (uint32_t)c.nseg * c.CK * 128u;
    const uint32_t xchg_bytes = c.need_xchg ? (uint32_t)(kMaxAcc * 4 * 2 * 64 * sizeof(float)) : 0u;
    // Weights of a (group, filter tile) stay resident in shared memory when they fit: two buffers (the next group's
    // weights load while the current group computes) up to 40 KB each, one buffer (the switch waits for the MMAs
    // of the outgoing group) up to 144 KB; larger filter banks stream with the input stages.
    c.bres_stride = (b_tile + 1023u) & ~1023u;
    c.b_res = b_tile <= 40u * 1024u ? 2 : (b_tile <= 144u * 1024u ? 1 : 0);
    if (c.b_res == 2 && c.groups * c.NT == 1) c.b_res = 1;   // a single filter bank: nothing to switch to
    {   // a single resident buffer must still leave room for two input stages
        const uint32_t a_only = (a_bytes + 1023u) & ~1023u;
        if (c.b_res == 1 && c.bres_stride + 2u * a_only + xchg_bytes + 1024u > (uint32_t)kMaxDynSmem) c.b_res = 0;
        // loading a large filter bank up front only pays when a CTA reuses it over several pixel tiles
        if (!fuse && c.b_res == 1 && b_tile > 40u * 1024u && c.MT < (c.s2h ? 1 : (deep_ring ? 2 : 4)) * sm_count) c.b_res = 0;
    }
    if (fuse && c.b_res == 1 && c.groups * c.NT > 1) c.b_res = 0;   // the group changes every tile: stream, or two buffers
    c.egroups = 2;
    c.threads = kThreads;
    c.tmem_cols = kTmemCols;
    uint32_t budget_total = 200u * 1024u;
    const uint32_t w2_bytes = fuse ? (uint32_t)c.groups * (uint32_t)c.Kt * (uint32_t)C2 * 4u : 0u;   // resident pointwise weights
    uint32_t a2_bytes = fuse ? 2u * 4u * (uint32_t)c.Kt * 128u : 0u;                                   // one A2 operand buffer per epilogue group
    if (fuse) {
        budget_total = (uint32_t)kMaxDynSmem - 2048u - w2_bytes - a2_bytes;
        c.nacc = 2;
    }
    // Light configuration, two CTAs per SM: one epilogue group, two accumulators in 256 TMEM columns, one resident
    // weight buffer and half the shared memory.  The two CTAs hide each other's start-up, barrier and drain
    // latencies, and a CTA of the next kernel in the stream can start while one of this kernel's is still at work.
    {
        const uint32_t light_total = 110u * 1024u;
        const uint32_t st_bytes = (a_bytes + 1023u) & ~1023u;
        const int kst = (vt / c.nr) * c.chunks;
        const bool fits = !fuse && 2 * c.Np <= 256 && b_tile <= 40u * 1024u &&
                          c.bres_stride + (uint32_t)(c.tapb ? 1 : (kst == 1 ? 2 : kst + 1)) * st_bytes + xchg_bytes + 1024u <= light_total;
        // the fused block in the same shape: one grouped issuer (warp 1), the second MMA warp issues the pointwise MMAs
        const bool fits_fused = fuse && c.groups * c.NT == 1 && 2 * c.Np + C2 <= 256 && b_tile <= 40u * 1024u &&
                                c.bres_stride + 2u * st_bytes + xchg_bytes + ((w2_bytes + 1023u) & ~1023u) + a2_bytes / 2u + 2048u <= light_total;
        if (fits_fused) a2_bytes /= 2u;
        if (fits || fits_fused) {
            c.b_res = 1;
            c.nacc = 2;
            c.issuers = fits_fused ? 1 : 2;
            c.egroups = 1;
            c.threads = 32 * kEpi2First;       // producer, first MMA warp, first epilogue group, second MMA warp
            c.tmem_cols = 256;
            budget_total = light_total - 1024u - (fits_fused ? ((w2_bytes + 1023u) & ~1023u) + a2_bytes + 1024u : 0u);
        }
    }
    c.nt_fast = (!c.b_res && c.NT > 1) ? 1 : 0;
    c.stage_bytes = ((c.pair ? 2u : 1u) * a_bytes + (c.b_res ? 0u : (uint32_t)c.nr * blk) + 1023u) & ~1023u;
    if (c.pair) budget_total = 216u * 1024u;          // three 68 KB stages
    if (deep_ring && (c.b_res == 1 || c.s2h)) budget_total = (uint32_t)kMaxDynSmem - 2048u;
    const uint32_t budget = budget_total - (uint32_t)c.b_res * c.bres_stride - xchg_bytes;
    int st = (int)(budget / c.stage_bytes);
    if (st > 8) st = 8;
    if (st < 2 && !c.tapb) st = 2;
    if (st < 1) st = 1;
    c.stages = st;
    c.xchg_off = (uint32_t)c.stages * c.stage_bytes + (uint32_t)c.b_res * c.bres_stride;
    c.smem_bytes = (size_t)c.xchg_off + xchg_bytes + 1024;
    c.grid = c.egroups == 1 ? (c.num_tiles < 2 * sm_count ? c.num_tiles : 2 * sm_count)
                            : (c.num_tiles < sm_count ? c.num_tiles : sm_count);
    // With a single resident weight buffer a switch of (group, filter tile) stalls the pipeline, so the CTAs split
    // into one set per pair and no CTA ever switches (two buffers hide the switch; there the plain order keeps all
    // SMs busy and balanced).
    c.cps = 0;
    c.fuse = fuse ? 1 : 0;
    c.ball = (fuse && c.b_res == 2 && c.groups * c.NT == 2) ? 1 : 0;   // both banks of a two-group block stay resident
    c.C2 = C2;
    c.n_gn = c.groups * c.NT;
    c.div_ngn = make_fastdiv((uint32_t)c.n_gn);
    c.d2_col = c.nacc * c.Np;
    c.d2_bufs = (fuse && c.d2_col + 2 * C2 <= c.tmem_cols) ? 2 : 1;
    c.w2_off = (uint32_t)c.smem_bytes - 1024u;             // behind the stages (and the exchange area)
    c.a2_off = c.w2_off + ((w2_bytes + 1023u) & ~1023u);
    c.w2_goff = kHeaderBytes + sizeof(float) * (size_t)c.groups * c.NT * vt * c.chunks * c.Np * c.CK;
    if (fuse) {
        c.smem_bytes = (size_t)c.a2_off + a2_bytes + 1024;
        if (c.egroups == 2) c.issuers = 2;
        const int ctas = c.egroups == 1 ? 2 * sm_count : sm_count;
        c.grid = c.MT < ctas ? c.MT : ctas;                // a CTA takes whole pixel tiles (all groups of each)
    }
    {
        const int n_gn = c.groups * c.NT;
        if (!fuse && c.b_res == 1 && n_gn > 1 && c.grid >= n_gn) {
            c.cps = c.grid / n_gn;                   // CTAs per (group, filter tile)
            if (c.cps > c.MT) c.cps = c.MT;
            c.grid = c.cps * n_gn;
        }
    }
    return c;
}

IgemmCfg igemm_config(const Shape& s, int sm_count) { return igemm_config_c2(s, sm_count, 0); }

// ---- fused block: grouped 3x3 followed by a pointwise (1x1, groups = 1) convolution C_out -> C2 ------------------------
bool igemm_block_supported(const Shape& s, int C2) {
    if (!s.square() || !igemm_supported(s) || s.KH != 3 || s.stride != 1 || s.dilation != 1 || C2 < 16 || C2 > 256 || C2 % 16 != 0) return false;   // C2 is the N of one MMA
    const IgemmCfg c = igemm_config_c2(s, kLayoutSMs, C2);
    if (c.NT != 1 || c.need_xchg || c.padded || c.nacc != 2) return false;
    if (c.d2_col + C2 > c.tmem_cols) return false;
    if ((uint32_t)c.groups * (uint32_t)c.Kt * (uint32_t)C2 * 4u >= (1u << 20)) return false;   // one barrier phase takes the whole of W2
    return c.stages >= 2 && c.smem_bytes <= (size_t)kMaxDynSmem;
}

size_t igemm_block_packed_bytes(const Shape& s, int C2) {
    const IgemmCfg c = igemm_config_c2(s, kLayoutSMs, C2);
    return c.w2_goff + sizeof(float) * (size_t)c.groups * c.Kt * C2;
}

namespace {
// Pointwise weights w2[C2][C_out] -> one K-major operand image per merged group: [k/8][k%8/4][n/8][n%8][4 channels],
// k = channel of the group's Kt grouped outputs, n = pointwise output channel; values rounded to TF32.
__global__ void block_pack_w2_kernel(int groups, int Kt, int C2, int C_mid, const float* __restrict__ w2, uint32_t* __restrict__ dst) {
    const size_t total = (size_t)groups * Kt * C2;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        size_t t = i;
        const int e = (int)(t % 4); t /= 4;
        const int n8 = (int)(t % 8); t /= 8;
        const int nb = (int)(t % (C2 / 8)); t /= (C2 / 8);
        const int k2 = (int)(t % 2); t /= 2;
        const int k8 = (int)(t % (Kt / 8));
        const int g = (int)(t / (Kt / 8));
        const int k = k8 * 8 + k2 * 4 + e, n = nb * 8 + n8;
        const float v = w2[(size_t)n * C_mid + (size_t)g * Kt + k];
        uint32_t u;
        asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(u) : "f"(v));
        dst[i] = u;
    }
}
}  // namespace

// Tag of a packed blob of this variant: the shape tag extended by every configuration field the packed layout depends
// on.  Merge width, filter tile and stage width follow the stride, the batch and the plane size, so weights packed
// under a descriptor of another batch, plane or stride either have the same layout (and are accepted) or another tag
// (and the kernel reports GCONV_ERR_PACK_MISMATCH); they are never read in the wrong layout.
static uint32_t igemm_tag(const Shape& s, const IgemmCfg& c) {
    uint32_t h = pack_tag(s, GCONV_VARIANT_IGEMM_TF32);
    const int v[10] = {c.merge, c.groups, c.Cg, c.Kg, c.CK, c.chunks, c.Kt, c.NT, c.Np, c.pw};
    for (int i = 0; i < 10; ++i) h ^= (uint32_t)v[i] + 0x9e3779b9u + (h << 6) + (h >> 2);
    return h;
}
static uint32_t block_tag(const Shape& s, const IgemmCfg& c, int C2) { return igemm_tag(s, c) ^ (0xB10C0000u + (uint32_t)C2); }

cudaError_t igemm_block_pack(const Shape& s, int C2, const float* w, const float* w2, void* packed, cudaStream_t st) {
    const IgemmCfg c = igemm_config_c2(s, kLayoutSMs, C2);
    const size_t total = (size_t)c.groups * c.NT * 3 * c.chunks * c.Np * c.CK;
    int blocks = (int)((total + 255) / 256 < 2368 ? (total + 255) / 256 : 2368);
    igemm_pack_kernel<<<blocks, 256, 0, st>>>(s, c, w, reinterpret_cast<uint32_t*>(packed), block_tag(s, c, C2));
    const size_t t2 = (size_t)c.groups * c.Kt * C2;
    blocks = (int)((t2 + 255) / 256 < 2368 ? (t2 + 255) / 256 : 2368);
    block_pack_w2_kernel<<<blocks, 256, 0, st>>>(c.groups, c.Kt, C2, s.C_out, w2,
                                                 reinterpret_cast<uint32_t*>(reinterpret_cast<uint8_t*>(packed) + c.w2_goff));
    return cudaGetLastError();
}

size_t igemm_packed_bytes(const Shape& s) {
    const IgemmCfg c = igemm_config(s, 148);
    return kHeaderBytes + sizeof(float) * (size_t)c.groups * c.NT * (c.pw ? 1 : 3) * c.chunks * c.Np * c.CK;
}

cudaError_t igemm_pack(const Shape& s, const float* w, void* packed, cudaStream_t st) {
    const IgemmCfg c = igemm_config(s, 148);
    const size_t total = (size_t)c.groups * c.NT * (c.pw ? 1 : 3) * c.chunks * c.Np * c.CK;
    int blocks = (int)((total + 255) / 256 < 2368 ? (total + 255) / 256 : 2368);
    igemm_pack_kernel<<<blocks, 256, 0, st>>>(s, c, w, reinterpret_cast<uint32_t*>(packed), igemm_tag(s, c));
    return cudaGetLastError();
}

static cudaError_t igemm_launch(const Shape& s_true, int C2, const float* x_in, const void* packed, float* y, Status* status,
                                int sm_count, cudaStream_t st, float* scratch, const IgemmLaunchOpts& opts);

cudaError_t igemm_forward(const Shape& s_true, const float* x_in, const void* packed, float* y, Status* status, int sm_count,
                          cudaStream_t st, float* scratch, const IgemmLaunchOpts& opts) {
    return igemm_launch(s_true, 0, x_in, packed, y, status, sm_count, st, scratch, opts);
}

cudaError_t igemm_block_forward(const Shape& s, int C2, const float* x, const void* packed, float* y2, Status* status, int sm_count,
                                cudaStream_t st, const IgemmLaunchOpts& opts) {
    return igemm_launch(s, C2, x, packed, y2, status, sm_count, st, nullptr, opts);
}

static cudaError_t igemm_launch(const Shape& s_true, int C2, const float* x_in, const void* packed, float* y, Status* status,
                                int sm_count, cudaStream_t st, float* scratch, const IgemmLaunchOpts& opts) {
    IgemmCfg c = igemm_config_c2(s_true, sm_count, C2);
    if (opts.wait_us > 0) c.wait_us = opts.wait_us;
    c.dbg_skip = opts.dbg_skip;
    Shape s = as_3x3(s_true);
    const float* x = x_in;
    if (c.padded) {
        if (scratch == nullptr) return cudaErrorInvalidValue;
        const IgemmGeom ge = igemm_geom(s);
        const size_t planes = (size_t)s.N * s.C_in;
        const size_t total = planes * ge.Hp * (ge.Wp / 4);
        const int blocks = (int)((total + 255) / 256 < (size_t)sm_count * 16 ? (total + 255) / 256 : (size_t)sm_count * 16);
        const FastDiv div_plane = make_fastdiv((uint32_t)(ge.Hp * (ge.Wp / 4))), div_row = make_fastdiv((uint32_t)(ge.Wp / 4));
        if (total < (1ull << 32))
            igemm_pad_kernel<uint32_t><<<blocks, 256, 0, st>>>(x_in, scratch, planes, s.H, s.W, ge.Hp, ge.Wp, div_plane, div_row);
        else
            igemm_pad_kernel<uint64_t><<<blocks, 256, 0, st>>>(x_in, scratch, planes, s.H, s.W, ge.Hp, ge.Wp, div_plane, div_row);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        s.H = ge.Hp;
        s.W = ge.Wp;
        x = scratch;
    }
    EncodeTiledFn encode = get_encode_fn();
    if (encode == nullptr) return cudaErrorNotSupported;
    CUtensorMap xmap;
    const cuuint64_t HW = (cuuint64_t)s.H * s.W;
    const cuuint64_t dims[3] = {HW, (cuuint64_t)s.C_in, (cuuint64_t)s.N};
    const cuuint64_t strides[2] = {HW * 4, HW * 4 * (cuuint64_t)s.C_in};
    const cuuint32_t box[3] = {32, (cuuint32_t)c.CK, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    if (c.soft) {
        memset(&xmap, 0, sizeof(xmap));      // the gather producer uses no swizzled map (and odd planes cannot have one)
    } else {
        const CUresult r = encode(&xmap, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float*>(x), dims, strides, box, estr,
                                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
    }
    // 4-D view for whole-tile copies: (pixel, channel, 32-pixel segment, image); the segment axis re-walks the
    // pixel axis in steps of 128 bytes, so one box covers nseg consecutive segments.
    IgemmCfg cfg = c;
    CUtensorMap xmap4 = xmap;
    cfg.fast4 = 0;
    if (c.soft) {
        // gather producer: raw boxes of (boxpx flat pixels, CK channels) of one image, unswizzled; planes that are not a
        // multiple of 16 bytes are fetched by plain bulk copies instead (no map)
        if (!c.raw_bulk) {
            const cuuint32_t boxr[3] = {(cuuint32_t)c.boxpx, (cuuint32_t)c.CK, 1};
            if (encode(&xmap4, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float*>(x), dims, strides, boxr, estr,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
                return cudaErrorInvalidValue;
            cfg.fast4 = 1;   // the second map is in use (prefetch its descriptor)
        }
    } else if (c.rowbox) {
        // (column, channel, row segment, row, image); the segment axis steps (W - 32) columns
        const cuuint64_t dims5[5] = {(cuuint64_t)s.W, (cuuint64_t)s.C_in, (cuuint64_t)c.SR, (cuuint64_t)s.H, (cuuint64_t)s.N};
        const cuuint64_t strides5[4] = {HW * 4, c.SR == 2 ? (cuuint64_t)(s.W - 32) * 4 : 128, (cuuint64_t)s.W * 4,
                                        HW * 4 * (cuuint64_t)s.C_in};
        const cuuint32_t box5[5] = {32, (cuuint32_t)c.CK, (cuuint32_t)(c.s2h ? 1 : c.SR), (cuuint32_t)(c.s2h ? 9 : (c.pw ? c.R : c.R + 2)), 1};
        const cuuint32_t estr5[5] = {1, 1, 1, 1, 1};
        if (encode(&xmap4, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 5, const_cast<float*>(x), dims5, strides5, box5, estr5,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
        cfg.fast4 = 1;   // the second map is in use (prefetch it)
    } else if (c.nr == 3 && !c.tapb && HW % 32 == 0) {
        // Halo stages of segment or flat-row tiles: (pixel in segment, channel, segment of the plane, image).  The box
        // starts wseg segments before the tile; segments before or after the plane are out of range and read as zeros,
        // so the first and last tiles of a plane are whole boxes too.
        const cuuint64_t dims4[4] = {32, (cuuint64_t)s.C_in, HW / 32, (cuuint64_t)s.N};
        const cuuint64_t strides4[3] = {HW * 4, 128, HW * 4 * (cuuint64_t)s.C_in};
        const cuuint32_t box4[4] = {32, (cuuint32_t)c.CK, (cuuint32_t)c.nseg, 1};
        const cuuint32_t estr4[4] = {1, 1, 1, 1};
        if (encode(&xmap4, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, const_cast<float*>(x), dims4, strides4, box4, estr4,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS)
            cfg.fast4 = 2;
        else
            xmap4 = xmap;
    } else if (!c.tapb && c.seg_fstep == 32 && (!c.seg_mode || c.SPI % 4 == 0)) {
        const cuuint64_t dims4[4] = {HW, (cuuint64_t)s.C_in, 8, (cuuint64_t)s.N};
        const cuuint64_t strides4[3] = {HW * 4, 128, HW * 4 * (cuuint64_t)s.C_in};
        const cuuint32_t box4[4] = {32, (cuuint32_t)c.CK, (cuuint32_t)c.nseg, 1};
        const cuuint32_t estr4[4] = {1, 1, 1, 1};
        if (encode(&xmap4, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, const_cast<float*>(x), dims4, strides4, box4, estr4,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS)
            cfg.fast4 = 1;
        else
            xmap4 = xmap;
    }
    using KernelFn = void (*)(const CUtensorMap, const CUtensorMap, const Shape, const IgemmCfg, const uint32_t*, float*, Status*, uint32_t,
                              const float*);
    static const KernelFn kernels[kFamilies] = {igemm_tf32_kernel<0>, igemm_tf32_kernel<1>, igemm_tf32_kernel<2>,
                                                igemm_tf32_kernel<3>, igemm_tf32_kernel<4>, igemm_tf32_kernel<5>,
                                                igemm_tf32_kernel<6>, igemm_tf32_kernel<7>, igemm_tf32_kernel<8>,
                                                igemm_tf32_kernel<9>, igemm_tf32_kernel<10>, igemm_tf32_kernel<11>,
                                                igemm_tf32_kernel<12>, igemm_tf32_kernel<13>,
                                                igemm_tf32_kernel<14>, igemm_tf32_kernel<15>, igemm_tf32_kernel<16>,
                                                igemm_tf32_kernel<17>, igemm_tf32_kernel<18>, igemm_tf32_kernel<19>, igemm_tf32_kernel<20>,
                                                igemm_tf32_kernel<21>, igemm_tf32_kernel<22>, igemm_tf32_kernel<23>,
                                                igemm_tf32_kernel<24>, igemm_tf32_kernel<25>, igemm_tf32_kernel<26>, igemm_tf32_kernel<27>, igemm_tf32_kernel<28>, igemm_tf32_kernel<29>, igemm_tf32_kernel<30>};
    int fam = 0;
    for (int f = 1; f < kFamilies && fam == 0; ++f)
        if (family_matches(f, s, cfg)) fam = f;
    if (cfg.pair && family(fam).pair != 1) return cudaErrorInvalidValue;   // the generic instantiation has no pair-tile code
    if (cfg.soft && cfg.egroups == 2 && family(fam).soft != cfg.soft) return cudaErrorInvalidValue;   // 29 warps: only the wide-group gather instantiations take them
    static bool attr_set[64][kFamilies] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64 || !attr_set[dev][fam]) {
        cudaError_t e = cudaFuncSetAttribute(kernels[fam], cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynSmem);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) attr_set[dev][fam] = true;
    }
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3((unsigned)c.grid);
    lc.blockDim = dim3((unsigned)c.threads);
    lc.dynamicSmemBytes = c.smem_bytes;
    lc.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    // Without the attribute the kernel starts only after everything before it in the stream has completed and is
    // visible (griddepcontrol.* are then no-ops): used for the first forward after any weight packing, because the
    // kernel reads the packed weights before its dependency wait.
    lc.numAttrs = opts.pdl ? 1 : 0;
    return cudaLaunchKernelEx(&lc, kernels[fam], xmap, xmap4, s, cfg, reinterpret_cast<const uint32_t*>(packed), y, status,
                              C2 > 0 ? block_tag(s_true, c, C2) : igemm_tag(s_true, c), x);
}


}  // namespace gconv
