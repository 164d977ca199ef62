// Internal declarations shared by the host API and the kernel translation units of libgconv.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/gconv.h"

namespace gconv {
struct Status;
struct Shape {
    int N, C_in, H, W, C_out, KH, KW, stride, pad, dilation, groups;   // stride, pad, dilation: the row axis (S_h of Algorithm 1)
    int Cg, Kg, H_out, W_out;
    int stride_w, pad_w, dilation_w;                                   // the column axis (S_w); equal to the row values on square problems
    __host__ __device__ bool square() const { return stride_w == stride && pad_w == pad && dilation_w == dilation; }
};
}  // namespace gconv

// The descriptor behind gconv_desc_t.
struct gconv_desc {
    gconv::Shape s;
    int variant;                 // resolved variant (never AUTO)
    int forced;                  // 1 if set by gconv_desc_set_variant
    gconv::Status* status_dev;   // lazily allocated device status block
    int device;                  // device the status block lives on (-1 = none yet)
    int sm_count;
    int last_cuda_error;
    int last_detail;             // detail word that came with the last non-zero device status (which wait, which thread block)
    float* workspace;            // caller-owned device workspace attached by gconv_desc_set_workspace (nullptr = none)
    size_t workspace_bytes;
    unsigned long long pack_epoch_seen;   // value of the process-wide pack counter at this descriptor's last forward
    int wait_us;                 // time limit of one bounded wait inside a kernel, microseconds (0 = the default, one second)
    int dbg_skip;                // failure-path test hook: stage fill that CTA 0's producer leaves out (-1 = none)
};

namespace gconv {

constexpr int kHeaderBytes = 64;  // packed-weight blob header; keeps the payload 16-byte aligned
constexpr uint32_t kMagic = 0x47434e56u;  // "GCNV"

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

// Division by a run-time constant as multiply-high + shift; exact for numerators below 2^31.
struct FastDiv {
    uint32_t mul, shr, div;
    __device__ __forceinline__ void divmod(uint32_t n, uint32_t& q, uint32_t& r) const {
        const uint32_t qq = (div != 1) ? (__umulhi(n, mul) >> shr) : n;
        r = n - qq * div;
        q = qq;
    }
};
FastDiv make_fastdiv(uint32_t d);

// DIRECT_TILED, narrow groups (Kg in {1,2,4,8}): one thread per (image, group, row strip, 4-pixel chunk).
struct RowsCfg {
    FastDiv div_xq, div_yt, div_g;
    uint32_t items;
    int PR, vec, pad01;
};
bool rows_supported(const Shape& s);
RowsCfg rows_config(const Shape& s);
cudaError_t rows_forward(const Shape& s, const float* x, const void* packed, float* y, Status* status, cudaStream_t st);

// DIRECT_TILED, depthwise stream kernel: a warp holds `subs` row strips of XQ lanes each.
struct DwCfg {
    int XQ, subs, RH, chunks;   // lanes per row, rows' strips per warp, output rows per thread, row chunks per plane
    FastDiv div_chunks;
    uint32_t items, blocks;
};
// depthwise on small planes (direct_dw_plane.cu): batches of whole planes through shared memory
struct DwPlaneCfg {
    int PB, upp;                 // planes per batch, units (one strip of one or two output rows) per plane
    uint32_t planes, batches, grid, threads, smem_bytes;
    FastDiv div_upp, div_c;
};
bool dw_plane_supported(const Shape& s);
DwPlaneCfg dw_plane_config(const Shape& s, int sm_count);
cudaError_t dw_plane_forward(const Shape& s, const float* x, const void* packed, float* y, Status* status, int sm_count,
                             cudaStream_t st);
bool dw_supported(const Shape& s);
DwCfg dw_config(const Shape& s, int sm_count);
cudaError_t dw_forward(const Shape& s, const float* x, const void* packed, float* y, Status* status, int sm_count,
                       cudaStream_t st);

// DIRECT_TILED: launch geometry chosen on the host from the shape.
struct TiledCfg {
    int TXT, TY, KQ, GB, KT, CCH;          // x threads, rows, filter slabs, groups per CTA, filters per thread, channel chunk
    int IH, IW, IWP, LPR;                  // staged patch rows, columns, padded row pitch, lanes per staged row
    int tiles_x, tiles_y, kblocks, gblocks;
    int threads;
    size_t smem;
};
bool tiled_supported(const Shape& s);
size_t tiled_packed_bytes(const Shape& s);
TiledCfg tiled_config(const Shape& s, int sm_count);
cudaError_t tiled_pack(const Shape& s, const float* w, void* packed, cudaStream_t st);
cudaError_t tiled_forward(const Shape& s, const float* x, const void* packed, float* y, Status* status, int sm_count,
                          cudaStream_t st);

// IGEMM_TF32: tile geometry of the tcgen05 implicit-GEMM kernel.
struct IgemmCfg {
    int merge, groups, Cg, Kg;   // adjacent groups presented as one (block-diagonal filters); sizes after merging
    int CK, chunks;          // channels per pipeline stage, stages per vertical tap
    int nr, nseg, wseg;      // vertical taps served by one stage (1 or 3), segments per stage, segments per image row
    int b_res;               // resident weight buffers in shared memory: 0 (weights stream with the stages), 1 or 2
    int nt_fast;             // tile order: filter tile fastest (streamed weights) instead of pixel tile fastest
    uint32_t bres_stride;    // bytes between the two resident weight buffers
    int Kt, NT, Np;          // filters per tile, filter tiles per group, MMA N (3*Kt padded to 16)
    int seg_mode;            // 1: a tile is any four 32-pixel segments (W divides 32); 0: a tile is R whole rows
    int SPI, R, RB, MT;      // segments per image; rows per tile, row blocks per image; pixel tiles in total
    int seg_fstep;           // flat-pixel step between consecutive segments of an image
    int need_xchg;           // rows may straddle a warp boundary in the epilogue
    int nacc;                // accumulator buffers in the TMEM ring
    int issuers;             // MMA-issuing warps (2 or 4), one per accumulator buffer
    int egroups, threads;    // epilogue groups of eight warps (1 or 2) and the block size that goes with them
    int cps;                 // CTAs per (group, filter tile) when the grid is split into one set per pair, else 0
    int tapb;                // one stage holds three blocks of four segments, one per vertical tap (small planes)
    // fused grouped + pointwise block (0 for the plain convolution)
    int fuse, C2, n_gn, d2_col;   // pointwise output channels, (group, filter tile) pairs per pixel tile, TMEM column of its accumulator
    int pw;                       // pointwise layer, stride 1: one vertical tap per chunk, one accumulator per filter (N = Kt)
    int soft;                     // gather producer: raw input rows land in a ring by bulk copy, copy warps build the operand stages from
                                  // them (1: stride 1, three vertical-tap blocks; 2: stride 2, even/odd column blocks per tap)
    int sub_h, sub_w;             // 1: a stride of 2 on that axis, taken as the even rows (columns) of the stride-1 result when it is stored
    int rps, IPT;                 // gather tilings: output rows per 32-lane segment; whole images per tile (1: a tile is part of one image)
    int boxpx, pieces, raw_whole, raw_bulk;   // raw part = `pieces` boxes of boxpx flat pixels x CK channels; parts hold whole planes; one 1-D copy per part
    int raw_stages;               // depth of the raw ring
    uint32_t raw_off, raw_bytes;  // shared-memory offset of the raw ring, bytes per raw buffer
    FastDiv div_boxpx;
    int ball;                     // every (group, filter tile) keeps a resident weight buffer of its own: no switches
    int d2_bufs;                  // pointwise accumulators in TMEM (2 when the columns allow: alternate pixel tiles)
    uint32_t w2_off, a2_off;      // shared-memory offsets of the resident pointwise weights and of the two A2 buffers
    size_t w2_goff;               // byte offset of the pointwise weight blocks inside the packed buffer
    FastDiv div_ngn;
    int tmem_cols;           // TMEM columns the CTA allocates (power of two >= nacc * Np)
    uint32_t xchg_off;       // offset of the edge-lane exchange area in dynamic shared memory
    int fast4;               // a second tensor map for whole-tile copies is available
    int padded, Hv, Wv;      // the kernel computes on a zero-padded copy of x; valid extent of the plane
    int s2h, lbo_segs;       // stride-2 row tiles (four output rows of one segment, nine staged input rows); segments between M blocks
    int rowbox, SR;          // tile = R whole rows of SR 32-pixel segments each (widths that do not divide 32)
    int pair, MTr;           // pair tiles: a stage holds the input of two pixel tiles and one set of streamed weights (MT counts pairs, MTr tiles)
    int num_tiles, stages, grid;
    FastDiv div_nt;                   // (group, filter tile) index -> group
    FastDiv div_mt, div_spi, div_w;   // tile -> (group/filter tile, pixel tile); pixel tile -> (image, segment or row block); pixel -> (row, column)
    uint32_t stage_bytes;
    size_t smem_bytes;
    uint32_t wait_us;        // time limit of one bounded wait, microseconds
    int dbg_skip;            // failure-path test hook: the stage fill CTA 0's producer leaves out (-1 = none)
};
// Per-launch options of the tensor-core variant.
struct IgemmLaunchOpts {
    bool pdl;                // launch with programmatic stream serialization (set-up overlaps the previous kernel's tail)
    uint32_t wait_us;        // 0 = default
    int dbg_skip;            // -1 = none
};
bool igemm_supported(const Shape& s);
IgemmCfg igemm_config(const Shape& s, int sm_count);
size_t igemm_packed_bytes(const Shape& s);
cudaError_t igemm_pack(const Shape& s, const float* w, void* packed, cudaStream_t st);
// fused block: grouped 3x3 (this shape) followed by a pointwise convolution C_out -> C2, one kernel, no intermediate in HBM
bool igemm_block_supported(const Shape& s, int C2);
size_t igemm_block_packed_bytes(const Shape& s, int C2);
cudaError_t igemm_block_pack(const Shape& s, int C2, const float* w, const float* w2, void* packed, cudaStream_t st);
cudaError_t igemm_block_forward(const Shape& s, int C2, const float* x, const void* packed, float* y2, Status* status, int sm_count,
                                cudaStream_t st, const IgemmLaunchOpts& opts);
size_t igemm_scratch_bytes(const Shape& s);   // device workspace the forward needs (padded copy of x), 0 for most shapes
cudaError_t igemm_forward(const Shape& s, const float* x, const void* packed, float* y, Status* status, int sm_count,
                          cudaStream_t st, float* scratch, const IgemmLaunchOpts& opts);

}  // namespace gconv
