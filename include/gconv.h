/*
 * libgconv -- forward grouped 2-D convolution for NVIDIA B200 (sm_100a), fp32 NCHW.
 *
 * The operation is the grouped convolution G(g) of Section II of the paper ("Optimizing Grouped
 * Convolutions on Edge Devices"): C_out filters are split into g groups and each group sees only
 * its own C_in/g input channels.  With Cg = C_in/groups (the paper's CPG), Kg = C_out/groups (the
 * paper's KPG), in the index form of the convolution stage of Algorithm 1 (cross-correlation on
 * the zero-padded input, no kernel flip):
 *
 *   y[n, g*Kg + k, p, q] = sum_{c<Cg} sum_{r<KH} sum_{s<KW}
 *       x[n, g*Cg + c, p*stride + r*dilation - pad, q*stride + s*dilation - pad] * w[g*Kg + k, c, r, s]
 *
 *   H_out = floor((H + 2*pad - dilation*(KH-1) - 1)/stride) + 1, likewise W_out.
 *
 * Layouts (Section III-A footnote: row-major 4-D arrays):
 *   x  [N, C_in, H, W]            fp32, device memory
 *   w  [C_out, Cg, KH, KW]        fp32, device memory
 *   y  [N, C_out, H_out, W_out]   fp32, device memory
 *
 * Conventions for every call:
 *   - C linkage, no exceptions cross the boundary; every call that can fail returns an int status,
 *     GCONV_OK (0) on success.
 *   - "device" pointers are CUDA device pointers of the current device, "host" pointers are host
 *     memory.  The caller owns every buffer (the workspace of the few layers that need one included)
 *     and the stream; the library owns only the descriptor and a 16-byte device status block it
 *     allocates on the first pack/forward call of a descriptor.  No other device memory is ever
 *     allocated by the library.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  pack and
 *     forward only enqueue work on it and return without synchronising.
 *   - Device pointers must be 16-byte aligned (GCONV_ERR_ALIGNMENT otherwise).
 *   - There is no CPU fallback: without a CUDA device pack/forward return GCONV_ERR_CUDA.
 */
#ifndef GCONV_H_
#define GCONV_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct gconv_desc *gconv_desc_t; /* opaque; created/destroyed by the library */

enum gconv_status {
    GCONV_OK = 0,
    GCONV_ERR_NULL = 1,          /* a required pointer argument is NULL */
    GCONV_ERR_INVALID_ARG = 2,   /* a shape parameter is out of range or channels do not divide by groups */
    GCONV_ERR_UNSUPPORTED = 3,   /* the requested kernel variant cannot run this shape */
    GCONV_ERR_ALIGNMENT = 4,     /* a device pointer is not 16-byte aligned */
    GCONV_ERR_CUDA = 5,          /* a CUDA runtime/driver call failed; see gconv_last_cuda_error */
    GCONV_ERR_PACK_MISMATCH = 6, /* device status: w_packed was packed for another shape or variant */
    GCONV_ERR_TIMEOUT = 7,       /* device status: a bounded wait inside a kernel ran out */
    GCONV_ERR_TOO_LARGE = 8,     /* the layer does not fit the fixed scratch of gconv_forward_host_static */
    GCONV_ERR_WORKSPACE = 9      /* the layer needs a workspace (gconv_workspace_bytes) and none large enough is attached */
};

/* Kernel variants.  The numeric tolerance of a result follows the variant that produced it:
 * max|y - y_ref| / max|y_ref| <= 1e-5 for the FP32 variants, <= 5e-3 for the TF32 variant. */
enum gconv_variant_id {
    GCONV_VARIANT_AUTO = 0,           /* let the selector choose (default) */
    GCONV_VARIANT_DIRECT_GENERIC = 1, /* FP32 FFMA, one thread per output, any shape */
    GCONV_VARIANT_DIRECT_TILED = 2,   /* FP32 FFMA, shared-memory halo + register tiles; 3x3, dilation 1, narrow groups;
                                         depthwise 3x3 (pad 1) and 5x5 (pad 2) on a software-pipelined stream kernel */
    GCONV_VARIANT_IGEMM_TF32 = 3      /* TF32 tcgen05 implicit GEMM per (merged) group; 3x3 with pad = dilation or 1x1 with pad 0,
                                         stride 1 or 2 (per axis: gconv_desc_create_2d), W <= 128; dilation > 1 only with
                                         stride 1 on planes whose (padded) rows divide 32 pixels */
};

/*
 * gconv_desc_create -- describe one grouped-convolution problem (Section II; the divisibility rule
 * "input and output channels divisible by the number of groups" is Section III-B).
 *   out       host pointer receiving the handle (library-owned until gconv_desc_destroy).
 *   N..groups problem sizes; stride, pad and dilation apply to both spatial axes.
 * Host only: touches no device, so it works without a GPU.  Picks the kernel variant with the
 * built-in selector (a rule on the group width derived from measured timings; the choices that
 * depend on Cg, Kg, H*W and N -- tiling, filter tile, launch shape -- are made inside the variant).
 * Errors: GCONV_ERR_NULL (out), GCONV_ERR_INVALID_ARG (any size < 1, stride < 1, dilation < 1,
 * pad < 0, C_in or C_out not divisible by groups, empty output, or a tensor over 2^40 elements).
 */
int gconv_desc_create(gconv_desc_t *out, int N, int C_in, int H, int W, int C_out, int KH, int KW,
                      int stride, int pad, int dilation, int groups);

/*
 * gconv_desc_create_2d -- the same with one stride, padding and dilation per spatial axis: Algorithm 1 of the paper
 * reads input row oh*S_h + kh and column ow*S_w + kw, i.e. it carries a stride for each axis.
 *   y[n, g*Kg + k, p, q] = sum_{c, r, s} x[n, g*Cg + c, p*stride_h + r*dilation_h - pad_h, q*stride_w + s*dilation_w - pad_w]
 *                                        * w[g*Kg + k, c, r, s]
 *   H_out = floor((H + 2*pad_h - dilation_h*(KH-1) - 1)/stride_h) + 1, W_out likewise with the _w values.
 * With equal values per axis it is gconv_desc_create.  Of the problems whose axes differ the tensor-core variant takes
 * 3x3 filters with pad 1, dilation 1 and a stride of 2 on one axis only (width a multiple of 4): it computes the stride-1
 * layer and stores its even rows or columns.  Every other such problem (padding or dilation per axis, other strides)
 * runs on the FP32 generic variant within the FP32 tolerance; gconv_variant_supported says which applies.  Host only.
 * Errors as gconv_desc_create, each condition applied per axis.
 */
int gconv_desc_create_2d(gconv_desc_t *out, int N, int C_in, int H, int W, int C_out, int KH, int KW,
                         int stride_h, int stride_w, int pad_h, int pad_w, int dilation_h, int dilation_w, int groups);

/* Frees the descriptor and its device status block.  NULL is accepted. */
int gconv_desc_destroy(gconv_desc_t desc);

/* Output spatial size from the floor formula above.  Host only. */
int gconv_out_shape(gconv_desc_t desc, int *H_out, int *W_out);

/* Multiply-accumulate count of the layer, Eq. (2) of the paper:
 * N*C_in*C_out*KH*KW*H_out*W_out/groups.  Returns -1 for a NULL descriptor. */
long long gconv_macs(gconv_desc_t desc);

/* Size in bytes of the packed-weight buffer for the descriptor's current variant (0 for NULL). */
size_t gconv_packed_bytes(gconv_desc_t desc);

/* The variant the descriptor will run (never GCONV_VARIANT_AUTO), or -1 for NULL. */
int gconv_variant(gconv_desc_t desc);

/* 1 if `variant` can run this shape, else 0. */
int gconv_variant_supported(gconv_desc_t desc, int variant);

/*
 * Force a variant (tests, selector training) or return to the selector's choice with
 * GCONV_VARIANT_AUTO.  Packed weights are variant-specific: call before gconv_pack_weights and
 * re-pack after changing it.  Errors: GCONV_ERR_NULL, GCONV_ERR_INVALID_ARG (unknown id),
 * GCONV_ERR_UNSUPPORTED (the variant cannot run this shape; the descriptor is left unchanged).
 */
int gconv_desc_set_variant(gconv_desc_t desc, int variant);

/*
 * gconv_pack_weights -- the kernel-reshaping stage (first stage of Algorithm 1, Section III-B:
 * it does not depend on the input, so it is done once ahead of time).  Reorders (and, for the TF32
 * variant, rounds to TF32 with round-to-nearest) w[C_out, Cg, KH, KW] into the layout the
 * descriptor's variant reads, prefixed by a 64-byte header that names shape and variant.
 *   w_ochw    device, fp32 [C_out, Cg, KH, KW], read only.
 *   w_packed  device, gconv_packed_bytes(desc) bytes, written.  The blob is position independent
 *             and may be copied, saved and reloaded.
 * One kernel launch on `stream`.  Errors: GCONV_ERR_NULL, GCONV_ERR_ALIGNMENT, GCONV_ERR_CUDA.
 */
int gconv_pack_weights(gconv_desc_t desc, const float *w_ochw, void *w_packed, void *stream);

/*
 * gconv_forward -- the grouped convolution itself (Section II; Algorithm 1's input-reshaping,
 * convolution and output-reshaping stages fused into one kernel: the input tile is staged in
 * shared memory and y is written directly in NCHW).
 *   x_nchw    device, fp32 [N, C_in, H, W], read only; must not overlap y.
 *   w_packed  device, produced by gconv_pack_weights on a descriptor of the same shape and variant.
 *   y_nchw    device, fp32 [N, C_out, H_out, W_out], every element written.
 * Kernel launches only, on `stream`; allocates nothing; deterministic (no atomics on y).  A w_packed made for
 * another shape or variant -- or under a descriptor whose batch, plane size or stride led to another packed layout --
 * is detected on the device: y is left unwritten and gconv_last_status reports GCONV_ERR_PACK_MISMATCH.
 * A few layers need a workspace (see gconv_workspace_bytes); without one attached the call enqueues nothing and
 * returns GCONV_ERR_WORKSPACE.  Errors: GCONV_ERR_NULL, GCONV_ERR_ALIGNMENT, GCONV_ERR_WORKSPACE, GCONV_ERR_CUDA.
 */
int gconv_forward(gconv_desc_t desc, const float *x_nchw, const void *w_packed, float *y_nchw, void *stream);

/*
 * Workspace (the role of Algorithm 1's input-reshaping stage, Section III-B: a rearranged copy of the padded input).
 * The tensor-core variant stages its input with bulk tensor copies, whose rows must be multiples of 16 bytes.  Layers
 * whose width is not a multiple of 4 therefore either build their stages with copy warps (no workspace) or, where
 * that path does not apply, compute on a zero-padded copy of x kept in a caller-owned device workspace:
 *   gconv_workspace_bytes     bytes the descriptor's current variant needs; 0 for every layer whose width is a
 *                             multiple of 4, for the FP32 variants, and for the layers of this kind that the copy
 *                             warps serve (gconv_forward_launches reports 1 for them, 2 when a workspace is used).
 *   gconv_desc_set_workspace  attach a device buffer of at least that size (16-byte aligned, caller-owned, must stay
 *                             valid while forwards of this descriptor are in flight); NULL detaches.  Forwards of ONE
 *                             descriptor that overlap on the GPU would race on it: give concurrent streams their own
 *                             descriptors.  Host only; errors: GCONV_ERR_NULL, GCONV_ERR_ALIGNMENT.
 */
size_t gconv_workspace_bytes(gconv_desc_t desc);
int gconv_desc_set_workspace(gconv_desc_t desc, void *workspace, size_t bytes);

/*
 * gconv_forward_host -- the same operation (Section II) for callers whose activations live in host memory:
 * copies x to the device, runs gconv_forward and copies y back, all enqueued on `stream` in order.
 *   x_host    host, fp32 [N, C_in, H, W] (pinned memory makes the copies asynchronous).
 *   y_host    host, fp32 [N, C_out, H_out, W_out], written when the stream reaches that point.
 *   x_stage, y_stage   device staging buffers of the sizes of x and y, caller-owned.
 *   w_packed  device, as for gconv_forward.
 * Errors as gconv_forward.
 */
int gconv_forward_host(gconv_desc_t desc, const float *x_host, const void *w_packed, float *y_host,
                       float *x_stage, float *y_stage, void *stream);

/*
 * gconv_forward_host_static -- gconv_forward_host for callers that are not allowed to allocate
 * device memory (no counterpart in the paper; it exists for deployment reasons only).  Think of a
 * plugin living inside an application whose allocator owns the GPU, a service that fixes its memory
 * at start-up, or a loop that cannot take the device-wide synchronisation a cudaMalloc implies.
 * It calls no cudaMalloc/cudaFree and no allocating library routine: the status block, the staging
 * room for x and y and the workspace of the layers that need one live in one static device array
 * inside the library (16 MiB + 256 bytes, held by every GPU that loads the library until the
 * process ends).
 *   x_host    host, fp32 [N, C_in, H, W], read.
 *   w_packed  device, from gconv_pack_weights on a descriptor of the same shape and variant.
 *   y_host    host, fp32 [N, C_out, H_out, W_out], written.
 * Limit: x, y and gconv_workspace_bytes, each rounded up to 256 bytes, must fit in 16 MiB together;
 * larger layers return GCONV_ERR_TOO_LARGE and nothing is enqueued.
 * The call enqueues clear-status, copy-in, the kernel of the descriptor's variant and copy-out on
 * `stream`, then SYNCHRONISES the stream and returns GCONV_OK or the status the kernel recorded
 * (GCONV_ERR_PACK_MISMATCH, GCONV_ERR_TIMEOUT); so when it returns, y_host is complete.
 * Because it synchronises, the call cannot be part of a stream capture.
 * The first call made with a given device current resolves the static array's device address for
 * that device (cudaGetSymbolAddress, under a mutex); make that first call before any stream capture
 * is begun anywhere in the process.
 * All calls share the one array, which still holds the previous call's data: the status block is
 * cleared and the staging regions are rewritten on every call, so results never depend on it, but
 * calls that overlap on the GPU (two streams, two threads) race and must be serialised by the caller.
 * Errors: GCONV_ERR_NULL, GCONV_ERR_ALIGNMENT (w_packed), GCONV_ERR_TOO_LARGE, GCONV_ERR_CUDA.
 */
int gconv_forward_host_static(gconv_desc_t desc, const float *x_host, const void *w_packed, float *y_host, void *stream);

/*
 * Fused block: the grouped 3x3 convolution of the descriptor followed by a pointwise (1x1, groups = 1, no bias)
 * convolution C_out -> C2, the block that replaces a standard convolution in Section II of the paper ("G(g)": a
 * grouped convolution followed by a pointwise one that re-mixes the channels).  One kernel: the grouped result of a
 * 128-pixel tile never leaves the SM (TMEM -> shared memory -> second tensor-core contraction), so x is read once
 * and only y2 is written.  Runs on the tensor-core variant whatever variant the descriptor resolved to.
 *
 *   y2[n, k2, p, q] = sum_{o < C_out} w2[k2, o] * y[n, o, p, q],   y = the descriptor's grouped convolution of x
 *
 * gconv_block_supported  1 if the pair (descriptor, C2) can run fused, else 0: 3x3, pad 1, stride 1, dilation 1,
 *                        W a multiple of 4 and at most 62 or equal to 64 wide planes only where the grouped kernel
 *                        needs no edge exchange, merged group width a multiple of 8 with at most 64 filters per
 *                        group, C2 a multiple of 16 from 16 to 256 with 2 * 3 * (filters per merged group) + C2 <= 512,
 *                        and the resident pointwise weights (C_out * C2 * 4 bytes) must leave room for two input
 *                        stages.  "Supported" is not "faster than two launches": fusing pays on large planes
 *                        (32x32 and up), small planes with several groups per pixel tile run faster unfused.
 * gconv_block_packed_bytes  size of the packed buffer holding both weight tensors (0 if unsupported).
 * gconv_block_pack_weights  w_ochw device fp32 [C_out, C_in/groups, 3, 3]; w2 device fp32 [C2, C_out]; both rounded
 *                        to TF32 while packing; asynchronous on `stream`.
 * gconv_block_forward    x device fp32 [N, C_in, H, W]; y2 device fp32 [N, C2, H_out, W_out]; asynchronous on
 *                        `stream`; both TF32 contractions accumulate in FP32, the intermediate is kept in FP32 and
 *                        consumed as TF32.  Tolerance: max|y2 - ref| / max|ref| <= 5e-3 against the oracle's grouped
 *                        convolution followed by its 1x1 convolution.
 * Errors: GCONV_ERR_NULL, GCONV_ERR_ALIGNMENT, GCONV_ERR_UNSUPPORTED, GCONV_ERR_CUDA; device status as gconv_forward.
 */
int gconv_block_supported(gconv_desc_t desc, int C2);
size_t gconv_block_packed_bytes(gconv_desc_t desc, int C2);
int gconv_block_pack_weights(gconv_desc_t desc, int C2, const float *w_ochw, const float *w2, void *w_packed, void *stream);
int gconv_block_forward(gconv_desc_t desc, int C2, const float *x, const void *w_packed, float *y2, void *stream);

/* Number of kernel launches one gconv_forward of this descriptor enqueues (for launch accounting). */
int gconv_forward_launches(gconv_desc_t desc);

/*
 * Failure-path controls (the paper has no counterpart).  Every wait inside the tensor-core kernel is bounded: when one
 * runs out the kernel records GCONV_ERR_TIMEOUT, every role leaves, copies in flight are waited for, tensor memory is
 * freed and the kernel returns; the context stays usable.
 *   wait_limit_us  time limit of one wait in microseconds; <= 0 restores the default (one second).
 *   skip_stage     test hook: >= 0 makes the first thread block's producer leave out that stage fill (no copy is
 *                  issued, its barrier is never armed), so the consumer's wait on it runs out and the forward reports
 *                  GCONV_ERR_TIMEOUT through gconv_last_status, y partly unwritten; -1 switches it off.  Nothing
 *                  faults, traps or waits longer than the limit.
 * Host only.  Errors: GCONV_ERR_NULL.
 */
int gconv_desc_set_debug(gconv_desc_t desc, int wait_limit_us, int skip_stage);

/*
 * Synchronises `stream`, then reads and clears the descriptor's device status word: GCONV_OK, or
 * the first of GCONV_ERR_PACK_MISMATCH / GCONV_ERR_TIMEOUT a kernel of this descriptor recorded.
 * A kernel that records an error returns early; it never traps.  GCONV_ERR_CUDA if the sync fails.
 */
int gconv_last_status(gconv_desc_t desc, void *stream);

/* The cudaError_t (as int) of the last failed CUDA call made for this descriptor, 0 if none. */
int gconv_last_cuda_error(gconv_desc_t desc);

/* The detail word recorded with the last non-zero device status gconv_last_status returned for this descriptor: for
 * GCONV_ERR_TIMEOUT the wait that gave up (50 + buffer: depthwise plane batches waiting for their bulk copy;
 * 100 + stage: producer waiting for a free stage; 150/160 + buffer: raw ring;
 * 200 + buffer: accumulator free; 300/800 + stage: MMA waiting for a stage fill; 400 + buffer: epilogue waiting for an
 * accumulator; 500 + buffer: edge exchange; 600/700 + buffer: filter bank; 9xx: fused block), 1000 and up when a drain
 * wait ran out as well; for GCONV_ERR_PACK_MISMATCH the thread block that found it.  Host only; 0 if none. */
int gconv_last_status_detail(gconv_desc_t desc);

/* Static, NUL-terminated description of a status code. */
const char *gconv_status_string(int status);

/* Static name of a variant id ("direct_generic", ...), or "unknown". */
const char *gconv_variant_name(int variant);

#ifdef __cplusplus
}
#endif
#endif /* GCONV_H_ */
