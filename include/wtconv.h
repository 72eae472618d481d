/*
 * wtconv.h - C ABI of the B200 (sm_100a) WTConv library.
 *
 * The operator is the wavelet convolution of Algorithm 1 (Sec. 2.1 of the paper):
 *
 *   X^0 = x
 *   for l = 1..L:  Y^l = A X^(l-1)                 (2x2 orthonormal Haar analysis, Eq. 5)
 *                  Z^l = s^l (.) (Y^l *dw W^l)      (k x k depthwise conv on the 4C subband channels, then scale)
 *                  X^l = [Y^l]_LL                   (the raw low-pass band is carried down)
 *   R^(L+1) = 0
 *   for l = L..1:  R^l = A^T( ([Z^l]_LL + R^(l+1)) || [Z^l]_H )     (Haar synthesis)
 *   out = s^0 (.) (x *dw W^0 + b) + R^1
 *
 * evaluated with the three exact reformulations of Sec. 4: the analysis butterfly is
 * recomputed on chip (Sec. 4.1), the synthesis cascade is the bit-indexed closed form of
 * Proposition 2 (Sec. 4.2), and the scales are folded into the weights (Eq. 8) with the
 * gradients un-folded by Eq. 9 (Sec. 4.3).  The backward pass uses Sec. 2.2: the gradient
 * of analysis is synthesis and vice versa.
 *
 * Conventions fixed where the paper is silent:
 *   - "*dw" is a cross-correlation with zero padding R = k/2:
 *         (X *dw W)[y,x] = sum_{u,v} W[u,v] X[y+u-R, x+v-R].
 *   - An odd height/width is zero-padded on the bottom/right to even before each Haar
 *     level: H_l = ceil(H_(l-1)/2); each synthesis result is cropped back.
 *   - Subband order is (LL, LH, HL, HH); LH = (a+b-c-d)/2 carries the row sign, HL the
 *     column sign, for the 2x2 block [a b; c d].
 *
 * Memory and execution contract (every entry point unless it says otherwise):
 *   - Every pointer named "device" is a device pointer owned by the caller.  The library
 *     never allocates, frees or synchronises; work is enqueued on `stream` and is complete
 *     when the stream reaches that point.
 *   - Activations (x, out, grad_out, grad_x) are contiguous [B][C][H][W] in `desc->dtype`,
 *     base pointers 16-byte aligned.  Parameters and parameter gradients are float32 in
 *     every mode; all arithmetic and accumulation is float32.
 *       w0 [C][k][k]   s0 [C]   b0 [C] or NULL (no bias)
 *       wl [L][C][4][k][k]   sl [L][C][4]      (ignored, may be NULL, when L == 0)
 *   - Outputs are overwritten, never accumulated into.
 *   - `workspace` is device scratch of at least the size wtconv_workspace_bytes reports,
 *     256-byte aligned; its contents are undefined before and after a call.  Two calls
 *     that overlap in time need distinct workspaces.
 *   - Errors are returned as status codes before anything is launched; nothing traps or
 *     aborts.  A failed launch is reported as WTCONV_ERR_CUDA.
 */
#ifndef WTCONV_H_
#define WTCONV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum { WTCONV_F32 = 0, WTCONV_F16 = 1, WTCONV_BF16 = 2 } wtconv_dtype;

typedef enum {
    WTCONV_OK = 0,
    WTCONV_ERR_NULL = 1,        /* a required pointer is NULL */
    WTCONV_ERR_SHAPE = 2,       /* B, C, H or W < 1, or the tensor exceeds 2^31-1 elements per plane set limits */
    WTCONV_ERR_KERNEL_SIZE = 3, /* k not in {3, 5, 7} */
    WTCONV_ERR_LEVELS = 4,      /* L outside [0, WTCONV_MAX_LEVELS] */
    WTCONV_ERR_DTYPE = 5,
    WTCONV_ERR_ALIGNMENT = 6,   /* an activation pointer is not 16-byte aligned, or workspace not 256-byte aligned */
    WTCONV_ERR_WORKSPACE = 7,   /* workspace NULL or smaller than required */
    WTCONV_ERR_ALIAS = 8,       /* an output overlaps an input */
    WTCONV_ERR_ARCH = 9,        /* the current device is not compute capability 10.x */
    WTCONV_ERR_CUDA = 10,       /* a CUDA runtime call or launch failed */
    WTCONV_ERR_TIMEOUT = 11     /* a bounded device-side wait ran out (see wtconv_read_status) */
} wtconv_status;

#define WTCONV_MAX_LEVELS 8

/* desc->flags */
/* Never take the plane-resident kernels (used to test the tiled path).  This also keeps k = 3 on the per-level
 * kernels: by default a k = 3 layer whose shape the plane-resident k = 5 kernels serve is run through them with its
 * 3 x 3 filters copied into zero-bordered 5 x 5 tables at the head of the workspace (one small launch more per call,
 * two in the backward, which copies the inner 3 x 3 of the 5 x 5 weight gradients out; results are those of the
 * 3 x 3 layer exactly as defined; the block-per-plane kernels skip the border taps, the team and window kernels
 * multiply them with zeros). */
#define WTCONV_FLAG_TILED_ONLY 1u
/* Test aid for the timeout path of the bounded device-side waits: no bulk copy is issued at all and the wait
 * limit is tiny, so every wait for a copy runs out; the kernels record it in the status word and return
 * normally with nothing in flight (outputs are then invalid by design).  Never set it in production. */
#define WTCONV_FLAG_TEST_NO_COPY 2u
#define WTCONV_FLAG_NO_TEAM 4u /* never take the team kernels for small planes (used to test the block-per-plane kernels on them) */
#define WTCONV_FLAG_NO_WINDOW 64u /* never take the window kernels for large planes (used to test the tiled path on them) */
/* Large planes are served by the window kernels (levels 1-2 on chip, about 2.2 N elements of HBM traffic) when their
 * rows are not 16-byte multiples, and by the tiled kernels (per-level launches, Q_fused - 2 N of traffic, but faster
 * on this GPU when rows are aligned) otherwise; this flag takes the window kernels wherever they apply. */
#define WTCONV_FLAG_PREFER_WINDOW 128u
/* Comparator: run the layer as the chain of separate operators of Sec. 3.1 (analysis, depthwise conv, scale pass,
 * slice, add, concatenate, synthesis per level; base conv, scale pass, add), every intermediate in HBM, as plain
 * kernels of this library.  It is what the paper measures its fused kernels against (Eq. 2 vs Eq. 10, Tables 1-3);
 * in this mode wtconv_backward first re-runs the forward chain (the autograd tape) and then every operator's
 * gradient as its own launch, so it costs one reference training step.  Two further bits reproduce the cumulative
 * ablation of Table 8 on the forward chain: FUSED_ANALYSIS (butterfly on chip in the level conv kernel, Sec. 4.1),
 * COLLAPSED_SYNTHESIS (one closed-form pass, Sec. 4.2); with scale folding (Sec. 4.3) added on top the chain is
 * the paper's fused design = WTCONV_FLAG_TILED_ONLY.  Workspace sizes are far larger in this mode (query them). */
#define WTCONV_FLAG_REFERENCE_CHAIN 8u
#define WTCONV_FLAG_ABLATE_FUSED_ANALYSIS 16u
#define WTCONV_FLAG_ABLATE_COLLAPSED_SYNTHESIS 32u
/* Launch-plan overrides for the plane-resident kernels, for tuning experiments (0 = let the planner choose):
 *   bits  8-12  threads per block / 32 of the forward / input-gradient kernel
 *   bits 13-15  resident blocks per SM of that kernel
 *   bits 16-21  planes per work unit of that kernel (the only override the team kernels for tiny planes honour:
 *               planes per team unit, forward and backward)
 *   bits 22-27  planes per work unit of the backward kernels
 *   bit  28     never prefetch with bulk copies      bit 29  never use the fused backward kernel
 *   bit  30     only 4 x 8 register tiles            bit 31  only 4 x 4 register tiles
 * An override that cannot be met (shared memory, registers) makes the call fail with WTCONV_ERR_CUDA. */
#define WTCONV_TUNE(threads, blocks_per_sm, planes, bwd_planes)                                            \
    ((((uint32_t)(threads) / 32u) << 8) | ((uint32_t)(blocks_per_sm) << 13) | ((uint32_t)(planes) << 16) | \
     ((uint32_t)(bwd_planes) << 22))
#define WTCONV_TUNE_NO_BULK (1u << 28)
#define WTCONV_TUNE_NO_FUSED_BWD (1u << 29)
#define WTCONV_TUNE_TILE_8 (1u << 30)
#define WTCONV_TUNE_TILE_4 (1u << 31)

typedef struct {
    int32_t B, C, H, W; /* activation shape */
    int32_t k;          /* depthwise kernel size: 3, 5 or 7 */
    int32_t L;          /* decomposition levels, 0..WTCONV_MAX_LEVELS (0 = base path only) */
    int32_t dtype;      /* wtconv_dtype of the activations */
    uint32_t flags;
} wtconv_desc;

/* Static string for a status code (never NULL). */
const char *wtconv_status_string(wtconv_status st);

/* Level grid of Algorithm 1's Y^level: H_l = ceil(H / 2^level), same for W (level 0 = input).
 * Pure host integer math; errors: NULL, LEVELS (level < 0 or > WTCONV_MAX_LEVELS), SHAPE. */
wtconv_status wtconv_level_shape(const wtconv_desc *desc, int level, int32_t *Hl, int32_t *Wl);

/* Scratch bytes wtconv_forward / wtconv_backward need for this descriptor (host call, no CUDA).
 * Either output pointer may be NULL. */
wtconv_status wtconv_workspace_bytes(const wtconv_desc *desc, size_t *fwd_bytes, size_t *bwd_bytes);

/* Name of the kernel family a descriptor dispatches to ("team" = small planes, several per thread team; "plane" =
 * one block per whole plane in shared memory; "window" = large planes cut into windows with levels 1-2 on chip;
 * "tiled" = per-level tiled kernels; "reference-chain" = the comparator).  Host call; returns NULL for
 * an invalid desc. */
const char *wtconv_plan_name(const wtconv_desc *desc);

/* Launch plan of a descriptor as text (threads per block, resident blocks per SM, planes per work unit, register
 * tile rows, prefetch ring depth; "ring=0" = the kernel waits for no copy).  Host call.  Errors: NULL, desc. */
wtconv_status wtconv_plan_describe(const wtconv_desc *desc, char *buf, size_t n);

/* Number of kernel launches one wtconv_forward / wtconv_backward call enqueues. */
wtconv_status wtconv_launch_count(const wtconv_desc *desc, int32_t *fwd_launches, int32_t *bwd_launches);

/* Forward pass of Algorithm 1 (device pointers).  out must not overlap x. */
wtconv_status wtconv_forward(const wtconv_desc *desc, const void *x,
                             const float *w0, const float *s0, const float *b0,
                             const float *wl, const float *sl,
                             void *out, void *workspace, size_t workspace_bytes, void *stream /* cudaStream_t */);

/* Backward pass (device pointers): given grad_out = dLoss/d out, writes
 *   grad_x [B][C][H][W] (dtype), grad_w0 [C][k][k], grad_s0 [C], grad_b0 [C] (NULL iff b0 is NULL),
 *   grad_wl [L][C][4][k][k], grad_sl [L][C][4]      (float32; Eq. 9 already applied).
 * Stateless: everything is recomputed from x, nothing saved by wtconv_forward is needed.
 * grad_x must not overlap x or grad_out.  The batch reduction of the parameter gradients is
 * deterministic (fixed-order partial sums, finished in float64). */
wtconv_status wtconv_backward(const wtconv_desc *desc, const void *x, const void *grad_out,
                              const float *w0, const float *s0, const float *b0,
                              const float *wl, const float *sl,
                              void *grad_x, float *grad_w0, float *grad_s0, float *grad_b0,
                              float *grad_wl, float *grad_sl,
                              void *workspace, size_t workspace_bytes, void *stream);

/* Device-side status of the last call that used `workspace` (device pointer; NULL = the array built into the
 * library that wtconv_backward_static uses, on the current device) with this descriptor: enqueues on
 * `stream` a one-thread kernel that evaluates the workspace's status words and a copy of the result into
 * *h_flag (a HOST int32, pinned if the copy is to be asynchronous).  Once the stream has reached this point, 0
 * means every bounded wait inside the kernels completed (the paper's kernels wait for nothing; ours wait only
 * for their own bulk copies); non-zero means a wait ran out and the outputs of that call are not valid (report
 * it as WTCONV_ERR_TIMEOUT).  For descriptors served by the tiled kernels, which wait for nothing, *h_flag is
 * set to 0 at once.  The library itself never synchronises, so it cannot return that code from wtconv_forward /
 * wtconv_backward.
 * How the words work: no call clears them (a clearing operation between two kernels would keep the second from
 * starting behind the tail of the first).  Every call stamps its launches with a fresh tag; a block whose wait
 * ran out stores the tag in the first word, block 0 stores it in the second, and the two are equal only if the
 * last call timed out.  A call replayed from a captured graph repeats its tag, so after one replay has timed out
 * the later replays of that graph read as timed out as well.
 * Errors: NULL, the descriptor's own errors, ALIGNMENT (workspace), CUDA. */
wtconv_status wtconv_read_status(const wtconv_desc *desc, void *workspace, int32_t *h_flag, void *stream);

/* Backward pass for callers that cannot hand over a workspace.  (The paper has no counterpart: it never
 * discusses where its kernels' scratch comes from.)
 *
 * Some hosts of this library may not allocate device memory at the point where they call the backward pass:
 * an inference or training runtime that froze its memory plan at start-up, a plug-in that is only given the
 * input and output buffers, or a latency-critical loop in which cudaMalloc (which may synchronise the device
 * and can fail once memory is fragmented) is off limits.  This variant of wtconv_backward needs no workspace
 * argument: its scratch is a WTCONV_STATIC_SCRATCH_BYTES array built into the library image (so each GPU that
 * loads the library carries that much memory until the process exits).  It calls no cudaMalloc, cudaFree or
 * any other allocating routine.
 *
 * Same arguments, layouts, outputs and arithmetic as wtconv_backward, minus the workspace.  Differences:
 *   - WTCONV_ERR_WORKSPACE is returned, before anything is launched, when the descriptor needs more scratch
 *     than the built-in array holds (wtconv_workspace_bytes tells how much a descriptor needs; the shapes the
 *     whole-plane kernels serve need well under 1 MiB, large planes on the tiled path need far more).
 *   - The first call on each device looks up the array's device address (cudaGetSymbolAddress, with that
 *     device current); make that first call outside any stream capture.  Later calls on that device reuse it.
 *   - All calls on one device share the one array, and it keeps whatever the last call left in it.  No call
 *     depends on what it finds there (what must start at zero is cleared, the rest is written before it is
 *     read), so stale contents are harmless, but two calls whose kernels overlap on the GPU (different
 *     streams) race on it: serialise them, or use wtconv_backward with two workspaces.
 *   - The kernels' status word lives in the array too: read it with wtconv_read_status(desc, NULL, ...).
 *   - WTCONV_ERR_ARCH (device is not compute capability 10.x) is reported before the array is looked up. */
#define WTCONV_STATIC_SCRATCH_BYTES (8u << 20)
wtconv_status wtconv_backward_static(const wtconv_desc *desc, const void *x, const void *grad_out,
                                     const float *w0, const float *s0, const float *b0,
                                     const float *wl, const float *sl,
                                     void *grad_x, float *grad_w0, float *grad_s0, float *grad_b0,
                                     float *grad_wl, float *grad_sl, void *stream);

/* One training step from HOST memory: copies x, grad_out and the parameters to the device,
 * runs wtconv_forward and wtconv_backward, and copies out, grad_x and the parameter
 * gradients back, all asynchronously on `stream` (the host buffers should be pinned for the
 * copies to overlap; they must stay valid until the stream reaches this point).
 * Every h_* pointer is a HOST pointer with the layouts above; `workspace` is DEVICE scratch of
 * at least wtconv_step_host_workspace_bytes.  h_b0 / h_grad_b0 may both be NULL.
 * Copies overlap the kernels: large batches are processed in up to eight chunks whose uploads, kernels and
 * downloads run on `stream` and two library-internal streams (per device, created on the first call), and the
 * chunks' parameter gradients are added in chunk order; small ones send the forward result back while grad_out
 * is still being uploaded.  `stream` waits for the internal streams, so everything is complete when `stream`
 * reaches this point.  The first call on a device must not happen inside a stream capture, and two calls
 * on one device must not overlap in time (they would share the internal streams' ordering, not their data). */
wtconv_status wtconv_step_host_workspace_bytes(const wtconv_desc *desc, size_t *bytes);
wtconv_status wtconv_step_host(const wtconv_desc *desc, const void *h_x, const void *h_grad_out,
                               const float *h_w0, const float *h_s0, const float *h_b0,
                               const float *h_wl, const float *h_sl,
                               void *h_out, void *h_grad_x, float *h_grad_w0, float *h_grad_s0, float *h_grad_b0,
                               float *h_grad_wl, float *h_grad_sl,
                               void *workspace, size_t workspace_bytes, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* WTCONV_H_ */
