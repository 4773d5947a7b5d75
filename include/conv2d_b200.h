/*
 * conv2d_b200 -- forward 2-D convolution for NVIDIA B200 (sm_100a), C ABI.
 *
 * The operation is the one optimised by Chen, Chen, Chen and Hu, "Optimizing
 * Memory Efficiency for Convolution Kernels on Kepler GPUs" (DAC 2017): a
 * C-channel image convolved with a bank of filters, one output map per filter
 * (Fig. 3a), in the paper's two cases -- one input channel (Section 3,
 * Algorithm 1) and many input channels (Section 4, Algorithm 2).
 *
 *     y[n,k,p,q] = sum_{c,r,s} x[n,c,p+r,q+s] * w[k,c,r,s]
 *     P = H-R+1, Q = W-S+1        (stride 1, no padding, filter not flipped)
 *
 * Symbols: N images, C input channels, H x W image, K filters, R x S taps,
 * P x Q output map.  (The paper has no batch, calls the filter count F and the
 * square filter size K, and uses H, W for its thread-block tile.)  Outputs are
 * anchored at the top-left pixel of their window: a tile needs extra input
 * only beyond its right and bottom edges (Section 3.1).
 *
 * Conventions shared by every entry point
 *   - x, w, y and workspace are DEVICE pointers unless an argument is named
 *     *_host.  Tensors are dense, contiguous, row-major fp32: x[N][C][H][W],
 *     w[K][C][R][S], y[N][K][P][Q].  Base addresses must be 16-byte aligned.
 *   - All memory is owned by the caller.  y must not overlap x, w or the
 *     workspace.  y is overwritten (no accumulation into prior contents).
 *   - Calls enqueue work on `cuda_stream` (a cudaStream_t passed as void*;
 *     NULL is the default stream) and return without synchronising, except
 *     conv2d_get_status and conv2d_fwd_host, which wait for the stream.
 *   - The library allocates no device memory.  There is no CPU fallback: on
 *     a machine without a usable sm_100 device every launch entry returns
 *     CONV2D_ERR_ARCH or CONV2D_ERR_CUDA.
 *   - Errors are reported by return code only; nothing is thrown.  Argument
 *     errors are detected before anything is enqueued.
 */
#ifndef CONV2D_B200_H
#define CONV2D_B200_H

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    CONV2D_OK = 0,
    CONV2D_ERR_NULL = 1,           /* a required pointer is NULL */
    CONV2D_ERR_SHAPE = 2,          /* non-positive extent, R > H, S > W, or a size beyond 32-bit element indexing */
    CONV2D_ERR_ALIGN = 3,          /* x, w, y or workspace not 16-byte aligned */
    CONV2D_ERR_WORKSPACE = 4,      /* workspace smaller than conv2d_fwd_workspace_size reports */
    CONV2D_ERR_UNSUPPORTED = 5,    /* no kernel instance for this algorithm/shape combination */
    CONV2D_ERR_ARCH = 6,           /* current device is not compute capability 10.x */
    CONV2D_ERR_CUDA = 7,           /* a CUDA runtime call failed (cudaGetLastError is left set) */
    CONV2D_ERR_DEVICE_TIMEOUT = 8  /* a bounded on-device wait expired; outputs of that launch are invalid */
} conv2d_status_t;

typedef enum {
    CONV2D_ALGO_AUTO = 0,  /* tensor cores (TF32) where an instance exists, else fp32 FMA */
    CONV2D_ALGO_FFMA = 1,  /* fp32 fused multiply-add on the CUDA cores; error <= 1e-5 * sum|x*w| */
    CONV2D_ALGO_TF32 = 2,  /* operands reduced to TF32 (rounded to nearest; truncated for 1 x 1 filters, see
                              conv2d_fwd_general), fp32 accumulation on tcgen05; error <= 2e-3 * sum|x*w| */
    CONV2D_ALGO_16BIT = 3  /* workspace query only: the size conv2d_fwd_general_16bit needs */
} conv2d_algo_t;

typedef enum {
    CONV2D_OPERAND_BF16 = 0,  /* bfloat16: the upper 16 bits of an IEEE fp32 */
    CONV2D_OPERAND_FP16 = 1   /* IEEE binary16 */
} conv2d_operand_t;

/* `flags` bits */
enum {
    /* The workspace already holds the filters of this exact call (same w contents,
       K, C, R, S and algorithm) in the kernel's internal order, left there by an
       earlier call: skip the re-ordering launch. */
    CONV2D_FLAG_WEIGHTS_PACKED = 1u
};

/*
 * Workspace query (host only, touches no device).
 * Writes to *bytes the workspace size conv2d_fwd_general needs for this shape
 * and algorithm: 0 for CONV2D_ALGO_FFMA; for TF32 (and AUTO) a 256-byte status
 * block followed by the filters re-ordered for the tensor-core kernel (the
 * counterpart of the transposed, padded filter block that Section 4.2 / Fig. 6
 * builds in shared memory, done once per call instead of once per thread block).
 * Returns CONV2D_ERR_UNSUPPORTED if `algo` is TF32 and no instance fits.
 */
conv2d_status_t conv2d_fwd_workspace_size(int N, int C, int H, int W, int K, int R, int S,
                                          conv2d_algo_t algo, size_t* bytes);

/*
 * Plan query (host only, touches no device; no counterpart in the paper, whose tilings are fixed per filter
 * size in its Table 1).  Writes into `text` one NUL-terminated line of space-separated key=value pairs that
 * describe how the tensor-core path (algo = TF32, AUTO or 16BIT) would cut this shape into work items:
 * addressing mode, rows of the M operand, pixels per item, item and grid counts, and which part of the
 * tensor-core work ends up in stored outputs (mma_useful_px: stored pixels / accumulator columns computed;
 * mma_useful_flops: 2*N*K*C*R*S*P*Q / flops of all MMAs issued).  "tensor_core=0" when no instance fits.
 * Returns CONV2D_ERR_WORKSPACE when text_bytes is too small (512 is enough), CONV2D_ERR_UNSUPPORTED for
 * algo = FFMA.
 */
conv2d_status_t conv2d_fwd_plan_describe(int N, int C, int H, int W, int K, int R, int S,
                                         conv2d_algo_t algo, char* text, size_t text_bytes);

/*
 * Special case, one input channel (Section 3, Algorithm 1).
 *   x [N][1][H][W], w [K][1][R][S], y [N][K][P][Q]; fp32 FMA arithmetic.
 * The filters are small in this case (Section 3.2) and are kept on chip for the
 * whole call: every thread block copies them into shared memory and reads them
 * with broadcast loads.  Tuned instances exist for R = S in {1, 3, 5, 7}; images
 * with W % 4 == 0 and at least 1024 output columns take the wide kernel that
 * stages input rows with bulk (TMA) copies; every other shape is computed by a
 * slower shape-agnostic kernel, never rejected.  N must not exceed 65535.
 * (A benchmark-only variant selected by an environment switch keeps the filters
 * in a per-device constant-memory bank instead; calls using it on different
 * streams must not overlap.)
 * workspace may be NULL (none is used); flags must be 0.
 */
conv2d_status_t conv2d_fwd_single_channel(const float* x, const float* w, float* y,
                                          int N, int H, int W, int K, int R, int S,
                                          void* workspace, size_t workspace_bytes,
                                          unsigned flags, void* cuda_stream);

/*
 * General case, C input channels (Section 4, Algorithm 2).
 *   x [N][C][H][W], w [K][C][R][S], y [N][K][P][Q].
 * algo = FFMA: register-tiled fp32 kernel (each thread accumulates a block of
 *   filters x horizontally adjacent outputs, as in Section 4.1-4.2); no workspace.
 * algo = TF32: implicit-GEMM on the tcgen05 tensor cores with the accumulator
 *   in tensor memory; needs the workspace reported by conv2d_fwd_workspace_size
 *   (16-byte aligned).  Its first 256 bytes are a status block: the filter
 *   re-ordering step of each call clears it, a call with CONV2D_FLAG_WEIGHTS_PACKED
 *   leaves it as it is (so a time-out stays visible until the next full call).
 *   1 x 1 filters with H*W and C multiples of 4 (C <= 8192) take a kernel whose
 *   operands and output all move by tensor-map (TMA) copies straight from and to
 *   the caller's tensors.  Up to 256 channels: no filter re-ordering (the flag is
 *   accepted and has no effect), the kernel clears the status block itself, and the
 *   tensor core truncates both fp32 operands to TF32 instead of the rounding to
 *   nearest the other shapes get (worst case 1.97e-3 * sum|x*w|, still inside the
 *   bound).  More channels: a short kernel first rounds the filters to nearest TF32
 *   into the workspace (what CONV2D_FLAG_WEIGHTS_PACKED then skips) and only the
 *   image is truncated (worst case below 1.6e-3 * sum|x*w|).  With more than 128
 *   filters the blocks may work in cluster pairs on two-SM MMAs; results do not
 *   depend on which form runs beyond the order of the fp32 additions.  Very deep
 *   layers on few pixels (1536 channels or more) may be computed as two halves of
 *   the contraction that are added into y after the call has zero-filled it; the
 *   result does not depend on timing.
 *   Layers with few output tiles (e.g. 14 x 14 images) split the contraction over
 *   a two-block cluster; results do not depend on timing.
 * algo = AUTO: TF32 when an instance exists and the workspace suffices, else FFMA.
 * C == 1 is accepted and gives the same result as the single-channel entry.
 */
conv2d_status_t conv2d_fwd_general(const float* x, const float* w, float* y,
                                   int N, int C, int H, int W, int K, int R, int S,
                                   conv2d_algo_t algo,
                                   void* workspace, size_t workspace_bytes,
                                   unsigned flags, void* cuda_stream);

/*
 * General case with 16-bit operands (Section 4, Algorithm 2, with the shorter data types
 * that Section 6 names as the next step).  Section 2.1's rule -- make the unit a thread
 * moves as wide as the memory's access width -- is applied to the tensor-core operand
 * layout: one 16-byte unit holds 8 channels where the TF32 path holds 4 fp32.
 *   x16 [N][C][H][W], w16 [K][C][R][S]: both of the element type `operand` names,
 *   y [N][K][P][Q]: fp32.  Products are exact, accumulation is fp32 on tcgen05 (kind::f16):
 *   the error against exact arithmetic on the given 16-bit values is <= 1e-5 * sum|x*w|.
 * Same kernel, tiling and status block as CONV2D_ALGO_TF32; the workspace size comes from
 * conv2d_fwd_workspace_size(..., CONV2D_ALGO_16BIT, ...), and CONV2D_FLAG_WEIGHTS_PACKED has the
 * same meaning (same operand type included).  All four pointers are device pointers and must
 * be 16-byte aligned; workspace is required.
 * Returns CONV2D_ERR_UNSUPPORTED when no tensor-core instance fits the shape or `operand`
 * is not one of the two values.
 */
conv2d_status_t conv2d_fwd_general_16bit(const void* x16, const void* w16, float* y,
                                         int N, int C, int H, int W, int K, int R, int S,
                                         conv2d_operand_t operand,
                                         void* workspace, size_t workspace_bytes,
                                         unsigned flags, void* cuda_stream);

/*
 * General case with zero padding (the paper convolves the valid extent only; this is the "same"-style
 * variant users of convolution layers ask for):
 *   y[n,k,p,q] = sum_{c,r,s} xz[n,c,p+r-pad_h,q+s-pad_w] * w[k,c,r,s],  xz = x inside the image, 0 outside,
 *   P = H + 2*pad_h - R + 1, Q = W + 2*pad_w - S + 1, y [N][K][P][Q].
 * With the tensor-core algorithms the kernel applies the padding while it stages the image; otherwise the call
 * zero-extends x into the workspace with one extra kernel and then runs conv2d_fwd_general on the extended
 * image.  Every algorithm and every property of that entry applies.  The workspace size comes
 * from conv2d_fwd_padded_workspace_size (the general workspace for the extended image, then the extended
 * image itself); it is required for every algorithm, 16-byte aligned, and its first 256 bytes are the
 * status block as usual.  pad_h, pad_w >= 0.  CONV2D_FLAG_WEIGHTS_PACKED keeps its meaning.
 * algo is AUTO, FFMA or TF32.  N * C must not exceed 65535 (CONV2D_ERR_UNSUPPORTED otherwise, as for an unknown
 * flag or algorithm; all of these are checked before anything is enqueued).
 */
conv2d_status_t conv2d_fwd_padded_workspace_size(int N, int C, int H, int W, int K, int R, int S,
                                                 int pad_h, int pad_w, conv2d_algo_t algo, size_t* bytes);
conv2d_status_t conv2d_fwd_general_padded(const float* x, const float* w, float* y,
                                          int N, int C, int H, int W, int K, int R, int S,
                                          int pad_h, int pad_w, conv2d_algo_t algo,
                                          void* workspace, size_t workspace_bytes,
                                          unsigned flags, void* cuda_stream);

/*
 * General case with zero padding and a stride (not in the paper, which has stride 1):
 *   y[n,k,p,q] = sum_{c,r,s} xz[n,c,stride*p+r-pad_h,stride*q+s-pad_w] * w[k,c,r,s],
 *   P = (H + 2*pad_h - R) / stride + 1, Q = (W + 2*pad_w - S) / stride + 1 (integer division), y [N][K][P][Q].
 * The call rewrites the problem as a stride-1 convolution over stride*stride times as many channels
 * ("space to depth": channel (c,a,b) of the rewritten image holds the pixels whose row is a and whose column
 * is b modulo the stride; the filters are split the same way) with two extra kernels into the workspace and
 * then runs conv2d_fwd_general on it: the same multiply-adds as the definition plus zeros, every algorithm.
 * 1 <= stride <= 8.  Workspace from conv2d_fwd_strided_workspace_size; required, 16-byte aligned, status
 * block first.  With CONV2D_FLAG_WEIGHTS_PACKED the rewritten filters of the previous call are reused too.
 * algo is AUTO, FFMA or TF32; N * C must not exceed 65535 (CONV2D_ERR_UNSUPPORTED otherwise, checked before
 * anything is enqueued).
 */
conv2d_status_t conv2d_fwd_strided_workspace_size(int N, int C, int H, int W, int K, int R, int S,
                                                  int pad_h, int pad_w, int stride, conv2d_algo_t algo, size_t* bytes);
conv2d_status_t conv2d_fwd_general_strided(const float* x, const float* w, float* y,
                                           int N, int C, int H, int W, int K, int R, int S,
                                           int pad_h, int pad_w, int stride, conv2d_algo_t algo,
                                           void* workspace, size_t workspace_bytes,
                                           unsigned flags, void* cuda_stream);

/*
 * General case on the tensor cores for callers that cannot hand over scratch memory.
 * (The paper has no counterpart; this is a packaging variant of conv2d_fwd_general with
 * algo = CONV2D_ALGO_TF32, same kernels, same results.)
 *
 * Who needs it: code that runs where device allocation is off the table -- inside a
 * latency-critical loop that must not touch the allocator, in a process whose memory pool was
 * sized up front and is fully handed out, or in a plug-in that is only given its input and
 * output buffers.  Such callers cannot call cudaMalloc (or a framework allocator) to obtain the
 * workspace that conv2d_fwd_general asks for.
 *
 * Here the status block and the re-ordered filters live in a fixed array of
 * 256 + 8 MiB bytes inside the library's device image: every GPU on which the library is
 * loaded gives up that much memory until the process exits.  The call allocates and frees
 * nothing, on the device or through any library.  Shapes whose re-ordered filters
 * need more (conv2d_fwd_workspace_size(..., CONV2D_ALGO_TF32) > 256 + 8 MiB) are rejected with
 * CONV2D_ERR_WORKSPACE before anything is enqueued; shapes without a tensor-core instance with
 * CONV2D_ERR_UNSUPPORTED.
 *
 * The first call on each device looks up the array's device address (a one-time set-up under a
 * lock, with that device current); make that first call outside any stream capture.
 * The array is shared by all calls on a device and keeps the previous call's contents: each
 * call clears the status block and rewrites every filter word it will read, so stale contents
 * are never used, but two calls whose kernels can overlap on the GPU (calls on different
 * streams without an ordering between them) race on it.  Issue these calls on one stream per
 * device, or order them with events.
 *
 * x, w, y: device pointers as for conv2d_fwd_general.  wait = 0: enqueue and return;
 * wait != 0: also wait for the stream and return CONV2D_ERR_DEVICE_TIMEOUT if a bounded
 * on-device wait expired.  After a wait = 0 call, conv2d_get_status(NULL, cuda_stream) on the
 * same device reports such a time-out (the array's status word stays set until the next call
 * of this entry point clears it).
 */
conv2d_status_t conv2d_fwd_general_noalloc(const float* x, const float* w, float* y,
                                           int N, int C, int H, int W, int K, int R, int S,
                                           int wait, void* cuda_stream);

/*
 * Host-buffer convenience path (no counterpart in the paper): x_host and
 * w_host are copied to the caller's device buffers x, w on the stream, the
 * convolution runs (single-channel kernel when C == 1, else conv2d_fwd_general
 * with `algo`), y is copied back into y_host and the stream is synchronised.
 * Host buffers should be page-locked for the copies to run at full speed.
 * Returns the first error met, or the device status after synchronising
 * (CONV2D_ERR_DEVICE_TIMEOUT if a bounded on-device wait expired).  The
 * workspace is the one conv2d_fwd_general would need for `algo`; it may be
 * NULL / 0 bytes when no tensor-core kernel can run (C == 1, algo = FFMA), and
 * it is only read for a status when the tensor-core kernel ran.
 */
conv2d_status_t conv2d_fwd_host(const float* x_host, const float* w_host, float* y_host,
                                float* x, float* w, float* y,
                                int N, int C, int H, int W, int K, int R, int S,
                                conv2d_algo_t algo,
                                void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Waits for `cuda_stream`, then reads the device's time-out words: the one the
 * single-channel kernels raise (read and cleared), the status word of the fixed
 * array of conv2d_fwd_general_noalloc if that entry has run on the current
 * device, and the status block at the start of `workspace` unless it is NULL.
 * Returns CONV2D_OK, CONV2D_ERR_DEVICE_TIMEOUT if a kernel gave up on a bounded
 * wait, or CONV2D_ERR_CUDA if the stream reported an error.
 */
conv2d_status_t conv2d_get_status(const void* workspace, void* cuda_stream);

/* Static, NUL-terminated description of a status code. */
const char* conv2d_status_string(conv2d_status_t status);

/*
 * Number of kernels this library has launched in the calling process since it
 * was loaded (all entry points, all streams); for accounting in benchmarks.
 */
unsigned long long conv2d_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* CONV2D_B200_H */
