// General case on the tcgen05 tensor cores: implicit-GEMM direct convolution with fp32 accumulators in
// tensor memory (the contraction of Section 4, Algorithm 2).  fp32 inputs run as TF32 (kind::tf32, K = 8
// per instruction), bf16 / fp16 inputs as kind::f16 (K = 16); a 64-byte staged unit is 16 fp32 or 32
// 16-bit channels of one pixel, so both share every shared-memory layout and descriptor.
//
// Mapping of the paper's design onto B200
//   * GEMM view: M = a block of 128 (or 64) filters, N = the pixels of a work item, contraction over
//     (channel, tap).  The accumulator block rAcc[F_T][W_T] of Algorithm 2 becomes a filters x pixels fp32
//     tile in tensor memory (lanes = filters, columns = pixels); a work item is any multiple of 32 pixels
//     up to 512, covered by one or two MMAs per K step.  (With the pixels as M a 128-filter problem needs
//     twice as many instructions, and the single issuing thread is what limits the rate.)
//   * Flat addressing: pixels are numbered in one sequence j = (n*H + h)*W + w over the whole batch.  For
//     tap (r,s) the input needed by output j is pixel j + r*W + s of the same channel, a pure shift.  Per
//     block of channels ONE run of tile_px + (R-1)*W + (S-1) pixels is staged ("block plus halo to the
//     right and below", Section 3.1/4.1) and every tap reads it through a descriptor whose start address
//     is shifted by r*W + s rows: the row reuse of Section 4.2 (one staged input row serves all
//     horizontal taps) extended to the vertical taps, with no im2col buffer.  Outputs whose window wraps
//     over the right or bottom image edge are computed but not stored.
//   * Patch addressing (wide images): the item is a rectangle of one image, patch_w columns wide, staged
//     row after row; the tap shift becomes r*patch_w + s and the halo (R-1) patch rows instead of (R-1)
//     image rows.  See ItemGeom.
//   * Few channels: taps are folded into the channel dimension (see make_plan), so that a staged channel
//     block is not mostly padding.
//   * Shared-memory operand layout: K-major, no swizzle: [channel/4][row][4 channels], i.e. each row
//     (pixel or filter) of a chunk is one 16-byte unit and rows are 16 bytes apart.  This is the
//     transposed staging of Fig. 6 (adjacent units belong to adjacent rows) in the unit size the tensor
//     core reads, and it is what makes a start address at any pixel legal.
//   * The filters are re-ordered once per call into exactly that layout in the workspace
//     ([filter block][channel block][tap][chunk][filter][unit], fp32 rounded to TF32) and either kept in
//     shared memory for the life of the block or streamed with 1-D bulk (TMA) copies through an mbarrier
//     ring.  Activations cannot be moved by TMA: NCHW has the pixels, not the channels, contiguous, and a
//     tiled copy cannot transpose nor start at a 4-byte offset; eight producer warps gather them
//     (coalesced along pixels, 128-bit loads where the alignment allows), round fp32 to TF32 and write
//     16-byte units.
//   * Persistent blocks, one per SM, walk over the work items round-robin.  Warp roles: warp 0 streams
//     filter stages, warp 1 (one thread) issues tcgen05.mma and owns the tensor-memory allocation, eight
//     warps stage activations (in up to four groups that fill different stages concurrently), four warps
//     drain finished accumulators through a shared-memory transposition so that a store instruction
//     writes adjacent outputs of one map (the coalesced write-back that Section 4.2 leaves out); for the
//     block's last item the other eight warps join the drain.  All rings run across item boundaries, so
//     the loads of the next item proceed under the MMAs of the current one (the prefetch of Algorithm 2),
//     and where two accumulator sets fit into the 512 tensor-memory columns the write-back of item i
//     overlaps the MMAs of item i+1.
//   * The kernel is launched with programmatic stream serialization: everything before grid_dep_wait()
//     touches only this block's shared and tensor memory and overlaps the preceding kernel's tail.
//   * Every wait is bounded; on expiry the block raises a flag, stops storing, frees its tensor memory and
//     the status word in the workspace becomes non-zero.
#include <cstdio>
#include <cstdlib>
#include <mutex>

#include "common.cuh"
#include "ptx.cuh"
#include "tc_plan.cuh"
#include "tc_repack.cuh"
#include "tc_kernel.cuh"

namespace conv2d_b200 {


bool tf32_supported(const Shape& sh)
{
    return make_plan(sh).ok || pointwise_tma_supported(sh, false);
}

size_t tf32_workspace_bytes(const Shape& sh)
{
    const Plan p = make_plan(sh);
    const size_t general = p.ok ? packed_floats(p) * sizeof(float) : 0;
    const size_t pointwise = pointwise_tma_workspace_extra(sh, false);
    return kStatusBytes + (general > pointwise ? general : pointwise);
}

bool b16_supported(const Shape& sh)
{
    return make_plan(sh, true).ok || pointwise_tma_supported(sh, true);
}

size_t b16_workspace_bytes(const Shape& sh)
{
    const Plan p = make_plan(sh, true);
    if (!p.ok) return kStatusBytes;
    return kStatusBytes + packed_floats(p) * sizeof(float);
}

// One line of text about the plan for `sh`: which addressing, item size, grid, and how much of the tensor-core work
// is useful.  mma_useful_px = stored output pixels / accumulator columns computed (the flat run and the patches also
// compute windows that wrap over an image edge); mma_useful_flops = 2*N*K*C*R*S*P*Q / flops of all MMAs issued
// (this also counts filter rows, channels and stacked taps that are zero padding).
int describe_tensor_core_plan(const Shape& sh, bool b16, char* text, size_t text_bytes)
{
    {
        const int n = describe_pointwise_tma_plan(sh, b16, text, text_bytes);
        if (n >= 0) return n;
    }
    const Plan p = make_plan(sh, b16);
    if (!p.ok) return snprintf(text, text_bytes, "tensor_core=0");
    const double out_px = (double)sh.N * sh.P * sh.Q;
    const double cols = (double)p.supertiles * p.tile_px;
    const double rows = p.swap ? p.n_tile : kTileM;                     // rows of the M operand
    const double ncols = p.swap ? (double)p.supertiles * p.tile_px * p.n_blocks
                                : (double)p.supertiles * p.mt * p.n_blocks * p.n_tile;
    const double kdim = (double)p.cblks * (b16 ? 2 * kCB : kCB) * p.taps;
    double issued = 2.0 * rows * ncols * kdim;
    if (p.pair_compact) issued *= (double)p.cb_bytes / ((double)p.taps * kCB * p.n_tile * 4);    // lone taps are 64-row MMAs
    const double useful = 2.0 * out_px * sh.K * sh.C * sh.R * sh.S;
    return snprintf(text, text_bytes,
                    "tensor_core=1 kernel=general_tc addressing=%s filters_as=%s m_rows=%d tile_px=%d px_groups=%d acc_sets=%d items=%lld grid=%d "
                    "ksplit=%d cluster=%d resident_filters=%d stacked_taps=%d stacked_compact=%d fold=%dx%d patch_w=%d smem_bytes=%zu "
                    "mma_useful_px=%.4f mma_useful_flops=%.4f",
                    p.patch_w ? "patch" : "flat", p.swap ? "M" : "N", (int)rows, p.tile_px, p.px_groups, p.nbuf,
                    (long long)p.supertiles * p.n_blocks * p.ksplit, p.grid, p.ksplit, p.cluster, p.resident, p.pair_taps, p.pair_compact,
                    p.fold_r, p.fold_s, p.patch_w, p.smem_bytes, out_px / cols, useful / issued);
}

namespace {
// workspace_bytes: checked against the plan's need here, so that a call plans only once (the planner reads two
// dozen environment switches and costs ~2 us); SIZE_MAX = the caller has checked already.
conv2d_status_t launch_tensor_core(const void* x_any, const void* w_any, float* y, const Shape& sh, bool b16, bool fp16,
                                   void* workspace, size_t workspace_bytes, bool weights_packed, cudaStream_t stream)
{
    const float* x = static_cast<const float*>(x_any);   // 16-bit operands: re-read as such inside the kernel
    const float* w = static_cast<const float*>(w_any);
    {
        // 1 x 1 filters on suitably aligned tensors: the kernel whose operands and output all move by tensor-map copies
        const conv2d_status_t st = launch_pointwise_tma(x_any, w_any, y, sh, b16, fp16, workspace, workspace_bytes, weights_packed, stream);
        if (st != CONV2D_ERR_UNSUPPORTED) return st;
    }
    const Plan p = make_plan(sh, b16);
    if (!p.ok) return CONV2D_ERR_UNSUPPORTED;
    if (env_int("CONV2D_B200_TF32_VERBOSE", 0) != 0)
        fprintf(stderr, "conv2d plan: n_tile %d n_blocks %d tile_px %d groups %d nbuf %d npix %d cblks %d taps %d stacked %d "
                "fold %dx%d patch_w %d tw %d rows %d cols %d a_stages %d cbg %d b_stages %d tps %d resident %d ksplit %d "
                "items %lld grid %d smem %zu\n",
                p.n_tile, p.n_blocks, p.tile_px, p.px_groups, p.nbuf, p.npix, p.cblks, p.taps, p.pair_taps, p.fold_r, p.fold_s,
                p.patch_w, p.patch_tw, p.patch_rows, p.patch_cols, p.a_stages, p.cbg, p.b_stages, p.tps, p.resident, p.ksplit,
                (long long)p.supertiles * p.n_blocks * p.ksplit, p.grid, p.smem_bytes);
    if (workspace_bytes < kStatusBytes + packed_floats(p) * sizeof(float)) return CONV2D_ERR_WORKSPACE;
    unsigned* status = static_cast<unsigned*>(workspace);
    float* wp = reinterpret_cast<float*>(static_cast<unsigned char*>(workspace) + kStatusBytes);

    if (!weights_packed) {
        const long long total = (long long)packed_floats(p);
        const FoldedFilter ff{sh.C, sh.R, sh.S, p.fold_r, p.fold_s};
        const long long lanes = (long long)p.n_blocks * p.cblks * kChunks * p.n_tile * (b16 ? 8 : 4);   // one thread per element of a tap's slice
        long long blocks = (lanes + 255) / 256;
        if (blocks > sm_count() * 16LL) blocks = sm_count() * 16LL;
        const size_t tile_bytes = (size_t)8 * kCB * 4 * p.taps;       // 8 filters x one channel block x taps
        if (p.fold_r * p.fold_s == 1 && tile_bytes <= 48 * 1024 && p.n_tile % 8 == 0 && !p.pair_taps) {
            const dim3 grid((unsigned)(p.n_blocks * p.n_tile / 8), (unsigned)p.cblks);
            int threads = (8 * kChunks * p.taps + 31) / 32 * 32;          // one 16-byte unit per thread in the store phase
            threads = threads < 128 ? 128 : (threads > 1024 ? 1024 : threads);
            // (launched the ordinary way: it starts only when the previous call's kernel, which may still
            // be reading the workspace, has finished; measured no gain from overlapping its launch)
            if (b16)
                repack_filters_tiled_kernel<unsigned short, 8><<<grid, threads, tile_bytes, stream>>>(
                    static_cast<const unsigned short*>(w_any), reinterpret_cast<unsigned short*>(wp), status, sh.K, sh.C,
                    p.taps, p.n_tile, p.cblks);
            else
                repack_filters_tiled_kernel<float, 4><<<grid, threads, tile_bytes, stream>>>(w, wp, status, sh.K, sh.C, p.taps,
                                                                                             p.n_tile, p.cblks);
        } else if (b16)
            repack_filters_kernel<unsigned short, 8><<<(unsigned)blocks, 256, 0, stream>>>(
                static_cast<const unsigned short*>(w_any), reinterpret_cast<unsigned short*>(wp), status, sh.K, ff,
                p.taps, p.n_tile, p.cblks, lanes, p.pair_taps + p.pair_compact);
        else
            repack_filters_kernel<float, 4><<<(unsigned)blocks, 256, 0, stream>>>(w, wp, status, sh.K, ff, p.taps,
                                                                                  p.n_tile, p.cblks, lanes, p.pair_taps + p.pair_compact);
        count_launch();
        if (cudaGetLastError() != cudaSuccess) return CONV2D_ERR_CUDA;
    }

    // The attribute belongs to a (function, device) pair: set once per device.  (A benign race: two threads
    // may both set it.)
    static bool attr_set_on[64] = {};
    int dev_id = 0;
    if (cudaGetDevice(&dev_id) != cudaSuccess || dev_id < 0 || dev_id >= 64) return CONV2D_ERR_CUDA;
    bool& attr_set = attr_set_on[dev_id];
    if (!attr_set) {
        void (*all[])(KernelArgs) = {general_tc_kernel<false, false, false, false>, general_tc_kernel<true, false, false, false>,
                                     general_tc_kernel<false, true, false, false>,  general_tc_kernel<true, true, false, false>,
                                     general_tc_kernel<false, false, true, false>,  general_tc_kernel<true, false, true, false>,
                                     general_tc_kernel<false, false, false, true>,  general_tc_kernel<true, false, false, true>,
                                     general_tc_kernel<false, false, true, true>,   general_tc_kernel<true, false, true, true>,
                                     general_tc_kernel<false, false, false, false, true>, general_tc_kernel<true, false, false, false, true>};
        for (auto k : all)
            if (cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemLimit) != cudaSuccess)
            return CONV2D_ERR_CUDA;
        attr_set = true;
    }
    KernelArgs a{};
    a.x = x; a.wp = wp; a.y = y; a.status = status;
    a.N = sh.N; a.C = sh.C; a.H = sh.H; a.W = sh.W; a.K = sh.K; a.P = sh.P; a.Q = sh.Q;
    a.patch_w = p.patch_w; a.patch_tw = p.patch_tw; a.patch_rows = p.patch_rows; a.patch_cols = p.patch_cols;
    a.row_pitch = p.patch_w ? p.patch_w : sh.W;
    a.pad_h = sh.pad_h; a.pad_w = sh.pad_w;
    a.fold_r = p.fold_r; a.fold_s = p.fold_s; a.R = sh.R / p.fold_r; a.S = sh.S / p.fold_s;
    a.HW = sh.H * sh.W;
    a.total_pix = sh.N * sh.H * sh.W;
    a.n_tile = p.n_tile; a.n_blocks = p.n_blocks; a.mt = p.mt; a.tile_px = p.tile_px; a.px_groups = p.px_groups; a.nbuf = p.nbuf; a.npix = p.npix; a.cstride = chunk_stride(p.npix);
    a.cblks = p.cblks; a.taps = p.taps;
    a.a_stages = p.a_stages; a.b_stages = p.b_stages; a.tps = p.tps;
    a.cbg = p.cbg; a.groups = (p.cblks + p.cbg - 1) / p.cbg; a.resident = p.resident; a.swap = p.swap;
    a.vec = 1;
    for (int v = 4; v >= 2; v >>= 1)       // v adjacent accumulator columns must be v adjacent, aligned outputs of one row
        if ((p.patch_w ? p.patch_tw : sh.W) % v == 0 && sh.Q % v == 0 && ((long long)sh.P * sh.Q) % v == 0 &&
            reinterpret_cast<uintptr_t>(y) % (4 * v) == 0) { a.vec = v; break; }
    a.vec_shift = a.vec == 4 ? 2 : (a.vec == 2 ? 1 : 0);
    a.pair_compact = p.pair_compact; a.cb_bytes = (int)p.cb_bytes;
    a.pair_taps = p.pair_taps; a.s_slots = p.s_slots; a.s_step = p.pair_taps ? 2 : 1; a.item_stride = p.tile_px - p.ovl;
    a.div_HW = FastDiv(a.HW); a.div_W = FastDiv(sh.W); a.div_npix = FastDiv(p.npix);
    a.div_qn = FastDiv(p.npix / 4 > 0 ? p.npix / 4 : 1); a.div_patch_w = FastDiv(p.patch_w ? p.patch_w : 1);
    a.xchg_slots = p.xchg_slots;
    a.xchg_bytes = (int)xchg_area_bytes(p.xchg_slots);
    // (the helper warps of the last item's write-back: measured no gain for the two-block cluster, whose single item
    // per block is short: 34.0 us without them, 35.4 us with them on 32 x 256 x 14 x 14 -> 256 maps)
    a.helpers = (p.swap && !p.cluster && (size_t)p.a_stages * p.cbg * kCB * chunk_stride(p.npix) * 4 >= 2 * kXposeBytes &&
                 env_int("CONV2D_B200_TF32_HELPERS", 1) != 0) ? 1 : 0;
    a.quad = ((p.patch_w ? (sh.W % 4 == 0 && sh.pad_w % 4 == 0) : (sh.H * sh.W) % 4 == 0) && p.fold_r * p.fold_s == 1 && env_int("CONV2D_B200_TF32_QUAD", 1) != 0) ? 1 : 0;
    {
        // as many producer groups as can each still cover a stage in one pass (one memory round trip)
        const long long per_pass = a.quad ? kProducers : (long long)kProducers * kUnitsPerThread;
        const long long stage_work = (long long)(a.quad ? p.npix / 4 : p.npix) * p.cbg;
        int g = 1;
        while (g < 4 && g * 2 <= p.a_stages && stage_work * (g * 2) <= per_pass) g *= 2;
        a.pgroups = env_int("CONV2D_B200_TF32_PGROUPS", g);
        if (a.pgroups != 1 && a.pgroups != 2 && a.pgroups != 4) a.pgroups = 1;
        while (a.pgroups > p.a_stages) a.pgroups /= 2;
    }
    a.fp16 = fp16 ? 1 : 0;
    a.pair = (b16 && (p.patch_w ? (sh.W % 2 == 0 && sh.pad_w % 2 == 0) : (sh.H * sh.W) % 2 == 0) && p.fold_r * p.fold_s == 1 && env_int("CONV2D_B200_B16_PAIR", 1) != 0) ? 1 : 0;
    a.items = p.supertiles * p.n_blocks * p.ksplit;
    a.ksplit = p.ksplit;
    a.div_ksplit = FastDiv(p.ksplit); a.div_n_blocks = FastDiv(p.n_blocks);
    a.div_groups_lo = FastDiv(a.groups / p.ksplit > 0 ? a.groups / p.ksplit : 1);
    a.div_groups_hi = FastDiv((a.groups + p.ksplit - 1) / p.ksplit);
    a.div_per_image = FastDiv(p.patch_w ? p.patch_rows * p.patch_cols : 1); a.div_patch_cols = FastDiv(p.patch_w ? p.patch_cols : 1);
    a.patch_item_rows = p.patch_w ? p.tile_px / p.patch_w : 0;
    // Failure-detection test hooks (host-side injection only): a short wait bound and one filter copy that is
    // never issued, so that a bounded wait expires and the time-out path can be checked without hanging anything.
    a.max_polls = (unsigned)env_int("CONV2D_B200_TF32_MAX_POLLS", 1 << 22);
    a.rot = env_int("CONV2D_B200_TF32_ROT", b16 ? 1 : 0) != 0 ? 1 : 0;
    a.test_drop_stage = env_int("CONV2D_B200_TF32_TEST_DROP_STAGE", -1);
    a.tmem_cols = (unsigned)p.tmem_cols;
    a.early_x = (!weights_packed && (p.ksplit == 1 || p.cluster) && env_int("CONV2D_B200_TF32_EARLY_X", 1) != 0) ? 1 : 0;
    if (p.ksplit > 1 && !p.cluster &&
        cudaMemsetAsync(y, 0, (size_t)sh.N * sh.K * sh.P * sh.Q * sizeof(float), stream) != cudaSuccess)
        return CONV2D_ERR_CUDA;
    // Programmatic dependent launch: the kernel's set-up (barriers, tensor-memory allocation) overlaps the
    // tail of whatever kernel precedes it on the stream; it waits for that kernel before it touches global memory.
    const bool fold = p.fold_r * p.fold_s > 1;
    void (*kernel)(KernelArgs);
    if (p.pair_taps && p.patch_w) kernel = b16 ? general_tc_kernel<true, false, true, true> : general_tc_kernel<false, false, true, true>;
    else if (p.pair_taps) kernel = b16 ? general_tc_kernel<true, false, false, true> : general_tc_kernel<false, false, false, true>;
    else if (p.patch_w) kernel = b16 ? general_tc_kernel<true, false, true, false> : general_tc_kernel<false, false, true, false>;
    else if (fold) kernel = b16 ? general_tc_kernel<true, true, false, false> : general_tc_kernel<false, true, false, false>;
    else kernel = b16 ? general_tc_kernel<true, false, false, false> : general_tc_kernel<false, false, false, false>;
    if (p.cluster) {
        kernel = b16 ? general_tc_kernel<true, false, false, false, true> : general_tc_kernel<false, false, false, false, true>;
        if (launch_pdl_cluster(kernel, dim3((unsigned)p.grid), dim3(kThreads), p.smem_bytes, stream, 2u, a) != cudaSuccess)
            return CONV2D_ERR_CUDA;
    } else if (launch_pdl(kernel, dim3((unsigned)p.grid), dim3(kThreads), p.smem_bytes, stream, a) != cudaSuccess) return CONV2D_ERR_CUDA;
    count_launch();
    return cudaGetLastError() == cudaSuccess ? CONV2D_OK : CONV2D_ERR_CUDA;
}
}  // namespace

conv2d_status_t launch_general_tf32(const float* x, const float* w, float* y, const Shape& sh,
                                    void* workspace, size_t workspace_bytes, bool weights_packed, cudaStream_t stream)
{
    return launch_tensor_core(x, w, y, sh, false, false, workspace, workspace_bytes, weights_packed, stream);
}

conv2d_status_t launch_general_b16(const void* x, const void* w, float* y, const Shape& sh, bool fp16,
                                   void* workspace, size_t workspace_bytes, bool weights_packed, cudaStream_t stream)
{
    return launch_tensor_core(x, w, y, sh, true, fp16, workspace, workspace_bytes, weights_packed, stream);
}

// ---------------------------------------------------------------- variant without caller-provided scratch
// Scratch of conv2d_fwd_general_noalloc: status block + re-ordered filters.  It lives in the module's
// device image, so every GPU that loads the library holds these bytes until the process exits.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocScratchBytes];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_noalloc_mu;
void* g_noalloc_scratch_of_device[kMaxDevices] = {};     // device address of the array, per device, once looked up
}  // namespace

// Reads the status word of the fixed array on the current device, if a call without caller scratch has run
// there (otherwise the word cannot be set and nothing is read).  The stream must already be idle.
cudaError_t noalloc_device_timeout(bool* raised)
{
    *raised = false;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return cudaSuccess;
    void* scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_noalloc_mu);
        scratch = g_noalloc_scratch_of_device[dev];
    }
    if (!scratch) return cudaSuccess;
    unsigned word = 0;
    const cudaError_t e = cudaMemcpy(&word, scratch, sizeof word, cudaMemcpyDeviceToHost);
    if (e == cudaSuccess) *raised = word != 0;
    return e;
}

conv2d_status_t launch_general_tf32_noalloc(const float* x, const float* w, float* y, const Shape& sh,
                                            bool wait, cudaStream_t stream)
{
    if (!tf32_supported(sh)) return CONV2D_ERR_UNSUPPORTED;
    if (tf32_workspace_bytes(sh) > kNoAllocScratchBytes) return CONV2D_ERR_WORKSPACE;

    // In host code the array's name is only a handle; the device address has to be asked for, once per
    // device, with that device current.
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return CONV2D_ERR_CUDA;
    void* scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_noalloc_mu);
        if (!g_noalloc_scratch_of_device[dev]) {
            void* p = nullptr;
            if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) return CONV2D_ERR_CUDA;
            g_noalloc_scratch_of_device[dev] = p;
        }
        scratch = g_noalloc_scratch_of_device[dev];
    }
    conv2d_status_t st = launch_general_tf32(x, w, y, sh, scratch, kNoAllocScratchBytes, /*weights_packed=*/false, stream);
    if (st != CONV2D_OK || !wait) return st;
    if (cudaStreamSynchronize(stream) != cudaSuccess) return CONV2D_ERR_CUDA;
    unsigned word = 0;
    if (cudaMemcpy(&word, scratch, sizeof word, cudaMemcpyDeviceToHost) != cudaSuccess) return CONV2D_ERR_CUDA;
    return word == 0 ? CONV2D_OK : CONV2D_ERR_DEVICE_TIMEOUT;
}

}  // namespace conv2d_b200
