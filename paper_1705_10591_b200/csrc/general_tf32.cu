// General case on the tcgen05 tensor cores: implicit-GEMM direct convolution, TF32 operands,
// fp32 accumulators in tensor memory (the contraction of Section 4, Algorithm 2).
//
// Mapping of the paper's design onto B200
//   * GEMM view: rows = output pixels, columns = filters, contraction over (channel, tap).
//     The accumulator block rAcc[F_T][W_T] of Algorithm 2 becomes a 128-pixel x n_tile-filter
//     fp32 tile in tensor memory; a thread block owns `mt` such tiles for adjacent pixels.
//   * Pixels are numbered in one flat sequence j = (n*H + h)*W + w over the whole batch.  For tap
//     (r,s) the input needed by output j is the pixel j + r*W + s of the same channel, a pure
//     shift.  A thread block therefore stages, per block of kCB channels, ONE run of
//     mt*128 + (R-1)*W + (S-1) pixels ("block plus halo to the right and below", Section 3.1/4.1)
//     and every tap reads it through a descriptor whose start address is shifted by r*W + s rows:
//     the row reuse of Section 4.2 (one staged input row serves all horizontal taps) extended to
//     the vertical taps, with no im2col buffer.  Outputs whose window wraps over the right or
//     bottom image edge are computed but not stored.
//   * Shared-memory operand layout: K-major, no swizzle: [channel/4][row][4 channels], i.e. each
//     row (pixel or filter) of a 4-channel chunk is one 16-byte unit and rows are 16 bytes apart.
//     This is the transposed staging of Fig. 6 (adjacent units belong to adjacent rows) in the
//     unit size the tensor core reads, and it is what makes a start address at any pixel legal.
//   * The filters are re-ordered once per call into exactly that layout in the workspace
//     ([filter block][channel block][tap][channel/4][filter][4], rounded to TF32) and streamed
//     with 1-D bulk (TMA) copies through an mbarrier ring.  Activations cannot be moved by TMA:
//     NCHW has the pixels, not the channels, contiguous, and a tiled copy cannot transpose nor
//     start at a 4-byte offset; eight producer warps gather them (coalesced along pixels),
//     round to TF32 and write 16-byte units.
//   * Warp roles: warp 0 streams filter chunks, warp 1 (one thread) issues tcgen05.mma and owns
//     the tensor-memory allocation, warps 2-9 stage activations and afterwards drain the
//     accumulators (lane = pixel, so the 32 lanes of a warp store 32 adjacent outputs of one map:
//     the coalesced write-back that Section 4.2 leaves out).
//   * Every wait is bounded; on expiry the block raises a flag, skips its stores, frees its tensor
//     memory and the status word in the workspace becomes non-zero.
#include <mutex>

#include "common.cuh"
#include "ptx.cuh"

namespace conv2d_b200 {
namespace {

using namespace ptx;

constexpr int kTileM = 128;                 // pixels per accumulator tile (UMMA M)
constexpr int kCB = 16;                     // channels per staged block (two UMMA K steps of 8)
constexpr int kChunks = kCB / 4;            // 16-byte channel chunks per block
constexpr int kProducerWarps = 8;
constexpr int kProducers = kProducerWarps * 32;
constexpr int kThreads = 64 + kProducers;   // warp 0: filter copies, warp 1: MMA issue, then the workers
constexpr int kMaxBStages = 8;
constexpr size_t kSmemLimit = 227 * 1024;

struct Plan {
    int n_tile;       // filters per thread block (UMMA N), multiple of 16
    int n_blocks;     // thread-block columns over the filters
    int mt;           // accumulator tiles per thread block
    int npix;         // staged pixel rows per channel chunk
    int cblks;        // channel blocks
    int taps;
    int b_stages;
    int tmem_cols;    // power of two >= 32
    int supertiles;   // thread-block rows over the flat pixel sequence
    size_t smem_bytes;
    bool ok;
};

size_t smem_need(int mt, int npix, int n_tile, int b_stages)
{
    (void)mt;
    return 2 * (size_t)kCB * npix * 4 + (size_t)b_stages * kCB * n_tile * 4 + 512;
}

Plan make_plan(const Shape& sh)
{
    Plan p{};
    p.ok = false;
    const long long total_pix = (long long)sh.N * sh.H * sh.W;
    if (total_pix >= (1LL << 31) - (1LL << 20)) return p;     // flat pixel indices stay within int32
    const int kp16 = (sh.K + 15) / 16 * 16;
    p.n_blocks = (kp16 + 255) / 256;
    p.n_tile = ((sh.K + p.n_blocks - 1) / p.n_blocks + 15) / 16 * 16;
    if (p.n_blocks > 65535) return p;
    p.cblks = (sh.C + kCB - 1) / kCB;
    p.taps = sh.R * sh.S;
    p.b_stages = 4;
    const long long halo = (long long)(sh.R - 1) * sh.W + (sh.S - 1);
    const long long tiles = (total_pix + kTileM - 1) / kTileM;
    int best_mt = 0;
    long long best_cost = 0;
    for (int mt = 4; mt >= 1; mt >>= 1) {
        if (mt * p.n_tile > 512) continue;
        const long long npix = ((long long)mt * kTileM + halo + 7) / 8 * 8;
        if (npix > 16000) continue;
        if (smem_need(mt, (int)npix, p.n_tile, p.b_stages) > kSmemLimit) continue;
        const long long ctas = (tiles + mt - 1) / mt * p.n_blocks;
        const long long waves = (ctas + 147) / 148;
        const long long cost = waves * mt;
        if (best_mt == 0 || cost < best_cost) { best_mt = mt; best_cost = cost; }
    }
    if (best_mt == 0) return p;
    p.mt = best_mt;
    p.npix = (int)(((long long)p.mt * kTileM + halo + 7) / 8 * 8);
    p.supertiles = (int)((tiles + p.mt - 1) / p.mt);
    int cols = p.mt * p.n_tile;
    p.tmem_cols = 32;
    while (p.tmem_cols < cols) p.tmem_cols <<= 1;
    p.smem_bytes = smem_need(p.mt, p.npix, p.n_tile, p.b_stages);
    p.ok = true;
    return p;
}

size_t packed_floats(const Shape& sh, const Plan& p)
{
    (void)sh;
    return (size_t)p.n_blocks * p.cblks * p.taps * kCB * p.n_tile;
}

// ---------------------------------------------------------------- filter re-ordering
// wp[nb][cb][t][chunk][f][e] = tf32(w[nb*n_tile + f][cb*kCB + 4*chunk + e][t]), zero outside K, C.
__global__ void repack_filters_kernel(const float* __restrict__ w, float* __restrict__ wp,
                                      int K, int C, int taps, int n_tile, int cblks, long long total)
{
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
        long long r = i;
        const int e = (int)(r % 4); r /= 4;
        const int f = (int)(r % n_tile); r /= n_tile;
        const int chunk = (int)(r % kChunks); r /= kChunks;
        const int t = (int)(r % taps); r /= taps;
        const int cb = (int)(r % cblks); r /= cblks;
        const int nb = (int)r;
        const int k = nb * n_tile + f, c = cb * kCB + 4 * chunk + e;
        float v = 0.f;
        if (k < K && c < C) v = to_tf32_rna(__ldg(w + ((size_t)k * C + c) * taps + t));
        wp[i] = v;
    }
}

struct KernelArgs {
    const float* x;
    const float* wp;
    float* y;
    unsigned* status;
    int N, C, H, W, K, R, S, P, Q;
    int HW;
    int total_pix;
    int n_tile, mt, npix, cblks, taps, b_stages;
    unsigned tmem_cols;
};

__global__ void __launch_bounds__(kThreads, 1)
general_tf32_kernel(const KernelArgs a)
{
    extern __shared__ __align__(128) unsigned char smem[];
    const uint32_t a_stage_bytes = (uint32_t)kCB * a.npix * 4;
    const uint32_t b_stage_bytes = (uint32_t)kCB * a.n_tile * 4;
    unsigned char* a_smem = smem;
    unsigned char* b_smem = smem + 2 * a_stage_bytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(b_smem + (size_t)a.b_stages * b_stage_bytes);
    uint64_t* a_full = bars;                 // [2]
    uint64_t* a_empty = bars + 2;            // [2]
    uint64_t* b_full = bars + 4;             // [kMaxBStages]
    uint64_t* b_empty = bars + 4 + kMaxBStages;
    uint64_t* acc_full = bars + 4 + 2 * kMaxBStages;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_full + 1);
    volatile uint32_t* abort_flag = tmem_slot + 1;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int nb = blockIdx.y;
    const int j0 = blockIdx.x * a.mt * kTileM;              // first flat pixel of this block

    if (tid == 0) {
        for (int i = 0; i < 2; ++i) { mbar_init(&a_full[i], kProducers); mbar_init(&a_empty[i], 1); }
        for (int i = 0; i < a.b_stages; ++i) { mbar_init(&b_full[i], 1); mbar_init(&b_empty[i], 1); }
        mbar_init(acc_full, 1);
        *abort_flag = 0;
        fence_mbar_init();
    }
    __syncthreads();
    if (warp == 1) { tmem_alloc(tmem_slot, a.tmem_cols); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = *tmem_slot;

    const int steps = a.cblks * a.taps;                     // filter chunks this block consumes

    if (warp == 0) {
        // ---------------- filter chunks: global -> shared by bulk copy, one chunk per (channel block, tap)
        if (lane == 0) {
            const unsigned char* src = reinterpret_cast<const unsigned char*>(a.wp) + (size_t)nb * steps * b_stage_bytes;
            int issued = 0;
            for (int it = 0; it < steps; ++it) {
                const int s = it % a.b_stages;
                const uint32_t ph = (uint32_t)(it / a.b_stages) & 1u;
                if (!mbar_wait_bounded(&b_empty[s], ph ^ 1u, abort_flag)) break;
                mbar_arrive_expect_tx(&b_full[s], b_stage_bytes);
                bulk_g2s(b_smem + (size_t)s * b_stage_bytes, src + (size_t)it * b_stage_bytes, b_stage_bytes, &b_full[s]);
                ++issued;
            }
            if (*abort_flag) {
                // let copies already in flight land before the block's shared memory is released
                const int pending = issued < a.b_stages ? issued : a.b_stages;
                for (int i = 0; i < pending; ++i) {
                    const int it = issued - 1 - i;
                    uint32_t dummy = 0;
                    mbar_wait_bounded(&b_full[it % a.b_stages], (uint32_t)(it / a.b_stages) & 1u, &dummy, 1u << 16);
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issue (one thread)
        if (lane == 0) {
            const uint32_t idesc = idesc_tf32(kTileM, (uint32_t)a.n_tile);
            const uint32_t a_lbo = (uint32_t)a.npix * 16u, b_lbo = (uint32_t)a.n_tile * 16u;
            int it = 0;
            bool alive = true;
            for (int cb = 0; cb < a.cblks && alive; ++cb) {
                const int as = cb & 1;
                if (!mbar_wait_bounded(&a_full[as], (uint32_t)(cb >> 1) & 1u, abort_flag)) { alive = false; break; }
                tc_fence_after_sync();
                const uint32_t a_base = smem_u32(a_smem + (size_t)as * a_stage_bytes);
                for (int t = 0; t < a.taps; ++t, ++it) {
                    const int bs = it % a.b_stages;
                    if (!mbar_wait_bounded(&b_full[bs], (uint32_t)(it / a.b_stages) & 1u, abort_flag)) { alive = false; break; }
                    tc_fence_after_sync();
                    const uint32_t b_base = smem_u32(b_smem + (size_t)bs * b_stage_bytes);
                    const int r = t / a.S, s = t - r * a.S;
                    const uint32_t shift = (uint32_t)(r * a.W + s);
                    for (int m = 0; m < a.mt; ++m) {
#pragma unroll
                        for (int j = 0; j < kCB / 8; ++j) {
                            const uint64_t ad = smem_desc_kmajor_noswizzle(
                                a_base + ((uint32_t)(2 * j) * a.npix + (uint32_t)m * kTileM + shift) * 16u, a_lbo, 128u);
                            const uint64_t bd = smem_desc_kmajor_noswizzle(
                                b_base + (uint32_t)(2 * j) * b_lbo, b_lbo, 128u);
                            mma_tf32(tmem + (uint32_t)(m * a.n_tile), ad, bd, idesc, (cb | t | j) != 0);
                        }
                    }
                    mma_commit(&b_empty[bs]);       // frees the filter stage when these MMAs have read it
                }
                if (alive) mma_commit(&a_empty[as]);
            }
            if (alive) mma_commit(acc_full);
        }
    } else {
        // ---------------- workers: stage activations, then drain the accumulators
        const int wtid = tid - 64;
        bool alive = true;
        for (int cb = 0; cb < a.cblks && alive; ++cb) {
            const int as = cb & 1;
            if (!mbar_wait_bounded(&a_empty[as], ((uint32_t)(cb >> 1) & 1u) ^ 1u, abort_flag)) { alive = false; break; }
            float4* dst = reinterpret_cast<float4*>(a_smem + (size_t)as * a_stage_bytes);
            const int c0 = cb * kCB;
            for (int jj = wtid; jj < a.npix; jj += kProducers) {
                const int j = j0 + jj;
                float v[kCB];
#pragma unroll
                for (int e = 0; e < kCB; ++e) v[e] = 0.f;
                if (j < a.total_pix) {
                    const int n = j / a.HW, off = j - n * a.HW;
                    const float* src = a.x + ((size_t)n * a.C + c0) * a.HW + off;
#pragma unroll
                    for (int e = 0; e < kCB; ++e)
                        if (c0 + e < a.C) v[e] = __ldg(src + (size_t)e * a.HW);
                }
#pragma unroll
                for (int ch = 0; ch < kChunks; ++ch)
                    dst[ch * a.npix + jj] = make_float4(to_tf32_rna(v[4 * ch]), to_tf32_rna(v[4 * ch + 1]),
                                                        to_tf32_rna(v[4 * ch + 2]), to_tf32_rna(v[4 * ch + 3]));
            }
            fence_proxy_async_smem();
            mbar_arrive(&a_full[as]);
        }

        // tcgen05.ld is warp-collective: take the decision for the whole warp
        if (__all_sync(0xffffffffu, alive && mbar_wait_bounded(acc_full, 0u, abort_flag))) {
            tc_fence_after_sync();
            const int quarter = warp & 3;                    // tensor-memory lanes this warp may read
            const int half = (warp - 2) >> 2;                // the two warps of a quarter split the columns
            const size_t plane = (size_t)a.P * a.Q;
            for (int m = 0; m < a.mt; ++m) {
                const int j = j0 + m * kTileM + quarter * 32 + lane;
                bool ok = j < a.total_pix;
                int n = 0, p = 0, q = 0;
                if (ok) {
                    n = j / a.HW;
                    const int off = j - n * a.HW;
                    p = off / a.W;
                    q = off - p * a.W;
                    ok = (p < a.P) && (q < a.Q);
                }
                float* yb = a.y + ((size_t)n * a.K * a.P + p) * a.Q + q;
                for (int chunk = half; chunk < a.n_tile / 16; chunk += 2) {
                    uint32_t v[16];
                    tmem_ld16(tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(m * a.n_tile + chunk * 16), v);
                    tmem_ld_wait();
                    const int k0 = nb * a.n_tile + chunk * 16;
                    if (ok) {
#pragma unroll
                        for (int i = 0; i < 16; ++i)
                            if (k0 + i < a.K) yb[(size_t)(k0 + i) * plane] = __uint_as_float(v[i]);
                    }
                }
            }
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, a.tmem_cols);
    if (tid == 0 && *abort_flag) atomicExch(a.status, 1u);
}

}  // namespace

bool tf32_supported(const Shape& sh)
{
    return make_plan(sh).ok;
}

size_t tf32_workspace_bytes(const Shape& sh)
{
    const Plan p = make_plan(sh);
    if (!p.ok) return kStatusBytes;
    return kStatusBytes + packed_floats(sh, p) * sizeof(float);
}

conv2d_status_t launch_general_tf32(const float* x, const float* w, float* y, const Shape& sh,
                                    void* workspace, bool weights_packed, cudaStream_t stream)
{
    const Plan p = make_plan(sh);
    if (!p.ok) return CONV2D_ERR_UNSUPPORTED;
    unsigned* status = static_cast<unsigned*>(workspace);
    float* wp = reinterpret_cast<float*>(static_cast<unsigned char*>(workspace) + kStatusBytes);
    if (cudaMemsetAsync(status, 0, kStatusBytes, stream) != cudaSuccess) return CONV2D_ERR_CUDA;

    if (!weights_packed) {
        const long long total = (long long)packed_floats(sh, p);
        long long blocks = (total + 255) / 256;
        if (blocks > 148 * 16) blocks = 148 * 16;
        repack_filters_kernel<<<(unsigned)blocks, 256, 0, stream>>>(w, wp, sh.K, sh.C, p.taps, p.n_tile, p.cblks, total);
        count_launch();
        if (cudaGetLastError() != cudaSuccess) return CONV2D_ERR_CUDA;
    }

    static bool attr_set = false;   // per process; the attribute is per function and device-wide
    if (!attr_set) {
        if (cudaFuncSetAttribute(general_tf32_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemLimit) != cudaSuccess)
            return CONV2D_ERR_CUDA;
        attr_set = true;
    }
    KernelArgs a{};
    a.x = x; a.wp = wp; a.y = y; a.status = status;
    a.N = sh.N; a.C = sh.C; a.H = sh.H; a.W = sh.W; a.K = sh.K; a.R = sh.R; a.S = sh.S; a.P = sh.P; a.Q = sh.Q;
    a.HW = sh.H * sh.W;
    a.total_pix = sh.N * sh.H * sh.W;
    a.n_tile = p.n_tile; a.mt = p.mt; a.npix = p.npix; a.cblks = p.cblks; a.taps = p.taps; a.b_stages = p.b_stages;
    a.tmem_cols = (unsigned)p.tmem_cols;
    dim3 grid((unsigned)p.supertiles, (unsigned)p.n_blocks, 1);
    general_tf32_kernel<<<grid, kThreads, p.smem_bytes, stream>>>(a);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? CONV2D_OK : CONV2D_ERR_CUDA;
}

// ---------------------------------------------------------------- variant without caller-provided scratch
// Scratch of conv2d_fwd_general_noalloc: status block + re-ordered filters.  It lives in the module's
// device image, so every GPU that loads the library holds these bytes until the process exits.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocScratchBytes];

conv2d_status_t launch_general_tf32_noalloc(const float* x, const float* w, float* y, const Shape& sh,
                                            bool wait, cudaStream_t stream)
{
    if (!tf32_supported(sh)) return CONV2D_ERR_UNSUPPORTED;
    if (tf32_workspace_bytes(sh) > kNoAllocScratchBytes) return CONV2D_ERR_WORKSPACE;

    // In host code the array's name is only a handle; the device address has to be asked for, once per
    // device, with that device current.
    constexpr int kMaxDevices = 64;
    static std::mutex mu;
    static void* scratch_of_device[kMaxDevices] = {};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return CONV2D_ERR_CUDA;
    void* scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(mu);
        if (!scratch_of_device[dev]) {
            void* p = nullptr;
            if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) return CONV2D_ERR_CUDA;
            scratch_of_device[dev] = p;
        }
        scratch = scratch_of_device[dev];
    }
    conv2d_status_t st = launch_general_tf32(x, w, y, sh, scratch, /*weights_packed=*/false, stream);
    if (st != CONV2D_OK || !wait) return st;
    if (cudaStreamSynchronize(stream) != cudaSuccess) return CONV2D_ERR_CUDA;
    unsigned word = 0;
    if (cudaMemcpy(&word, scratch, sizeof word, cudaMemcpyDeviceToHost) != cudaSuccess) return CONV2D_ERR_CUDA;
    return word == 0 ? CONV2D_OK : CONV2D_ERR_DEVICE_TIMEOUT;
}

}  // namespace conv2d_b200
