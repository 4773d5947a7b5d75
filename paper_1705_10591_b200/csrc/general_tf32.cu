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

// Cycle counter read that the compiler may not move across memory operations or barriers.
__device__ __forceinline__ long long clock_now()
{
    long long t;
    asm volatile("mov.u64 %0, %%clock64;" : "=l"(t) :: "memory");
    return t;
}

constexpr int kTileM = 128;                 // pixels per accumulator tile (UMMA M)
constexpr int kCB = 16;                     // channels per staged block (two UMMA K steps of 8)
constexpr int kChunks = kCB / 4;            // 16-byte channel chunks per block
constexpr int kProducerWarps = 8;
constexpr int kProducers = kProducerWarps * 32;
constexpr int kThreads = 64 + kProducers;   // warp 0: filter copies, warp 1: MMA issue, then the workers
constexpr int kMaxBStages = 16;
constexpr int kMaxAStages = 4;
constexpr int kUnitsPerThread = 3;           // (pixel, channel block) units a producer thread keeps in flight per pass
constexpr size_t kSmemLimit = 227 * 1024;
constexpr size_t kSmemLimitHalf = 113 * 1024;    // two blocks per SM

struct Plan {
    int n_tile;       // filters per thread block (UMMA N), multiple of 16
    int n_blocks;     // thread-block columns over the filters
    int mt;           // accumulator tiles per thread block
    int npix;         // staged pixel rows per channel chunk
    int cblks;        // channel blocks
    int taps;
    int a_stages;
    int b_stages;
    int tps;          // taps per filter stage
    int blocks_per_sm;
    int cbg;          // channel blocks per activation stage
    int tmem_cols;    // power of two >= 32
    int supertiles;   // thread-block rows over the flat pixel sequence
    size_t smem_bytes;
    bool ok;
};

// b_stages counts filter stages of `tps` taps each
size_t smem_need(int a_stages, int npix, int n_tile, int b_stages, int tps = 1, int cbg = 1)
{
    return (size_t)a_stages * cbg * kCB * npix * 4 + (size_t)b_stages * tps * kCB * n_tile * 4 + 512;
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
    p.b_stages = 2;
    p.tps = 1;
    const long long halo = (long long)(sh.R - 1) * sh.W + (sh.S - 1);
    const long long tiles = (total_pix + kTileM - 1) / kTileM;
    // Tiles per block.  Heavy tiles (many taps x channel blocks): as many as tensor memory holds, so a
    // streamed filter stage is reused by up to 4 tiles, picked to minimise (waves x tiles per block).
    // Light tiles (1x1-like): the block is dominated by memory latency and write-back, so small blocks,
    // two resident per SM, overlap one block's loads and stores with the other's MMAs.
    const bool light = (long long)p.taps * p.cblks <= 16;
    int best_mt = 0;
    long long best_cost = 0;
    for (int mt = 4; mt >= 1; mt >>= 1) {
        if (mt * p.n_tile > 512) continue;
        if (light && mt > 1 && (tiles + mt - 1) / mt * p.n_blocks < 4 * 148) continue;
        const long long npix = ((long long)mt * kTileM + halo + 7) / 8 * 8;
        if (npix > 16000) continue;
        if (smem_need(2, (int)npix, p.n_tile, 2) > kSmemLimit) continue;
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

    // Two blocks per SM when tensor memory (512 columns) and shared memory allow it.
    const int chunk = kCB * p.n_tile * 4;
    size_t limit = kSmemLimit;
    p.blocks_per_sm = 1;
    if (p.tmem_cols <= 256 && smem_need(2, p.npix, p.n_tile, 2, 1) <= kSmemLimitHalf &&
        (size_t)2 * chunk * (p.taps < 4 ? p.taps : 4) + (size_t)2 * kCB * p.npix * 4 + 512 <= kSmemLimitHalf) {
        p.blocks_per_sm = 2;
        limit = kSmemLimitHalf;
    }
    p.a_stages = 2;
    // Filter stages: several taps per stage (up to 32 KB) so that the single MMA-issuing thread pays its
    // per-stage bookkeeping (barrier wait, commit) once per 16-32 MMAs; the ring should hold 64-128 KB in
    // flight to cover the L2 latency.
    p.tps = 32 * 1024 / chunk;
    if (p.tps < 1) p.tps = 1;
    if (p.tps > p.taps) p.tps = p.taps;
    p.b_stages = 2;
    while (p.tps > 1 && smem_need(p.a_stages, p.npix, p.n_tile, 3, p.tps) > limit) --p.tps;
    while (p.b_stages < 4 && smem_need(p.a_stages, p.npix, p.n_tile, p.b_stages + 1, p.tps) <= limit) ++p.b_stages;
    // Light tiles: an activation stage carries several channel blocks, so that one producer pass has
    // 32-48 loads per thread in flight (the block is bound by memory latency, not by the MMAs).
    p.cbg = 1;
    if (light) {
        while (p.cbg * 2 <= p.cblks && p.npix * p.cbg * 2 <= kProducers * kUnitsPerThread &&
               smem_need(p.a_stages, p.npix, p.n_tile, p.b_stages, p.tps, p.cbg * 2) <= limit) p.cbg *= 2;
    }
    while (p.b_stages < kMaxBStages && smem_need(p.a_stages, p.npix, p.n_tile, p.b_stages + 1, p.tps, p.cbg) <= limit &&
           (size_t)p.b_stages * p.tps * chunk < 128 * 1024) ++p.b_stages;
    p.smem_bytes = smem_need(p.a_stages, p.npix, p.n_tile, p.b_stages, p.tps, p.cbg);
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
__global__ void repack_filters_kernel(const float* __restrict__ w, float* __restrict__ wp, unsigned* __restrict__ status,
                                      int K, int C, int taps, int n_tile, int cblks, long long total)
{
    // the status block in front of the filters starts every (non-prepacked) call cleared
    if (blockIdx.x == 0 && threadIdx.x < kStatusBytes / sizeof(unsigned)) status[threadIdx.x] = 0u;
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
    int n_tile, mt, npix, cblks, taps, a_stages, b_stages, tps;
    int cbg, groups;        // channel blocks per activation stage, number of such groups
    unsigned tmem_cols;
};

// Producer helpers.  A stage holds `cbg` channel blocks of kCB channels for npix pixels, laid out
// [channel block][chunk][pixel] in 16-byte units.  A work unit is (channel block g, pixel jj), numbered
// i = g * npix + jj; thread t of the 256 producers owns units first + t, first + t + 256, ...  Consecutive
// lanes read consecutive pixels of one channel (coalesced) and write consecutive 16-byte units.
template <int CNT>
__device__ __forceinline__ void load_units(float (&v)[CNT][kCB], const KernelArgs& a, int j0, int cb0, int first, int wtid)
{
    const int units = a.npix * a.cbg;
#pragma unroll
    for (int u = 0; u < CNT; ++u) {
        const int i = first + u * kProducers + wtid;
#pragma unroll
        for (int e = 0; e < kCB; ++e) v[u][e] = 0.f;
        if (i < units) {
            const int g = i / a.npix, jj = i - g * a.npix;
            const int j = j0 + jj;
            const int c0 = (cb0 + g) * kCB;
            if (j < a.total_pix && c0 < a.C) {
                const int n = j / a.HW, off = j - n * a.HW;
                const float* src = a.x + ((size_t)n * a.C + c0) * a.HW + off;
#pragma unroll
                for (int e = 0; e < kCB; ++e)
                    if (c0 + e < a.C) v[u][e] = __ldg(src + (size_t)e * a.HW);
            }
        }
    }
}

template <int CNT>
__device__ __forceinline__ void store_units(const float (&v)[CNT][kCB], float4* dst, const KernelArgs& a, int first, int wtid)
{
    const int units = a.npix * a.cbg;
#pragma unroll
    for (int u = 0; u < CNT; ++u) {
        const int i = first + u * kProducers + wtid;
        if (i < units) {
            const int g = i / a.npix, jj = i - g * a.npix;
            float4* d = dst + (size_t)g * kChunks * a.npix + jj;
#pragma unroll
            for (int ch = 0; ch < kChunks; ++ch)
                d[ch * a.npix] = make_float4(to_tf32_rna(v[u][4 * ch]), to_tf32_rna(v[u][4 * ch + 1]),
                                             to_tf32_rna(v[u][4 * ch + 2]), to_tf32_rna(v[u][4 * ch + 3]));
        }
    }
}

__global__ void __launch_bounds__(kThreads, 2)
general_tf32_kernel(const KernelArgs a)
{
    extern __shared__ __align__(128) unsigned char smem[];
    const uint32_t a_block_bytes = (uint32_t)kCB * a.npix * 4;          // one channel block of a stage
    const uint32_t a_stage_bytes = a_block_bytes * (uint32_t)a.cbg;
    const uint32_t b_chunk_bytes = (uint32_t)kCB * a.n_tile * 4;     // one (channel block, tap)
    const uint32_t b_stage_bytes = b_chunk_bytes * (uint32_t)a.tps;
    unsigned char* a_smem = smem;
    unsigned char* b_smem = smem + (size_t)a.a_stages * a_stage_bytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(b_smem + (size_t)a.b_stages * b_stage_bytes);
    uint64_t* a_full = bars;                 // [kMaxAStages]
    uint64_t* a_empty = bars + kMaxAStages;  // [kMaxAStages]
    uint64_t* b_full = bars + 2 * kMaxAStages;             // [kMaxBStages]
    uint64_t* b_empty = b_full + kMaxBStages;
    uint64_t* acc_full = b_empty + kMaxBStages;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_full + 1);
    volatile uint32_t* abort_flag = tmem_slot + 1;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const long long t_entry = clock_now();
    const int nb = blockIdx.y;
    const int j0 = blockIdx.x * a.mt * kTileM;              // first flat pixel of this block

    if (tid == 0) {
        for (int i = 0; i < a.a_stages; ++i) { mbar_init(&a_full[i], kProducers); mbar_init(&a_empty[i], 1); }
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
    const int grp_first = (int)(blockIdx.x % (unsigned)a.groups);  // channel-block group this block starts with

    if (warp == 0) {
        // ---------------- filters: global -> shared by bulk copy, up to `tps` taps of one channel block per stage
        if (lane == 0) {
            const unsigned char* src = reinterpret_cast<const unsigned char*>(a.wp) + (size_t)nb * steps * b_chunk_bytes;
            int s = 0, issued = 0;
            uint32_t ph = 0;
            bool alive = true;
            // Blocks start at different channel-block groups (grp_first), so that at any moment they stream
            // different parts of the filter bank.  Order: groups rotated, channel blocks inside a group
            // ascending, taps ascending -- the order in which the MMA thread consumes them.
            for (int grp = 0; grp < a.groups && alive; ++grp) {
                int gr = grp + grp_first;
                if (gr >= a.groups) gr -= a.groups;
                for (int g = 0; g < a.cbg && alive; ++g) {
                    const int cbr = gr * a.cbg + g;
                    if (cbr >= a.cblks) break;
                    for (int t0 = 0; t0 < a.taps; t0 += a.tps) {
                        const int nt = min(a.tps, a.taps - t0);
                        if (!mbar_wait_bounded(&b_empty[s], ph ^ 1u, abort_flag)) { alive = false; break; }
                        const uint32_t bytes = b_chunk_bytes * (uint32_t)nt;
                        mbar_arrive_expect_tx(&b_full[s], bytes);
                        bulk_g2s(b_smem + (size_t)s * b_stage_bytes, src + ((size_t)cbr * a.taps + t0) * b_chunk_bytes, bytes, &b_full[s]);
                        ++issued;
                        if (++s == a.b_stages) { s = 0; ph ^= 1u; }
                    }
                }
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
            // Per MMA this thread only adds small constants to the low word of a descriptor: everything
            // that does not change is folded into a_lo_fixed / b_lo_fixed / desc_hi beforehand, because a
            // single thread issuing ~40 dependent integer instructions per MMA was slower than the MMA.
            const uint32_t idesc = idesc_tf32(kTileM, (uint32_t)a.n_tile);
            const uint32_t desc_hi = (128u >> 4) | (1u << 14);                  // SBO = 128 B, descriptor version 1
            const uint32_t a_lo_fixed = ((uint32_t)a.npix & 0x3FFFu) << 16;     // LBO = npix * 16 B
            const uint32_t b_lo_fixed = ((uint32_t)a.n_tile & 0x3FFFu) << 16;   // LBO = n_tile * 16 B
            const uint32_t a_kstep = 2u * (uint32_t)a.npix;                     // 8 channels further, in 16-byte units
            const uint32_t b_kstep = 2u * (uint32_t)a.n_tile;
            bool alive = true;
            long long t_first_mma = 0, wait_a = 0, wait_b = 0;   // diagnostics: operand-wait cycles of this thread
            int as = 0, bs = 0;
            uint32_t a_phase = 0, b_phase = 0, accumulate = 0;
            for (int grp = 0; grp < a.groups && alive; ++grp) {
                long long tw = clock_now();
                if (!mbar_wait_bounded(&a_full[as], a_phase, abort_flag)) { alive = false; break; }
                tc_fence_after_sync();
                wait_a += clock_now() - tw;
                if (grp == 0) t_first_mma = clock_now();
                int gr = grp + grp_first;
                if (gr >= a.groups) gr -= a.groups;
                uint32_t a_lo_block = a_lo_fixed | (smem_u32(a_smem + (size_t)as * a_stage_bytes) >> 4);
                for (int g = 0; g < a.cbg && alive; ++g, a_lo_block += a_block_bytes >> 4) {
                    if (gr * a.cbg + g >= a.cblks) break;
                    uint32_t row_shift = 0;                                      // r * W, in pixels (= 16-byte units)
                    int sx = 0;
                    for (int t0 = 0; t0 < a.taps; t0 += a.tps) {
                        const int nt = min(a.tps, a.taps - t0);
                        tw = clock_now();
                        if (!mbar_wait_bounded(&b_full[bs], b_phase, abort_flag)) { alive = false; break; }
                        tc_fence_after_sync();
                        wait_b += clock_now() - tw;
                        uint32_t b_lo = b_lo_fixed | (smem_u32(b_smem + (size_t)bs * b_stage_bytes) >> 4);
                        for (int t = 0; t < nt; ++t, b_lo += b_chunk_bytes >> 4) {
                            uint32_t a_lo = a_lo_block + row_shift + (uint32_t)sx;
                            uint32_t d = tmem;
                            for (int m = 0; m < a.mt; ++m, a_lo += kTileM, d += (uint32_t)a.n_tile) {
                                mma_tf32(d, ((uint64_t)desc_hi << 32) | a_lo, ((uint64_t)desc_hi << 32) | b_lo, idesc, accumulate != 0);
                                mma_tf32(d, ((uint64_t)desc_hi << 32) | (a_lo + a_kstep), ((uint64_t)desc_hi << 32) | (b_lo + b_kstep), idesc, true);
                            }
                            accumulate = 1;
                            if (++sx == a.S) { sx = 0; row_shift += (uint32_t)a.W; }
                        }
                        mma_commit(&b_empty[bs]);   // frees the filter stage when these MMAs have read it
                        if (++bs == a.b_stages) { bs = 0; b_phase ^= 1u; }
                    }
                }
                if (alive) mma_commit(&a_empty[as]);
                if (++as == a.a_stages) { as = 0; a_phase ^= 1u; }
            }
            if (alive) mma_commit(acc_full);
            if (blockIdx.x == 0 && blockIdx.y == 0) {
                // diagnostic time stamps of block (0,0), cycles since kernel entry: status words 2, 3
                a.status[2] = (unsigned)(t_first_mma - t_entry);
                a.status[3] = (unsigned)(clock_now() - t_entry);
                a.status[7] = (unsigned)wait_a;
                a.status[8] = (unsigned)wait_b;
            }
        }
    } else {
        // ---------------- workers: stage activations, then drain the accumulators
        const int wtid = tid - 64;
        bool alive = true;
        int as = 0;
        uint32_t a_phase = 0;
        // One stage = cbg consecutive channel blocks.  All loads of a pass (kUnitsPerThread units of 16
        // channels per thread) are issued before its first store, so a pass costs one memory round trip.
        const int units = a.npix * a.cbg;
        for (int grp = 0; grp < a.groups && alive; ++grp) {
            if (!mbar_wait_bounded(&a_empty[as], a_phase ^ 1u, abort_flag)) { alive = false; break; }
            float4* dst = reinterpret_cast<float4*>(a_smem + (size_t)as * a_stage_bytes);
            int gr = grp + grp_first;
            if (gr >= a.groups) gr -= a.groups;
            for (int first = 0; first < units; first += kProducers * kUnitsPerThread) {
                float v[kUnitsPerThread][kCB];
                load_units(v, a, j0, gr * a.cbg, first, wtid);
                store_units(v, dst, a, first, wtid);
            }
            fence_proxy_async_smem();
            mbar_arrive(&a_full[as]);
            if (++as == a.a_stages) { as = 0; a_phase ^= 1u; }
        }

        // tcgen05.ld is warp-collective: take the decision for the whole warp
        if (__all_sync(0xffffffffu, alive && mbar_wait_bounded(acc_full, 0u, abort_flag))) {
            tc_fence_after_sync();
            if (tid == 64 && blockIdx.x == 0 && blockIdx.y == 0) a.status[4] = (unsigned)(clock_now() - t_entry);
            const int quarter = warp & 3;                    // tensor-memory lanes this warp may read
            const int half = (warp - 2) >> 2;                // the two warps of a quarter split the columns
            const size_t plane = (size_t)a.P * a.Q;
            const int chunks_per_tile = a.n_tile / 16;
            const int total_chunks = a.mt * chunks_per_tile;
            const uint32_t lane_base = tmem + ((uint32_t)(quarter * 32) << 16);
            int cur_m = -1;
            bool ok = false;
            float* yb = a.y;
            // Issues the tensor-memory load of 16-column chunk c (chunks are numbered tile-major).
            auto load_chunk = [&](uint32_t (&v)[16], int c) {
                const int m = c / chunks_per_tile, ch = c - m * chunks_per_tile;
                tmem_ld16(lane_base + (uint32_t)(m * a.n_tile + ch * 16), v);
            };
            // Stores chunk c: this lane's pixel of 16 adjacent maps (the warp writes 32 adjacent pixels per map).
            auto store_chunk = [&](const uint32_t (&v)[16], int c) {
                const int m = c / chunks_per_tile, ch = c - m * chunks_per_tile;
                if (m != cur_m) {
                    cur_m = m;
                    const int j = j0 + m * kTileM + quarter * 32 + lane;
                    ok = j < a.total_pix;
                    if (ok) {
                        const int n = j / a.HW, off = j - n * a.HW;
                        const int p = off / a.W, q = off - p * a.W;
                        ok = (p < a.P) && (q < a.Q);
                        yb = a.y + ((size_t)n * a.K * a.P + p) * a.Q + q;
                    }
                }
                const int k0 = nb * a.n_tile + ch * 16;
                if (ok) {
                    float* o = yb + (size_t)k0 * plane;
#pragma unroll
                    for (int i = 0; i < 16; ++i, o += plane)
                        if (k0 + i < a.K) *o = __uint_as_float(v[i]);
                }
            };
            // Two register buffers: the load of the next chunk is in flight while the current one is stored.
            uint32_t va[16], vb[16];
            int c = half;
            if (c < total_chunks) load_chunk(va, c);
            while (c < total_chunks) {
                tmem_ld_wait();
                if (c + 2 < total_chunks) load_chunk(vb, c + 2);
                store_chunk(va, c);
                c += 2;
                if (c >= total_chunks) break;
                tmem_ld_wait();
                if (c + 2 < total_chunks) load_chunk(va, c + 2);
                store_chunk(vb, c);
                c += 2;
            }
            if (tid == 64 && blockIdx.x == 0 && blockIdx.y == 0) a.status[6] = (unsigned)(clock_now() - t_entry);
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (tid == 0 && blockIdx.x == 0 && blockIdx.y == 0) a.status[5] = (unsigned)(clock_now() - t_entry);
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

    if (!weights_packed) {
        const long long total = (long long)packed_floats(sh, p);
        long long blocks = (total + 255) / 256;
        if (blocks > 148 * 16) blocks = 148 * 16;
        repack_filters_kernel<<<(unsigned)blocks, 256, 0, stream>>>(w, wp, status, sh.K, sh.C, p.taps, p.n_tile, p.cblks, total);
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
    a.n_tile = p.n_tile; a.mt = p.mt; a.npix = p.npix; a.cblks = p.cblks; a.taps = p.taps;
    a.a_stages = p.a_stages; a.b_stages = p.b_stages; a.tps = p.tps;
    a.cbg = p.cbg; a.groups = (p.cblks + p.cbg - 1) / p.cbg;
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
