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
#include <cstdlib>
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
static_assert(kProducers == 256, "the producer group arithmetic assumes 256 producer threads");
constexpr int kEpilogueWarps = 4;
// Warp roles by warp index.  An SM has four warp schedulers and warp w is served by scheduler w % 4.  The
// single thread that issues the MMAs (warp 1) must never wait for an issue slot behind arithmetic-heavy
// warps -- measured: sharing its scheduler with two producer warps stretched each MMA issue from ~64 to
// 120-180 cycles -- so scheduler 1 hosts only that warp, one epilogue warp and two warps that only wait.
//   warp 0           filter copies (one thread)
//   warp 1           MMA issue (one thread), owner of the tensor-memory allocation
//   warps 4-7        epilogue, tensor-memory lane quarter = warp % 4
//   warps 2,3,8,10,11,12,14,15   activation producers (schedulers 0, 2, 3)
//   warps 9, 13      no work until the block's last item
//   warps 8-15       help to drain the block's last item once their own work is done (quarter = warp % 4)
constexpr int kThreads = 512;
__device__ __forceinline__ int producer_index(int warp)     // 0..7 for producer warps, -1 otherwise
{
    switch (warp) {
        case 2: return 0; case 3: return 1; case 8: return 2; case 10: return 3;
        case 11: return 4; case 12: return 5; case 14: return 6; case 15: return 7;
        default: return -1;
    }
}
constexpr int kMaxBStages = 16;
constexpr int kMaxAStages = 4;
constexpr int kUnitsPerThread = 3;          // (pixel, channel block) units a producer thread keeps in flight per pass
constexpr size_t kSmemLimit = 227 * 1024;
constexpr int kMaxTaps = 256;                // taps left as descriptor shifts (after folding)
constexpr size_t kBookBytes = 512 + kMaxTaps * 4;    // barriers, tensor-memory slot, flags + the table of tap shifts
constexpr int kXposePitch = 36;             // floats per row of the epilogue's transposition tile (16-byte aligned, conflict-free)
constexpr size_t kXposeBytes = (size_t)kEpilogueWarps * 32 * kXposePitch * 4;

struct Plan {
    int n_tile;       // filters per work item: 64 or 128 rows of the M operand (with the pixels as M: UMMA N, a multiple of 16)
    int n_blocks;     // work-item columns over the filters
    int mt;           // accumulator tiles per work item (pixels-as-M layout; informative otherwise)
    int tile_px;      // pixels per work item: mt * 128, or any multiple of 32 up to 512 in the operand-swap layout
    int px_groups;    // operand-swap layout: MMAs per K step (each covers n_mma = tile_px / px_groups pixels)
    int nbuf;         // accumulator sets in tensor memory (2: write-back overlaps the next item)
    int npix;         // staged pixel rows per channel chunk
    int cblks;        // channel blocks (of the folded channels, see fold_r/fold_s)
    int fold_r, fold_s;  // taps folded into the channel dimension: 1 or R rows, 1 or S columns
    int patch_w, patch_tw, patch_rows, patch_cols;   // patch addressing (patch_w = 0: flat pixel run), see ItemGeom
    int taps;
    int a_stages;
    int b_stages;
    int tps;          // taps per filter stage
    int cbg;          // channel blocks per activation stage
    int resident;     // 1: the whole filter block stays in shared memory for the life of the thread block
    int swap;         // 1: filters are the MMA's M operand, 256 pixels its N operand (K <= 128)
    int pair_taps;    // 1: at most 64 filters, horizontally adjacent taps stacked in one M = 128 operand (see make_plan)
    int s_slots;      // shift-table entries per filter row: S, or ceil(S / 2) with stacked taps
    int ovl;          // pixels by which consecutive flat items overlap (4 with stacked taps, else 0)
    int ksplit;       // 2: the channel blocks of a tile are shared by two work items that add into y
    int tmem_cols;    // power of two >= 32
    int supertiles;   // work-item rows over the flat pixel sequence
    int grid;
    size_t smem_bytes;
    bool ok;
};

// Distance between the 4-channel chunks of a staged channel block, in 16-byte units: the pixel count plus one, so
// that it is odd.  A producer lane writes four adjacent pixels (64 bytes) per chunk; with lanes 64 bytes apart a
// 128-bit store instruction would hit only two of the eight 16-byte bank groups (4-way conflict, ~1 M conflict
// cycles per launch in the profiles).  With an odd chunk stride, lanes that would collide write different chunks
// at the same time (each lane rotates its chunk order), and the eight lanes of a store phase cover all banks.
inline int chunk_stride(int npix) { return npix + 1; }

// b_stages counts filter stages of `tps` taps each; an activation stage holds `cbg` channel blocks.
size_t smem_need(int a_stages, int npix, int n_tile, int b_stages, int tps, int cbg)
{
    return (size_t)a_stages * cbg * kCB * chunk_stride(npix) * 4 + (size_t)b_stages * tps * kCB * n_tile * 4 + kBookBytes;
}

// b16: the operands are 16-bit floats, bf16 or fp16 (16-byte unit = 8 channels, 32 channels per staged block, K = 16 per MMA); the
// byte layout of every stage is the same as for TF32 (16 channels of 4 bytes).
Plan make_plan(const Shape& sh, bool b16 = false)
{
    Plan p{};
    p.ok = false;
    const long long total_pix = (long long)sh.N * sh.H * sh.W;
    if (total_pix >= (1LL << 31) - (1LL << 20)) return p;     // flat pixel indices stay within int32
    const int kp16 = (sh.K + 15) / 16 * 16;
    p.n_blocks = (kp16 + 255) / 256;
    p.n_tile = ((sh.K + p.n_blocks - 1) / p.n_blocks + 15) / 16 * 16;
    // Operand roles.  One tcgen05.mma costs its issuing thread ~60 cycles whatever its size (measured), so
    // an instruction must carry >= 128 cycles of tensor-pipe work to keep the pipe busy: N = 256.  For any
    // filter count that is possible with the pixels as the N operand: M = a block of 128 filters (zero
    // padded), N = 256 pixels, accumulator lanes = filters.  It also halves the filter bytes an item streams
    // per pixel compared with 128 pixels x 256 filters.
    // Up to 64 filters use M = 64 (one tcgen05.mma then covers 64 filters x 256 pixels; its accumulator
    // occupies lanes 0-15 of each 32-lane quarter -- established with a probe).
    p.swap = env_int("CONV2D_B200_TF32_SWAP", 1) != 0 ? 1 : 0;
    if (p.swap && kp16 <= 64 && env_int("CONV2D_B200_TF32_M64", 1) == 0) p.swap = 0;
    if (p.swap) {
        p.n_tile = kp16 <= 64 ? 64 : 128;                  // filters per block = rows of the M operand
        p.n_blocks = (kp16 + p.n_tile - 1) / p.n_tile;
    }
    const int set_cols = p.swap ? kTileM : p.n_tile;      // tensor-memory columns of one 128-pixel tile
    const int cbc = b16 ? 2 * kCB : kCB;                 // channels per staged block
    // Few input channels (first layers, the bridge between the one-channel and the many-channel case) would
    // leave most of a staged channel block as zero padding.  Then taps are folded into the channel dimension:
    // "channel" (c, r, s) of pixel j is x[c] at pixel j + r*W + s, so the contraction runs over C*fold_r*fold_s
    // channels and only the remaining R/fold_r x S/fold_s taps are descriptor shifts.  The fold with the
    // fewest MMAs (remaining taps x channel blocks) wins; ties keep more taps as shifts (fewer loads).
    // Every folded tap multiplies the producers' loads, so by default only 1-3 channels are folded (measured:
    // 3 channels 7 x 7 on 224 x 224: 0.91 ms folded, 1.06 ms not; 1 channel 5 x 5: 0.32 vs 0.40 ms; but
    // 8 channels 3 x 3 on 112 x 112: 0.175 vs 0.093 ms).  CONV2D_B200_TF32_FOLD = 2 folds whenever C < 16.
    p.fold_r = p.fold_s = 1;
    const bool padded = sh.pad_h != 0 || sh.pad_w != 0;      // needs patch addressing: no folding, filters as M
    if (padded && !p.swap) return p;
    const int fold_mode = padded ? 0 : env_int("CONV2D_B200_TF32_FOLD", 1);
    if (sh.C < cbc && (fold_mode == 2 || (fold_mode == 1 && sh.C <= 3))) {
        long long best = (long long)sh.R * sh.S * ((sh.C + cbc - 1) / cbc);
        const int cand[3][2] = {{1, sh.S}, {sh.R, 1}, {sh.R, sh.S}};
        for (const auto& f : cand) {
            const long long ceff = (long long)sh.C * f[0] * f[1];
            if (ceff > 4096) continue;
            const long long mmas = (long long)(sh.R / f[0]) * (sh.S / f[1]) * ((ceff + cbc - 1) / cbc);
            if (mmas < best) { best = mmas; p.fold_r = f[0]; p.fold_s = f[1]; }
        }
    }
    const int c_eff = sh.C * p.fold_r * p.fold_s;
    const int r_eff = sh.R / p.fold_r, s_eff = sh.S / p.fold_s;
    p.cblks = (c_eff + cbc - 1) / cbc;
    // Stacked taps.  With at most 64 filters an M = 64 instruction runs the tensor pipe at half its rate.  Instead
    // half of the rows of an M = 128 operand hold the filters' tap (r, s) and the other half their tap (r, s + 1),
    // both multiplied with the pixels shifted for (r, s): the accumulator row of tap (r, s + 1), column j + 1, then
    // holds what that tap contributes to output j, and the epilogue adds the two rows of a map one column apart
    // (rows are ordered so that both lie in the lane quarter of one epilogue warp).  A row of
    // S taps takes ceil(S / 2) instructions instead of S (an odd last tap has zeros in the upper half).  In the
    // flat pixel run the last column of an item has no right neighbour, so consecutive items overlap by 4 pixels.
    // It pays when the MMAs dominate an item: the stacked operand doubles the filter bytes per instruction (a bank
    // that was resident in shared memory may have to be streamed) and every block of the write-back reads two tile
    // rows per map.  Measured with 64 filters: 128 channels 5 x 5 on 32 x 32: 63.9 -> 46.8 us, 7 x 7: 110.5 ->
    // 74.4 us, 3 x 3: 31.7 -> 28.6 us; 64 channels 5 x 5 on 64 x 64 in bf16 (50 pairs of tap and channel block):
    // 24.3 -> 20.8 us; 64 channels 3 x 3 on 56 x 56 (36 pairs): 27.6 -> 30.6 us.  Hence from 48 (tap, channel block)
    // pairs on.  CONV2D_B200_TF32_PAIR_TAPS = 0 / 2: never / whenever possible.
    const int pair_mode = env_int("CONV2D_B200_TF32_PAIR_TAPS", 1);
    p.pair_taps = (p.swap && kp16 <= 64 && p.fold_r * p.fold_s == 1 && s_eff >= 2 && pair_mode != 0 &&
                   (pair_mode == 2 || (long long)r_eff * s_eff * p.cblks >= 48)) ? 1 : 0;
    if (p.pair_taps) p.n_tile = 128;
    p.s_slots = p.pair_taps ? (s_eff + 1) / 2 : s_eff;
    p.taps = r_eff * p.s_slots;
    if (p.taps > kMaxTaps) return p;
    const size_t extra = p.swap ? kXposeBytes : 0;       // epilogue transposition tile
    // Addressing mode.  In the flat pixel run the staged halo is (R-1) whole image rows; once that exceeds a
    // 256-pixel item the item is cut as a rectangle of the image instead (patch_w columns wide, of which the
    // first patch_tw produce outputs), whose halo is (R-1) patch rows.  The patch width with the least staged
    // pixels per output wins.
    p.patch_w = p.patch_tw = p.patch_rows = p.patch_cols = 0;
    const long long flat_halo = (long long)(r_eff - 1) * sh.W + (s_eff - 1);
    const int patch_mode = padded ? 2 : env_int("CONV2D_B200_TF32_PATCH", 1);       // 0 never, 1 when the flat halo is large, 2 always
    if (p.swap && p.fold_r * p.fold_s == 1 && patch_mode != 0) {
        double best_ratio = 0;
        for (int wp = 32; wp <= 128; wp *= 2) {
            const int tw = (wp - (s_eff - 1)) / 4 * 4;
            if (tw < 4) continue;
            const int th = 448 / wp > 0 ? 448 / wp : 1;                       // rows of a typical item
            const long long rows_p = (sh.P + th - 1) / th, cols_p = (sh.Q + tw - 1) / tw;
            const double ratio = (double)(rows_p * (th + r_eff - 1)) * wp * cols_p / ((double)sh.P * sh.Q);
            if (p.patch_w == 0 || ratio < best_ratio) { best_ratio = ratio; p.patch_w = wp; p.patch_tw = tw; }
        }
        // staged pixels per output of the flat run, for a 448-pixel item.  Patches also cost extra work items at
        // the ragged right edge and a narrower store run, so they must win clearly (measured: 3 x 3 on 224 x 224,
        // ratio 2.0 flat vs 1.3 in patches, is 10 % faster flat; 3 x 3 on 512 x 512, 3.3 vs 1.3, 20 % faster in patches;
        // 7 x 7 on 224 x 224, 4.2 vs 2.2, 20 % faster in patches).
        const double flat_ratio = (448.0 + flat_halo) / 448.0 * ((double)sh.H * sh.W) / ((double)sh.P * sh.Q);
        if (patch_mode == 1 && !(flat_ratio > 1.75 * best_ratio)) p.patch_w = p.patch_tw = 0;
        if (p.patch_w) p.patch_cols = (sh.Q + p.patch_tw - 1) / p.patch_tw;
    }
    if (padded && !p.patch_w) return p;
    p.ovl = (p.pair_taps && !p.patch_w) ? 4 : 0;
    const long long halo = p.patch_w ? (long long)(r_eff - 1) * p.patch_w + (s_eff - 1) : flat_halo;
    // work items along the pixels for an item of px pixels (0: px is not possible in this mode)
    auto pixel_items = [&](int px) -> long long {
        if (!p.patch_w) return px > p.ovl ? (total_pix + (px - p.ovl) - 1) / (px - p.ovl) : 0;
        if (px % p.patch_w) return 0;
        const int th = px / p.patch_w;
        return (long long)sh.N * ((sh.P + th - 1) / th) * p.patch_cols;
    };
    const long long tiles = (total_pix + kTileM - 1) / kTileM;
    const int chunk = kCB * p.n_tile * 4;
    const int sms = 148;

    const int forced_mt = env_int("CONV2D_B200_TF32_MT", 0);      // benchmark ablations only
    const size_t wbytes = (size_t)p.cblks * p.taps * chunk;        // re-ordered filters of one filter block
    auto npix_of = [&](int tile_px) { return (int)(((long long)tile_px + halo + 7) / 8 * 8); };

    // Light problems (1x1-like: few taps x channel blocks) with a small filter bank keep it resident in
    // shared memory: nothing is streamed, items are small (finest balance over the SMs, two accumulator
    // sets), and the rest of shared memory becomes a deep activation ring whose stages carry several
    // channel blocks (these items are bound by memory latency: one producer pass should have 32-48 loads
    // per thread in flight).  Any other bank that fits next to a two-stage activation ring is kept resident too
    // (64 filters of 64 x 3 x 3: 39 us resident vs 43 us streamed).
    p.resident = 0;
    const int resident_mode = env_int("CONV2D_B200_TF32_RESIDENT", 2);      // 0 never, 1 light problems only, 2 whenever it fits
    if (resident_mode != 0 && p.n_blocks == 1 && wbytes <= 152 * 1024 &&
        ((long long)p.taps * p.cblks <= 16 || resident_mode == 2)) {
        const int mt = forced_mt ? forced_mt : (p.swap ? 2 : 1);
        int res_px = mt * kTileM;
        if (p.swap && !p.patch_w && !forced_mt) {
            // When all pixels fit in one round of items of at most 512 pixels, one item per block is the better
            // cut (64 x 32 x 32 pixels with 1 x 1 filters: 448 pixels per item 19.9 us, 256 per item 22.1 us).
            const long long one_round = ((total_pix + sms - 1) / sms + p.ovl + 31) / 32 * 32;
            if (one_round >= 64 && one_round <= 512) res_px = (int)one_round;
        }
        {
            const int want = env_int("CONV2D_B200_TF32_TILE_PX", 0);
            if (p.swap && want >= 64 && want <= 512 && want % 32 == 0 && pixel_items(want) > 0) res_px = want;
        }
        const int npix = npix_of(res_px);
        if ((p.swap ? res_px : mt * set_cols) <= 512 && npix <= 16000 && wbytes + extra + (size_t)2 * kCB * chunk_stride(npix) * 4 + kBookBytes <= kSmemLimit) {
            p.resident = 1;
            p.mt = p.swap ? (res_px + kTileM - 1) / kTileM : mt;
            p.tile_px = res_px;
            p.npix = npix;
            p.cbg = 1;
            p.a_stages = 2;
            p.b_stages = 1;
            p.tps = p.taps;
            auto need = [&](int a_stages, int cbg) { return wbytes + extra + (size_t)a_stages * cbg * kCB * chunk_stride(npix) * 4 + kBookBytes; };
            while (p.cbg * 2 <= p.cblks && npix * p.cbg * 2 <= kProducers * kUnitsPerThread &&
                   need(p.a_stages, p.cbg * 2) <= kSmemLimit) p.cbg *= 2;
            while (p.a_stages < kMaxAStages && need(p.a_stages + 1, p.cbg) <= kSmemLimit) ++p.a_stages;
            p.smem_bytes = need(p.a_stages, p.cbg);
        }
    }

    if (!p.resident) {
        // Streamed filters.  Measured: all SMs together draw filter stages from L2 at no more than
        // ~5-6 TB/s, i.e. a 8 KB stage costs ~120 cycles on top of the MMAs that consume it unless it is
        // reused by several tiles.  More tiles per item (mt) amortise that; fewer tiles leave room for a
        // second accumulator set (hidden write-back) and balance better.  Cost in units of one tile's MMA
        // time: rounds x mt x (1 + stage cost / MMA time) + exposed write-back.
        const size_t kLimit = kSmemLimit - extra;
        const double stage_cycles = chunk / 66.0;           // one (tap, channel block) of filters through L2
        const int forced_px = env_int("CONV2D_B200_TF32_TILE_PX", 0);
        const bool ksplit_allowed = env_int("CONV2D_B200_TF32_KSPLIT", 1) != 0;
        int best_px = 0;
        double best_cost = 0;
        if (p.swap) {
            // Any multiple of 32 pixels per item: the item size follows from the pixel count and the 148 SMs
            // (64 x 32 x 32 pixels: 448 per item = 147 items in one round, where 512 would occupy 128 SMs).
            // One or two MMAs of equal width cover the item per K step; an MMA narrower than 128 pixels is
            // bound by its ~64-cycle issue cost.
            for (int px = 512; px >= 64; px -= 32) {
                if (forced_px ? px != forced_px : (forced_mt && px != forced_mt * kTileM)) continue;
                const int groups = (px + 255) / 256;
                if (px % (16 * groups)) continue;
                const int npix = npix_of(px);
                if (npix > 16000 || smem_need(2, npix, p.n_tile, 2, 1, 1) > kLimit) continue;
                if (pixel_items(px) == 0) continue;
                const long long items = pixel_items(px) * p.n_blocks;
                const long long rounds = (items + sms - 1) / sms;
                const int nbuf = 2 * px <= 512 ? 2 : 1;
                const double mma_step = groups * ((px / groups) / 2.0 > 64.0 ? (px / groups) / 2.0 : 64.0);
                const double tile_time = (double)p.taps * p.cblks * (2 * mma_step + stage_cycles);
                const double writeback = (nbuf == 1 ? 1.0 : 0.15) * (px / 128.0) * (3000.0 * p.n_tile / 128.0);
                double cost = rounds * (tile_time + 0.5 * writeback);
                // (items that leave half of the SMs idle are split in two along the channels further down)
                if (items * 2 <= sms && p.cblks >= 2 && ksplit_allowed) cost = 0.5 * tile_time + writeback;
                if (best_px == 0 || cost < best_cost) { best_px = px; best_cost = cost; }
            }
        } else {
            const double mma_cycles = p.n_tile > 128 ? p.n_tile / 2 : 90;   // per 128-pixel tile and K step
            for (int mt = 4; mt >= 1; mt >>= 1) {
                if (forced_mt && mt != forced_mt) continue;
                if (mt * set_cols > 512) continue;
                const int npix = npix_of(mt * kTileM);
                if (npix > 16000 || smem_need(2, npix, p.n_tile, 2, 1, 1) > kLimit) continue;
                const long long items = (tiles + mt - 1) / mt * p.n_blocks;
                const long long rounds = (items + sms - 1) / sms;
                const int nbuf = (2 * mt * set_cols <= 512) ? 2 : 1;
                const double tile_time = (double)p.taps * p.cblks * (mt * 2 * mma_cycles + stage_cycles);
                const double writeback = (nbuf == 1 ? 1.0 : 0.15) * mt * (3000.0 * p.n_tile / 128.0);
                const double cost = rounds * (tile_time + 0.5 * writeback);
                if (best_px == 0 || cost < best_cost) { best_px = mt * kTileM; best_cost = cost; }
            }
        }
        if (best_px == 0) return p;
        p.tile_px = best_px;
        p.mt = (best_px + kTileM - 1) / kTileM;
        p.npix = npix_of(p.tile_px);
        // Filter stages: several taps per stage (up to 48 KB, trimmed below until three stages fit) so that the
        // single MMA-issuing thread pays its per-stage bookkeeping (barrier wait, commit: ~90 cycles, measured
        // by varying the stage size) once per 16-48 MMAs; the ring should hold
        // 64-128 KB in flight to cover the L2 latency.
        p.a_stages = 2;
        p.cbg = 1;
        p.tps = env_int("CONV2D_B200_TF32_STAGE_KB", 48) * 1024 / chunk;
        if (p.tps < 1) p.tps = 1;
        if (p.tps > p.taps) p.tps = p.taps;
        p.b_stages = 2;
        while (p.tps > 1 && smem_need(p.a_stages, p.npix, p.n_tile, 3, p.tps, 1) > kLimit) --p.tps;
        while (p.b_stages < 4 && smem_need(p.a_stages, p.npix, p.n_tile, p.b_stages + 1, p.tps, 1) <= kLimit) ++p.b_stages;
        while (p.a_stages < kMaxAStages && p.taps <= 3 &&
               smem_need(p.a_stages + 1, p.npix, p.n_tile, p.b_stages, p.tps, p.cbg) <= kLimit - 32 * 1024) ++p.a_stages;
        while (p.b_stages < kMaxBStages && smem_need(p.a_stages, p.npix, p.n_tile, p.b_stages + 1, p.tps, p.cbg) <= kLimit &&
               (size_t)p.b_stages * p.tps * chunk < 128 * 1024) ++p.b_stages;
        p.smem_bytes = smem_need(p.a_stages, p.npix, p.n_tile, p.b_stages, p.tps, p.cbg) + extra;
    }

    const int item_cols = p.swap ? p.tile_px : p.mt * p.n_tile;     // tensor-memory columns of one accumulator set
    p.px_groups = p.swap ? (p.tile_px + 255) / 256 : p.mt;
    {
        const int want = env_int("CONV2D_B200_TF32_PX_GROUPS", 0);
        if (p.swap && want > 0 && want <= 2 && p.tile_px % (16 * want) == 0 && p.tile_px / want <= 256) p.px_groups = want;
    }
    p.nbuf = (2 * item_cols <= 512 && env_int("CONV2D_B200_TF32_NBUF", 2) != 1) ? 2 : 1;
    if (p.patch_w) p.patch_rows = (sh.P + p.tile_px / p.patch_w - 1) / (p.tile_px / p.patch_w);
    if (pixel_items(p.tile_px) <= 0 || pixel_items(p.tile_px) > 0x7fffffffLL) return p;
    p.supertiles = (int)pixel_items(p.tile_px);
    // Too few tiles for the machine (e.g. 14 x 14 images): two work items per tile, each contracting half of
    // the channel-block groups and adding into a zeroed output.
    const int n_groups = (p.cblks + p.cbg - 1) / p.cbg;
    p.ksplit = ((long long)p.supertiles * p.n_blocks * 2 <= sms && n_groups >= 2 &&
                env_int("CONV2D_B200_TF32_KSPLIT", 1) != 0) ? 2 : 1;
    const long long items = (long long)p.supertiles * p.n_blocks * p.ksplit;
    if (items > 0x7fffffffLL) return p;
    p.grid = (int)(items < sms ? items : sms);
    int cols = p.nbuf * item_cols;
    p.tmem_cols = 32;
    while (p.tmem_cols < cols) p.tmem_cols <<= 1;
    p.ok = true;
    return p;
}

size_t packed_floats(const Plan& p)
{
    return (size_t)p.n_blocks * p.cblks * p.taps * kCB * p.n_tile;
}

// ---------------------------------------------------------------- filter re-ordering
// wp[nb][cb][t][chunk][f][e] = tf32(w[nb*n_tile + f][cb*kCB + 4*chunk + e][t]), zero outside K, C.
// With folded taps, channel index vc = (c*fold_r + r_in)*fold_s + s_in and tap index t = r_out*(S/fold_s) + s_out
// stand for filter element w[k][c][r_out*fold_r + r_in][s_out*fold_s + s_in].
struct FoldedFilter {
    int C, R, S, fold_r, fold_s;
    // offset of that element inside filter k's C*R*S block, or -1 for channel padding
    __device__ __forceinline__ int offset(int vc, int t) const
    {
        const int frs = fold_r * fold_s;
        const int c = vc / frs, rem = vc - c * frs;
        if (c >= C) return -1;
        const int r_in = rem / fold_s, s_in = rem - r_in * fold_s;
        const int s_eff = S / fold_s;
        const int r_out = t / s_eff, s_out = t - r_out * s_eff;
        return (c * R + r_out * fold_r + r_in) * S + s_out * fold_s + s_in;
    }
};

// One thread per (filter block, channel block, 16-byte chunk, filter, element) walks over the taps: its reads
// are the contiguous taps of one (filter, channel) pair (cached lines are reused from tap to tap), and for
// each tap a warp writes 32 adjacent elements.  T = float (rounded to TF32) with 4 elements per chunk, or a
// 16-bit pattern with 8.
// stacked = 1: half of the rows of the 128-row block are the filters' tap (r, 2u), the other half their tap
// (r, 2u + 1) (zeros where S is odd and 2u + 1 = S); tap index t = r * ceil(S / 2) + u.
template <typename T, int EPC>
__global__ void repack_filters_kernel(const T* __restrict__ w, T* __restrict__ wp, unsigned* __restrict__ status,
                                      int K, FoldedFilter ff, int taps, int n_tile, int cblks, long long threads_total,
                                      int stacked)
{
    grid_dep_launch();      // the convolution kernel may set itself up while this one runs
    // the status block in front of the filters starts every (non-prepacked) call cleared
    if (blockIdx.x == 0 && threadIdx.x < kStatusBytes / sizeof(unsigned)) status[threadIdx.x] = 0u;
    const bool folded = ff.fold_r * ff.fold_s > 1;
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < threads_total; i += stride) {
        long long r = i;
        const int e = (int)(r % EPC); r /= EPC;
        const int f = (int)(r % n_tile); r /= n_tile;
        const int chunk = (int)(r % kChunks); r /= kChunks;
        const int cb = (int)(r % cblks); r /= cblks;
        const int nb = (int)r;
        // stacked taps: rows 32q .. 32q+15 are maps 16q .. 16q+15 with the left-hand tap of a pair, rows 32q+16 .. 32q+31
        // the same maps with the right-hand tap, so that both halves of a map lie in the same quarter of the
        // accumulator lanes (the quarter one epilogue warp can read)
        const int k = stacked ? ((f >> 5) << 4) + (f & 15) : nb * n_tile + f;
        const int upper = stacked ? (f >> 4) & 1 : 0;
        const int s_slots = (ff.S + 1) / 2;
        const int vc = (cb * kChunks + chunk) * EPC + e;
        const T* src = w + (size_t)k * ff.C * ff.R * ff.S;
        T* dst = wp + ((((size_t)nb * cblks + cb) * taps * kChunks + chunk) * n_tile + f) * EPC + e;
        const size_t tap_stride = (size_t)kChunks * n_tile * EPC;
        const bool live = k < K && (folded ? vc < ff.C * ff.fold_r * ff.fold_s : vc < ff.C);
        for (int t = 0; t < taps; ++t, dst += tap_stride) {
            T v = T(0);
            if (live) {
                int o = folded ? ff.offset(vc, t) : vc * taps + t;
                if (stacked) {
                    const int r = t / s_slots, sx = 2 * (t - r * s_slots) + upper;
                    o = sx < ff.S ? (vc * ff.R + r) * ff.S + sx : -1;
                }
                if (o >= 0) {
                    v = __ldg(src + o);
                    if (sizeof(T) == 4) v = (T)to_tf32_rna((float)v);
                }
            }
            *dst = v;
        }
    }
}

// Re-ordering through shared memory for unfolded filters: a block takes 8 filters x one channel block x all
// taps.  Its reads are runs of (channels per block) x taps contiguous elements per filter, its writes runs of
// 8 filters x EPC elements (128 bytes with fp32) per (tap, chunk): both sides coalesced.
template <typename T, int EPC>
__global__ void repack_filters_tiled_kernel(const T* __restrict__ w, T* __restrict__ wp, unsigned* __restrict__ status,
                                            int K, int C, int taps, int n_tile, int cblks)
{
    extern __shared__ __align__(16) unsigned char repack_smem[];
    T* tile = reinterpret_cast<T*>(repack_smem);                 // [8][cpb * taps]
    grid_dep_launch();
    if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x < kStatusBytes / sizeof(unsigned)) status[threadIdx.x] = 0u;
    constexpr int cpb = kChunks * EPC;                           // channels per block
    const int cb = blockIdx.y, k0 = blockIdx.x * 8, c0 = cb * cpb;
    const int row = cpb * taps;
    const int c_live = min(cpb, C - c0) * taps;                  // elements of a filter's run that exist
    // Load: whole 16-byte words where a filter's run is full and 16-byte aligned, single elements otherwise.
    constexpr int kVec = 16 / (int)sizeof(T);
    const bool vec_ok = c_live == row && row % kVec == 0 && ((size_t)C * taps) % kVec == 0 &&
                        reinterpret_cast<uintptr_t>(w) % 16 == 0;
    if (vec_ok) {
        const int row_v = row / kVec;
#pragma unroll 4
        for (int idx = threadIdx.x; idx < 8 * row_v; idx += blockDim.x) {       // (independent loads: several in flight)
            const int kk = idx / row_v, rem = idx - kk * row_v;
            uint4 v = make_uint4(0u, 0u, 0u, 0u);
            if (k0 + kk < K) {
                v = __ldg(reinterpret_cast<const uint4*>(w + ((size_t)(k0 + kk) * C + c0) * taps) + rem);
                if (sizeof(T) == 4) {
                    v.x = __float_as_uint(to_tf32_rna(__uint_as_float(v.x))); v.y = __float_as_uint(to_tf32_rna(__uint_as_float(v.y)));
                    v.z = __float_as_uint(to_tf32_rna(__uint_as_float(v.z))); v.w = __float_as_uint(to_tf32_rna(__uint_as_float(v.w)));
                }
            }
            reinterpret_cast<uint4*>(tile)[idx] = v;
        }
    } else {
#pragma unroll 4
        for (int idx = threadIdx.x; idx < 8 * row; idx += blockDim.x) {
            const int kk = idx / row, rem = idx - kk * row;
            T v = T(0);
            if (k0 + kk < K && rem < c_live) {
                v = __ldg(w + ((size_t)(k0 + kk) * C + c0) * taps + rem);
                if (sizeof(T) == 4) v = (T)to_tf32_rna((float)v);
            }
            tile[idx] = v;
        }
    }
    __syncthreads();
    // Store: one 16-byte unit (EPC channels of one filter and tap) per thread and step.
    const int nb = k0 / n_tile, f0 = k0 - nb * n_tile;
    T* dst = wp + ((size_t)nb * cblks + cb) * taps * kChunks * n_tile * EPC;
    for (int idx = threadIdx.x; idx < 8 * kChunks * taps; idx += blockDim.x) {
        const int kk = idx % 8;
        const int rest = idx / 8;
        const int chunk = rest % kChunks, t = rest / kChunks;
        const T* src = tile + kk * row + (chunk * EPC) * taps + t;
        T u[EPC];
#pragma unroll
        for (int e = 0; e < EPC; ++e) u[e] = src[e * taps];
        uint4 v;
        if (sizeof(T) == 4) {
            v = make_uint4(__float_as_uint((float)u[0]), __float_as_uint((float)u[1]), __float_as_uint((float)u[2]), __float_as_uint((float)u[3]));
        } else {
            v = make_uint4((unsigned)u[0] | ((unsigned)u[1] << 16), (unsigned)u[2 % EPC] | ((unsigned)u[3 % EPC] << 16),
                           (unsigned)u[4 % EPC] | ((unsigned)u[5 % EPC] << 16), (unsigned)u[6 % EPC] | ((unsigned)u[7 % EPC] << 16));
        }
        *reinterpret_cast<uint4*>(dst + (((size_t)t * kChunks + chunk) * n_tile + f0 + kk) * EPC) = v;
    }
}

// Division of a non-negative int below 2^31 by a divisor fixed per launch, as a multiply-high, an add and a
// shift (round-up method for invariant divisors): a plain 32-bit division is a ~35-instruction dependent chain,
// and the pixel decoding below sits on the critical path of every producer unit and every epilogue block.
struct FastDiv {
    uint32_t mul, shift;
    int d;
    FastDiv() : mul(0), shift(0), d(1) {}
    explicit FastDiv(int divisor) : d(divisor)
    {
        uint32_t l = 0;
        while ((1ull << l) < (unsigned long long)divisor) ++l;
        shift = l;
        mul = (uint32_t)((((1ull << l) - (unsigned long long)divisor) << 32) / (unsigned long long)divisor + 1ull);
    }
    __device__ __forceinline__ int div(int n) const { return (int)((__umulhi((uint32_t)n, mul) + (uint32_t)n) >> shift); }
    __device__ __forceinline__ int divmod(int n, int& rem) const { const int q = div(n); rem = n - q * d; return q; }
};

struct KernelArgs {
    const float* x;
    const float* wp;
    float* y;
    unsigned* status;
    int N, C, H, W, K, R, S, P, Q;
    int HW;
    int total_pix;
    FastDiv div_HW, div_W, div_npix, div_qn, div_patch_w;   // divisors of the pixel decoding (qn = npix / 4)
    int vec_shift;    // log2(vec)
    FastDiv div_ksplit, div_n_blocks, div_groups_lo, div_groups_hi, div_per_image, div_patch_cols;   // divisors of the item decoding
    int patch_item_rows;   // patch addressing: output rows of one item (tile_px / patch_w)
    int n_tile, n_blocks, mt, tile_px, px_groups, nbuf, npix, cblks, taps, a_stages, b_stages, tps;
    int rot;          // quad producers rotate their chunk order per lane (see there)
    int cstride;      // 16-byte units between the 4-channel chunks of a staged channel block (npix + 1: odd)
    int patch_w, patch_tw, patch_rows, patch_cols;   // patch addressing (PATCH kernels): staged row pitch, valid output
                                                      // columns per patch row, patches per image down and across
    int pad_h, pad_w; // zero padding (patch addressing only): staged pixel (row, col) is image pixel (row - pad_h, col - pad_w)
    int row_pitch;    // pixels between vertically adjacent taps in the staged sequence: W, or patch_w
    int fp16;         // 16-bit operands only: 1 = IEEE half, 0 = bf16
    int fold_r, fold_s;  // taps folded into the channel dimension (1, 1: none); R, S below are what is left as shifts
    int helpers;      // 1: warps 8-15 share the write-back of a block's last item (operand-swap layout only)
    int pgroups;      // producer groups (1, 2 or 4): stage k is filled by group k % pgroups
    int quad;         // producers load four adjacent pixels per 128-bit (fp32) or 64-bit (16-bit operands) word (needs H*W % 4 == 0)
    int pair;         // 16-bit operands only: producers load two adjacent pixels per 32-bit word (needs H*W even)
    int cbg, groups;        // channel blocks per activation stage, number of such groups
    int resident;           // filters loaded once per thread block instead of streamed
    int swap;               // operand roles swapped: accumulator lanes = filters, columns = pixels
    int vec;                // swap mode: adjacent pixels a lane stores as one unit (1, 2 or 4)
    int pair_taps;          // stacked taps: accumulator lanes 64-127 hold the right-hand tap of each pair, one column to the right
    int s_slots, s_step;    // shift-table entries per filter row and the horizontal shift between them (2 with stacked taps)
    int item_stride;        // flat addressing: pixels between the starts of consecutive items (tile_px minus the overlap)
    int ksplit;             // items per output tile (split of the contraction): 1 or 2
    unsigned max_polls;     // bound of every barrier wait
    int test_drop_stage;    // test hook: the filter copy with this ordinal is armed but never issued (-1: none)
    int items;              // work items = supertiles x n_blocks
    unsigned tmem_cols;
};

// Where the staged pixel sequence of a work item lives in the image.
//   flat  (PATCH = false): pixels of the whole batch numbered j = (n*H + h)*W + w; an item is the run
//          [j0, j0 + tile_px) plus its halo; vertically adjacent taps are W pixels apart.
//   patch (PATCH = true): an item is a rectangle of patch_rows... rows x patch_w columns of one image starting at
//          (row0, col0), stored row after row with pitch patch_w (the staged halo adds R-1 rows); vertically adjacent
//          taps are patch_w pixels apart.  Columns >= patch_tw of a patch row only feed outputs of the next patch and
//          are dropped.  This keeps the halo small on wide images, for which the flat run would not fit on chip.
struct ItemGeom {
    int j0;             // flat: first pixel
    int n, row0, col0;  // patch: image and top-left corner
};
// Staged pixel jj -> (image n, offset inside one H*W plane); false when the pixel lies outside the batch / the image.
template <bool PATCH>
__device__ __forceinline__ bool staged_pixel(const KernelArgs& a, const ItemGeom& g, int jj, int& n, int& off)
{
    if (PATCH) {
        int pcol;
        const int prow = a.div_patch_w.divmod(jj, pcol);
        const int h = g.row0 + prow - a.pad_h, wc = g.col0 + pcol - a.pad_w;
        n = g.n;
        off = h * a.W + wc;
        return (unsigned)h < (unsigned)a.H && (unsigned)wc < (unsigned)a.W;
    }
    const int j = g.j0 + jj;
    n = a.div_HW.divmod(j, off);
    return j < a.total_pix;
}
// Accumulator column jj -> output (n, p, q); false when that output does not exist (window wraps over an edge).
template <bool PATCH>
__device__ __forceinline__ bool output_pixel(const KernelArgs& a, const ItemGeom& g, int jj, int& n, int& p, int& q)
{
    if (PATCH) {
        int pcol;
        const int prow = a.div_patch_w.divmod(jj, pcol);
        n = g.n;
        p = g.row0 + prow;
        q = g.col0 + pcol;
        return pcol < a.patch_tw && p < a.P && q < a.Q;
    }
    const int j = g.j0 + jj;
    if (j >= a.total_pix || jj >= a.item_stride) return false;       // (columns past the stride belong to the next item)
    int off;
    n = a.div_HW.divmod(j, off);
    p = a.div_W.divmod(off, q);
    return p < a.P && q < a.Q;
}

// Producer helpers.  A stage holds `cbg` channel blocks of kCB channels for npix pixels, laid out
// [channel block][chunk][pixel] in 16-byte units.  A work unit is (channel block g, pixel jj), numbered
// i = g * npix + jj; thread t of the 256 producers owns units first + t, first + t + 256, ...  Consecutive
// lanes read consecutive pixels of one channel (coalesced) and write consecutive 16-byte units.
template <bool B16, bool FOLD, bool PATCH, int CNT>
__device__ __forceinline__ void load_units(float (&v)[CNT][kCB], const KernelArgs& a, const ItemGeom& geom, int cb0, int first, int wtid, int nthr)
{
    const int units = a.npix * a.cbg;
#pragma unroll
    for (int u = 0; u < CNT; ++u) {
        const int i = first + u * nthr + wtid;
#pragma unroll
        for (int e = 0; e < kCB; ++e) v[u][e] = 0.f;
        if (i < units) {
            int jj;
            const int g = a.div_npix.divmod(i, jj);
            if (FOLD) {
                // Folded taps: staged channel vc = (c, r, s) of pixel j is x[c] at pixel j + r*W + s (zero beyond
                // the image: such windows belong to outputs that are dropped anyway).
                constexpr int kPer = B16 ? 2 * kCB : kCB;             // channels per 64-byte unit
                int n, off;
                if (staged_pixel<false>(a, geom, jj, n, off)) {
                    const int frs = a.fold_r * a.fold_s;
                    const int vc0 = (cb0 + g) * kPer;
                    int c = vc0 / frs, rem = vc0 - c * frs;
                    int r = rem / a.fold_s, sft = rem - r * a.fold_s;
                    const size_t base = (size_t)n * a.C * a.HW + off;
#pragma unroll
                    for (int e = 0; e < kPer; ++e) {
                        const int shift = r * a.W + sft;
                        const bool in = c < a.C && off + shift < a.HW;
                        if (B16) {
                            unsigned h = 0;
                            if (in) h = __ldg(reinterpret_cast<const unsigned short*>(a.x) + base + (size_t)c * a.HW + shift);
                            const unsigned prev = __float_as_uint(v[u][e >> 1]);
                            v[u][e >> 1] = __uint_as_float((e & 1) ? (prev | (h << 16)) : h);
                        } else {
                            if (in) v[u][e] = __ldg(a.x + base + (size_t)c * a.HW + shift);
                        }
                        if (++sft == a.fold_s) { sft = 0; if (++r == a.fold_r) { r = 0; ++c; } }
                    }
                }
            } else if (B16 && !FOLD && a.pair) {
                // Unit = 2 adjacent pixels x 16 channels: every load is one aligned 32-bit word holding the
                // two pixels of one channel (H*W even keeps pairs aligned and inside one image).
                const int half_n = a.npix >> 1;
                const int h = jj / half_n, pp = jj - h * half_n;
                const int c0 = (cb0 + g) * 2 * kCB + kCB * h;
                int n, off;
                if (staged_pixel<PATCH>(a, geom, 2 * pp, n, off) && c0 < a.C) {
                    const unsigned short* src = reinterpret_cast<const unsigned short*>(a.x) + ((size_t)n * a.C + c0) * a.HW + off;
#pragma unroll
                    for (int e = 0; e < kCB; ++e)
                        if (c0 + e < a.C) v[u][e] = __uint_as_float(__ldg(reinterpret_cast<const unsigned*>(src + (size_t)e * a.HW)));
                }
            } else if (B16) {
                // 32 16-bit channels of this pixel, packed two per 32-bit word (lower channel in the low half)
                const int c0 = (cb0 + g) * 2 * kCB;
                int n, off;
                if (staged_pixel<PATCH>(a, geom, jj, n, off) && c0 < a.C) {
                    const unsigned short* src = reinterpret_cast<const unsigned short*>(a.x) + ((size_t)n * a.C + c0) * a.HW + off;
#pragma unroll
                    for (int e = 0; e < kCB; ++e) {
                        unsigned lo = 0, hi = 0;
                        if (c0 + 2 * e < a.C) lo = __ldg(src + (size_t)(2 * e) * a.HW);
                        if (c0 + 2 * e + 1 < a.C) hi = __ldg(src + (size_t)(2 * e + 1) * a.HW);
                        v[u][e] = __uint_as_float(lo | (hi << 16));
                    }
                }
            } else {
                const int c0 = (cb0 + g) * kCB;
                int n, off;
                if (staged_pixel<PATCH>(a, geom, jj, n, off) && c0 < a.C) {
                    const float* src = a.x + ((size_t)n * a.C + c0) * a.HW + off;
#pragma unroll
                    for (int e = 0; e < kCB; ++e)
                        if (c0 + e < a.C) v[u][e] = __ldg(src + (size_t)e * a.HW);
                }
            }
        }
    }
}

template <bool B16, int CNT>
__device__ __forceinline__ void store_units(const float (&v)[CNT][kCB], float4* dst, const KernelArgs& a, int first, int wtid, int nthr)
{
    const int units = a.npix * a.cbg;
#pragma unroll
    for (int u = 0; u < CNT; ++u) {
        const int i = first + u * nthr + wtid;
        if (i < units) {
            int jj;
            const int g = a.div_npix.divmod(i, jj);
            if (B16 && a.pair) {
                const int half_n = a.npix >> 1;
                const int h = jj / half_n, pp = jj - h * half_n;
                float4* d = dst + ((size_t)g * kChunks + 2 * h) * a.cstride + 2 * pp;
#pragma unroll
                for (int m = 0; m < 2; ++m) {       // 8 channels per 16-byte unit; word k = channels 2k, 2k+1
                    unsigned lo[4], hi[4];
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const unsigned w0 = __float_as_uint(v[u][8 * m + 2 * k]), w1 = __float_as_uint(v[u][8 * m + 2 * k + 1]);
                        lo[k] = __byte_perm(w0, w1, 0x5410);     // first pixel: low halves
                        hi[k] = __byte_perm(w0, w1, 0x7632);     // second pixel: high halves
                    }
                    d[m * a.cstride] = make_float4(__uint_as_float(lo[0]), __uint_as_float(lo[1]), __uint_as_float(lo[2]), __uint_as_float(lo[3]));
                    d[m * a.cstride + 1] = make_float4(__uint_as_float(hi[0]), __uint_as_float(hi[1]), __uint_as_float(hi[2]), __uint_as_float(hi[3]));
                }
                continue;
            }
            float4* d = dst + (size_t)g * kChunks * a.cstride + jj;
#pragma unroll
            for (int ch = 0; ch < kChunks; ++ch)
                d[ch * a.cstride] = B16 ? make_float4(v[u][4 * ch], v[u][4 * ch + 1], v[u][4 * ch + 2], v[u][4 * ch + 3])
                                      : make_float4(to_tf32_rna(v[u][4 * ch]), to_tf32_rna(v[u][4 * ch + 1]),
                                                    to_tf32_rna(v[u][4 * ch + 2]), to_tf32_rna(v[u][4 * ch + 3]));
        }
    }
}

// Work item -> (supertile, filter block, part of the contraction).  With ksplit = 2 two items share an
// output tile, each contracts half of the channel-block groups and both add their partial sums into y
// (zeroed beforehand); 0 + a + b does not depend on the order, so the result stays deterministic.
struct ItemInfo {
    int supertile, nb, g_begin, n_groups, rot;
    ItemGeom geom;
};
__device__ __forceinline__ ItemInfo decode_item(const KernelArgs& a, int item)
{
    ItemInfo it;
    // (multiply-high divisions: this runs at the head of every item on the MMA thread and on the producers)
    int part;
    const int rest = a.div_ksplit.divmod(item, part);
    it.supertile = a.div_n_blocks.divmod(rest, it.nb);
    it.g_begin = a.div_ksplit.div(part * a.groups);
    it.n_groups = a.div_ksplit.div((part + 1) * a.groups) - it.g_begin;
    // blocks stream the filter bank in rotated order (see kernel); n_groups is floor or ceil of groups / ksplit
    (it.n_groups == a.div_groups_lo.d ? a.div_groups_lo : a.div_groups_hi).divmod(rest, it.rot);
    it.geom.j0 = it.supertile * a.item_stride;
    it.geom.n = it.geom.row0 = it.geom.col0 = 0;
    if (a.patch_w) {
        int rem, pc;
        it.geom.n = a.div_per_image.divmod(it.supertile, rem);
        const int pr = a.div_patch_cols.divmod(rem, pc);
        it.geom.row0 = pr * a.patch_item_rows;
        it.geom.col0 = pc * a.patch_tw;
    }
    return it;
}

// All MMAs of one tap of one channel block in the filters-as-M layout: K steps 0 and 1 for GROUPS pixel groups
// of n_mma pixels.  d: accumulator column of group 0; px_lo / flt_lo: low words of the pixel and filter
// descriptors of K step 0 (the K step and the group add constants to the start-address field); acc = 0 only
// for the very first tap of an item.
template <bool B16, int GROUPS>
__device__ __forceinline__ void issue_tap(uint32_t d, uint32_t px_lo, uint32_t flt_lo, uint32_t px_kstep, uint32_t flt_kstep,
                                          uint32_t n_mma, uint32_t desc_hi, uint32_t idesc, uint32_t acc)
{
#define CONV2D_TAP_MMA(KIND)                                                                                  \
    asm volatile(                                                                                             \
        "{\n\t.reg .pred p, q;\n\t.reg .b64 f0, f1, x;\n\t.reg .b32 t, dd;\n\t"                                 \
        "setp.ne.b32 p, %8, 0;\n\tsetp.eq.b32 q, 0, 0;\n\t"                                                   \
        "mov.b64 f0, {%2, %6};\n\tadd.u32 t, %2, %4;\n\tmov.b64 f1, {t, %6};\n\t"                             \
        "mov.b64 x, {%1, %6};\n\t"                                                                            \
        "tcgen05.mma.cta_group::1.kind::" KIND " [%0], f0, x, %7, p;\n\t"                                      \
        "add.u32 t, %1, %3;\n\tmov.b64 x, {t, %6};\n\t"                                                      \
        "tcgen05.mma.cta_group::1.kind::" KIND " [%0], f1, x, %7, q;\n\t"                                      \
        "setp.ne.b32 q, %9, 0;\n\t"                                                                           \
        "@!q bra DONE_%=;\n\t"                                                                                \
        "add.u32 dd, %0, %5;\n\tadd.u32 t, %1, %5;\n\tmov.b64 x, {t, %6};\n\t"                               \
        "tcgen05.mma.cta_group::1.kind::" KIND " [dd], f0, x, %7, p;\n\t"                                      \
        "add.u32 t, t, %3;\n\tmov.b64 x, {t, %6};\n\t"                                                       \
        "tcgen05.mma.cta_group::1.kind::" KIND " [dd], f1, x, %7, q;\n\t"                                      \
        "DONE_%=:\n\t}"                                                                                       \
        ::"r"(d), "r"(px_lo), "r"(flt_lo), "r"(px_kstep), "r"(flt_kstep), "r"(n_mma), "r"(desc_hi), "r"(idesc), \
          "r"(acc), "n"(GROUPS == 2 ? 1 : 0) : "memory")
    if (B16) CONV2D_TAP_MMA("f16"); else CONV2D_TAP_MMA("tf32");
#undef CONV2D_TAP_MMA
}

template <bool B16, bool FOLD, bool PATCH, bool STACK>
__global__ void __launch_bounds__(kThreads, 1)
general_tc_kernel(const KernelArgs a)
{
    extern __shared__ __align__(128) unsigned char smem[];
    const uint32_t a_block_bytes = (uint32_t)kCB * a.cstride * 4;       // one channel block of a stage
    const uint32_t a_stage_bytes = a_block_bytes * (uint32_t)a.cbg;
    const uint32_t b_chunk_bytes = (uint32_t)kCB * a.n_tile * 4;        // one (channel block, tap)
    const uint32_t b_stage_bytes = b_chunk_bytes * (uint32_t)a.tps;
    unsigned char* a_smem = smem;
    unsigned char* b_smem = smem + (size_t)a.a_stages * a_stage_bytes;
    const size_t b_region_bytes = a.resident ? (size_t)a.cblks * a.taps * b_chunk_bytes : (size_t)a.b_stages * b_stage_bytes;
    float* xpose = reinterpret_cast<float*>(b_smem + b_region_bytes);            // only present (and used) when a.swap
    uint64_t* bars = reinterpret_cast<uint64_t*>(b_smem + b_region_bytes + (a.swap ? kXposeBytes : 0));
    uint64_t* a_full = bars;                               // [kMaxAStages]
    uint64_t* a_empty = a_full + kMaxAStages;              // [kMaxAStages]
    uint64_t* b_full = a_empty + kMaxAStages;              // [kMaxBStages]
    uint64_t* b_empty = b_full + kMaxBStages;              // [kMaxBStages]
    uint64_t* acc_full = b_empty + kMaxBStages;            // [2]
    uint64_t* acc_empty = acc_full + 2;                    // [2]
    uint64_t* tail_full = acc_empty + 2;                   // [1] the block's last item is complete (for warps 8-15)
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tail_full + 1);
    volatile uint32_t* abort_flag = tmem_slot + 1;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    volatile unsigned long long* t_entry = reinterpret_cast<volatile unsigned long long*>(tmem_slot + 2);
    uint32_t* tap_shift = tmem_slot + 4;                   // [taps] r * row_pitch + s of every tap, in staged pixels
    for (int t = tid; t < a.taps; t += kThreads) tap_shift[t] = (uint32_t)((t / a.s_slots) * a.row_pitch + (t % a.s_slots) * a.s_step);
    if (tid == 0) { unsigned long long t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); *t_entry = t; }

    if (tid == 0) {
        for (int i = 0; i < a.a_stages; ++i) { mbar_init(&a_full[i], kProducers / a.pgroups); mbar_init(&a_empty[i], 1); }
        for (int i = 0; i < a.b_stages; ++i) { mbar_init(&b_full[i], 1); mbar_init(&b_empty[i], 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(&acc_full[i], 1); mbar_init(&acc_empty[i], kEpilogueWarps); }
        mbar_init(tail_full, 1);
        *abort_flag = 0;
        fence_mbar_init();
    }
    __syncthreads();
    if (warp == 1) { tmem_alloc(tmem_slot, a.tmem_cols); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = *tmem_slot;
    // Everything above touched only this block's shared and tensor memory; it may overlap the tail of the
    // preceding kernel on the stream (the filter re-ordering of this call, or the previous call).  From here
    // on global memory is read and written.
    grid_dep_launch();
    grid_dep_wait();

    // Work item -> (supertile, filter block); blocks rotate the order of the channel-block groups by the
    // item number, so that at any moment they stream different parts of the filter bank.
    const int acc_cols = a.swap ? a.tile_px : a.mt * a.n_tile;   // tensor-memory columns of one accumulator set

    if (warp == 0) {
        // ---------------- filters: global -> shared by bulk copy, up to `tps` taps of one channel block per stage
        if (lane == 0) {
            int s = 0, issued = 0;
            uint32_t ph = 0;
            bool alive = true;
            if (a.resident) {
                // the whole filter bank (a single filter block in this mode), once, one bulk copy per channel
                // block, all on one barrier
                const unsigned char* src = reinterpret_cast<const unsigned char*>(a.wp);
                const uint32_t piece = b_chunk_bytes * (uint32_t)a.taps;
                mbar_arrive_expect_tx(&b_full[0], piece * (uint32_t)a.cblks);
                for (int cb = 0; cb < a.cblks; ++cb)
                    bulk_g2s(b_smem + (size_t)cb * piece, src + (size_t)cb * piece, piece, &b_full[0]);
                alive = false;          // nothing to stream
                if (*abort_flag) { uint32_t dummy = 0; mbar_wait_bounded(&b_full[0], 0u, &dummy, 1u << 16); }
            }
            for (int item = blockIdx.x; item < a.items && alive; item += gridDim.x) {
                const ItemInfo ii = decode_item(a, item);
                const int nb = ii.nb;
                const unsigned char* src = reinterpret_cast<const unsigned char*>(a.wp)
                                         + (size_t)nb * a.cblks * a.taps * b_chunk_bytes;
                for (int grp = 0; grp < ii.n_groups && alive; ++grp) {
                    int gr = grp + ii.rot;
                    if (gr >= ii.n_groups) gr -= ii.n_groups;
                    gr += ii.g_begin;
                    for (int g = 0; g < a.cbg && alive; ++g) {
                        const int cbr = gr * a.cbg + g;
                        if (cbr >= a.cblks) break;
                        for (int t0 = 0; t0 < a.taps; t0 += a.tps) {
                            const int nt = min(a.tps, a.taps - t0);
                            if (!mbar_wait_bounded(&b_empty[s], ph ^ 1u, abort_flag, a.max_polls)) { alive = false; break; }
                            const uint32_t bytes = b_chunk_bytes * (uint32_t)nt;
                            mbar_arrive_expect_tx(&b_full[s], bytes);
                            if (issued != a.test_drop_stage)     // (test hook: a dropped copy makes the consumer's wait expire)
                                bulk_g2s(b_smem + (size_t)s * b_stage_bytes, src + ((size_t)cbr * a.taps + t0) * b_chunk_bytes,
                                         bytes, &b_full[s]);
                            ++issued;
                            if (++s == a.b_stages) { s = 0; ph ^= 1u; }
                        }
                    }
                }
            }
            if (*abort_flag && !a.resident) {
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
            const uint32_t m_rows = a.swap ? (uint32_t)a.n_tile : (uint32_t)kTileM;
            const uint32_t n_mma = (uint32_t)(a.tile_px / a.px_groups);          // operand-swap layout: pixels per MMA
            const uint32_t n_cols = a.swap ? n_mma : (uint32_t)a.n_tile;
            const uint32_t idesc = B16 ? idesc_b16(m_rows, n_cols, a.fp16 != 0) : idesc_tf32(m_rows, n_cols);
            auto pack64 = [](uint32_t lo, uint32_t hi) {
                uint64_t r;
                asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
                return r;
            };
            auto mma = [](uint32_t d, uint64_t ad, uint64_t bd, uint32_t id, bool acc) {
                if (B16) mma_b16(d, ad, bd, id, acc); else mma_tf32(d, ad, bd, id, acc);
            };
            const uint32_t desc_hi = (128u >> 4) | (1u << 14);                  // SBO = 128 B, descriptor version 1
            const uint32_t a_lo_fixed = ((uint32_t)a.cstride & 0x3FFFu) << 16;  // LBO = chunk stride * 16 B
            const uint32_t b_lo_fixed = ((uint32_t)a.n_tile & 0x3FFFu) << 16;   // LBO = n_tile * 16 B
            const uint32_t a_kstep = 2u * (uint32_t)a.cstride;                  // 8 channels further, in 16-byte units
            const uint32_t b_kstep = 2u * (uint32_t)a.n_tile;
            bool alive = true;
            int as = 0, bs = 0, buf = 0;
            uint32_t a_phase = 0, b_phase = 0, acc_phase0 = 0, acc_phase1 = 0;
            // diagnostics of block 0 (status words 2..5): cycles this thread waited for activations and for a
            // free accumulator set, its total cycles, its item count
            long long wait_a = 0, wait_acc = 0, issue_cycles = 0;
            const long long t_begin = clock_now();
            if (blockIdx.x == 0) {
                unsigned long long t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
                a.status[6] = (unsigned)(t - *t_entry);          // ns from kernel entry to the start of the MMA loop
            }
            int n_items = 0;
            if (a.resident) {
                if (!mbar_wait_bounded(&b_full[0], 0u, abort_flag, a.max_polls)) alive = false;
                tc_fence_after_sync();
            }
            for (int item = blockIdx.x; item < a.items && alive; item += gridDim.x) {
                const ItemInfo ii = decode_item(a, item);
                // the accumulator set must have been drained by the epilogue of its previous item
                const uint32_t acc_phase = buf ? acc_phase1 : acc_phase0;
                long long tw = clock_now();
                if (!mbar_wait_bounded(&acc_empty[buf], acc_phase ^ 1u, abort_flag, a.max_polls)) { alive = false; break; }
                tc_fence_after_sync();
                wait_acc += clock_now() - tw;
                const uint32_t d0 = tmem + (uint32_t)(buf * acc_cols);
                uint32_t accumulate = 0;
                for (int grp = 0; grp < ii.n_groups && alive; ++grp) {
                    tw = clock_now();
                    if (!mbar_wait_bounded(&a_full[as], a_phase, abort_flag, a.max_polls)) { alive = false; break; }
                    tc_fence_after_sync();
                    wait_a += clock_now() - tw;
                    const long long t_issue0 = clock_now();
                    int gr = grp + ii.rot;
                    if (gr >= ii.n_groups) gr -= ii.n_groups;
                    gr += ii.g_begin;
                    uint32_t a_lo_block = a_lo_fixed | (smem_u32(a_smem + (size_t)as * a_stage_bytes) >> 4);
                    for (int g = 0; g < a.cbg && alive; ++g, a_lo_block += a_block_bytes >> 4) {
                        if (gr * a.cbg + g >= a.cblks) break;
                        uint32_t row_shift = 0;                                  // r * row pitch, in pixels (= 16-byte units)
                        int sx = 0, sc = 0;
                        for (int t0 = 0; t0 < a.taps; t0 += a.tps) {
                            const int nt = min(a.tps, a.taps - t0);
                            uint32_t b_lo;
                            if (a.resident) {
                                b_lo = b_lo_fixed | (smem_u32(b_smem + (size_t)(gr * a.cbg + g) * a.taps * b_chunk_bytes) >> 4);
                            } else {
                                if (!mbar_wait_bounded(&b_full[bs], b_phase, abort_flag, a.max_polls)) { alive = false; break; }
                                tc_fence_after_sync();
                                b_lo = b_lo_fixed | (smem_u32(b_smem + (size_t)bs * b_stage_bytes) >> 4);
                            }
                            if (a.swap && a.px_groups == 1) {
                                // M operand = the 128 filters of this stage, N operand = n_mma staged pixels.
                                // One MMA pair per tap carries less tensor-pipe work than this one thread needs to
                                // issue it with loop and address arithmetic around it (~230 cycles per MMA that
                                // way), so a tap is one block of straight-line code and its shift comes from a
                                // table, fetched one tap ahead.
                                const uint32_t* shift = tap_shift + t0;
                                uint32_t cur = shift[0];
#pragma unroll 3
                                for (int t = 0; t < nt; ++t, b_lo += b_chunk_bytes >> 4) {
                                    const uint32_t a_lo = a_lo_block + cur;
                                    cur = shift[t + 1 < nt ? t + 1 : t];
                                    issue_tap<B16, 1>(d0, a_lo, b_lo, a_kstep, b_kstep, n_mma, desc_hi, idesc, accumulate);
                                    accumulate = 1;
                                }
                            } else {
                                for (int t = 0; t < nt; ++t, b_lo += b_chunk_bytes >> 4) {
                                    uint32_t a_lo = a_lo_block + row_shift + (uint32_t)sx;
                                    uint32_t d = d0;
                                    if (a.swap) {
                                        // two pixel groups: four MMAs per tap keep the pipe busy (measured faster
                                        // when the compiler schedules the address arithmetic between them)
                                        const uint64_t bd0 = pack64(b_lo, desc_hi), bd1 = pack64(b_lo + b_kstep, desc_hi);
                                        mma(d, bd0, pack64(a_lo, desc_hi), idesc, accumulate != 0);
                                        mma(d, bd1, pack64(a_lo + a_kstep, desc_hi), idesc, true);
                                        mma(d + n_mma, bd0, pack64(a_lo + n_mma, desc_hi), idesc, accumulate != 0);
                                        mma(d + n_mma, bd1, pack64(a_lo + n_mma + a_kstep, desc_hi), idesc, true);
                                    } else {
                                        for (int m = 0; m < a.mt; ++m, a_lo += kTileM, d += (uint32_t)a.n_tile) {
                                            mma(d, ((uint64_t)desc_hi << 32) | a_lo, ((uint64_t)desc_hi << 32) | b_lo, idesc, accumulate != 0);
                                            mma(d, ((uint64_t)desc_hi << 32) | (a_lo + a_kstep),
                                                     ((uint64_t)desc_hi << 32) | (b_lo + b_kstep), idesc, true);
                                        }
                                    }
                                    accumulate = 1;
                                    sx += a.s_step;
                                    if (++sc == a.s_slots) { sc = 0; sx = 0; row_shift += (uint32_t)a.row_pitch; }
                                }
                            }
                            if (!a.resident) {
                                mma_commit(&b_empty[bs]);   // frees the filter stage when these MMAs have read it
                                if (++bs == a.b_stages) { bs = 0; b_phase ^= 1u; }
                            }
                        }
                    }
                    issue_cycles += clock_now() - t_issue0;
                    if (alive) mma_commit(&a_empty[as]);
                    if (++as == a.a_stages) { as = 0; a_phase ^= 1u; }
                }
                if (alive) mma_commit(&acc_full[buf]);
                if (alive && item + (int)gridDim.x >= a.items) mma_commit(tail_full);
                if (buf) acc_phase1 ^= 1u; else acc_phase0 ^= 1u;
                if (++buf == a.nbuf) buf = 0;
                ++n_items;
            }
            if (blockIdx.x == 0) {
                a.status[2] = (unsigned)wait_a;
                a.status[3] = (unsigned)wait_acc;
                a.status[4] = (unsigned)(clock_now() - t_begin);
                a.status[5] = (unsigned)n_items;
                a.status[9] = (unsigned)issue_cycles;
                unsigned long long t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
                a.status[7] = (unsigned)(t - *t_entry);          // ns from kernel entry to the last MMA issued
            }
        }
    } else {
    if (producer_index(warp) >= 0) {
        // ---------------- producers: stage activations, running ahead across item boundaries
        // The producer warps form `pgroups` groups; stage k of the block's stage sequence is filled by group
        // k % pgroups, so that several stages' memory round trips are in flight at once (a stage of a light
        // problem has fewer 16-channel units than there are producer threads).
        const int nthr_shift = a.pgroups == 4 ? 6 : (a.pgroups == 2 ? 7 : 8);     // kProducers = 256 threads; no divisions here:
        const int nthr = 1 << nthr_shift;                                         // this is on the path to the first load
        const int gid = (producer_index(warp) * 32 + lane) >> nthr_shift;
        const int wtid = (producer_index(warp) * 32 + lane) - gid * nthr;
        bool alive = true;
        int kstage = 0;
        int next_as = 0;                 // ring slot and phase of stage `kstage`, advanced without divisions
        uint32_t next_phase = 0;
        const int units = a.npix * a.cbg;
        for (int item = blockIdx.x; item < a.items && alive; item += gridDim.x) {
            const ItemInfo ii = decode_item(a, item);
            // One stage = cbg consecutive channel blocks.  All loads of a pass (kUnitsPerThread units of
            // 16 channels per thread) are issued before its first store: a pass costs one memory round trip.
            for (int grp = 0; grp < ii.n_groups && alive; ++grp, ++kstage) {
                const int as = next_as;
                const uint32_t a_phase = next_phase;
                if (++next_as == a.a_stages) { next_as = 0; next_phase ^= 1u; }
                if ((kstage & (a.pgroups - 1)) != gid) continue;         // pgroups is 1, 2 or 4
                if (!mbar_wait_bounded(&a_empty[as], a_phase ^ 1u, abort_flag, a.max_polls)) { alive = false; break; }
                float4* dst = reinterpret_cast<float4*>(a_smem + (size_t)as * a_stage_bytes);
                int gr = grp + ii.rot;
                if (gr >= ii.n_groups) gr -= ii.n_groups;
                gr += ii.g_begin;
                if (!B16 && !FOLD && a.quad) {
                    // H*W a multiple of 4: a thread fetches 4 adjacent pixels of each of the 16 channels with
                    // 128-bit loads (a quarter of the load instructions, which otherwise crowd the SM's memory
                    // pipeline that the MMA instructions pass through as well) and writes four 16-channel units.
                    const int qn = a.npix >> 2;
                    for (int i = wtid; i < qn * a.cbg; i += nthr) {
                        int pq;
                        const int g = a.div_qn.divmod(i, pq);
                        const int c0 = (gr * a.cbg + g) * kCB;
                        // Register group ch of this lane holds chunk (ch + rot) & 3: lanes whose 64-byte pieces
                        // would fall on the same banks write different chunks in the same instruction.  Measured:
                        // a gain with 16-bit operands (below) only; with fp32 inputs the rotation is left out,
                        // as it splits every 512-byte load instruction over four channel planes (slower from DRAM).
                        const int rot = a.rot ? (pq >> 1) & 3 : 0;
                        float4 v[kCB];
#pragma unroll
                        for (int e = 0; e < kCB; ++e) v[e] = make_float4(0.f, 0.f, 0.f, 0.f);
                        int n, off;
                        if (staged_pixel<PATCH>(a, ii.geom, 4 * pq, n, off) && c0 < a.C) {
                            const float* src = a.x + ((size_t)n * a.C + c0) * a.HW + off;
#pragma unroll
                            for (int ch = 0; ch < kChunks; ++ch) {
                                const int cc = ((ch + rot) & 3) << 2;                 // first channel of this register group
                                const float* sc = src + (size_t)cc * a.HW;
                                const int left = a.C - c0 - cc;                       // channels that exist from there on
#pragma unroll
                                for (int j = 0; j < 4; ++j)
                                    if (j < left) v[4 * ch + j] = __ldg(reinterpret_cast<const float4*>(sc + (size_t)j * a.HW));
                            }
                        }
                        float4* d = dst + (size_t)g * kChunks * a.cstride + 4 * pq;
#pragma unroll
                        for (int ch = 0; ch < kChunks; ++ch) {
                            float4* dc = d + ((ch + rot) & 3) * a.cstride;
                            dc[0] = make_float4(to_tf32_rna(v[4 * ch].x), to_tf32_rna(v[4 * ch + 1].x), to_tf32_rna(v[4 * ch + 2].x), to_tf32_rna(v[4 * ch + 3].x));
                            dc[1] = make_float4(to_tf32_rna(v[4 * ch].y), to_tf32_rna(v[4 * ch + 1].y), to_tf32_rna(v[4 * ch + 2].y), to_tf32_rna(v[4 * ch + 3].y));
                            dc[2] = make_float4(to_tf32_rna(v[4 * ch].z), to_tf32_rna(v[4 * ch + 1].z), to_tf32_rna(v[4 * ch + 2].z), to_tf32_rna(v[4 * ch + 3].z));
                            dc[3] = make_float4(to_tf32_rna(v[4 * ch].w), to_tf32_rna(v[4 * ch + 1].w), to_tf32_rna(v[4 * ch + 2].w), to_tf32_rna(v[4 * ch + 3].w));
                        }
                    }
                } else if (B16 && !FOLD && a.quad) {
                    // 16-bit operands, same idea: 64-bit loads of 4 adjacent pixels for each of the 32 channels of a
                    // block, then the 4 x 32 block is turned around in registers into four 64-byte units.
                    const int qn = a.npix >> 2;
                    for (int i = wtid; i < qn * a.cbg; i += nthr) {
                        int pq;
                        const int g = a.div_qn.divmod(i, pq);
                        const int c0 = (gr * a.cbg + g) * 2 * kCB;
                        const int rot = a.rot ? (pq >> 1) & 3 : 0;    // chunk rotation of this lane, as above
                        uint2 v[2 * kCB];
#pragma unroll
                        for (int e = 0; e < 2 * kCB; ++e) v[e] = make_uint2(0u, 0u);
                        int n, off;
                        if (staged_pixel<PATCH>(a, ii.geom, 4 * pq, n, off) && c0 < a.C) {
                            const unsigned short* src = reinterpret_cast<const unsigned short*>(a.x) + ((size_t)n * a.C + c0) * a.HW + off;
#pragma unroll
                            for (int ch = 0; ch < kChunks; ++ch) {
                                const int cc = ((ch + rot) & 3) << 3;
                                const unsigned short* sc = src + (size_t)cc * a.HW;
                                const int left = a.C - c0 - cc;
#pragma unroll
                                for (int j = 0; j < 8; ++j)
                                    if (j < left) v[8 * ch + j] = __ldg(reinterpret_cast<const uint2*>(sc + (size_t)j * a.HW));
                            }
                        }
                        float4* d = dst + (size_t)g * kChunks * a.cstride + 4 * pq;
#pragma unroll
                        for (int ch = 0; ch < kChunks; ++ch) {        // 8 channels per 16-byte unit; word k = channels 2k, 2k+1
                            float4* dc = d + ((ch + rot) & 3) * a.cstride;
                            unsigned p0[4], p1[4], p2[4], p3[4];
#pragma unroll
                            for (int k = 0; k < 4; ++k) {
                                const uint2 lo = v[8 * ch + 2 * k], hi = v[8 * ch + 2 * k + 1];
                                p0[k] = __byte_perm(lo.x, hi.x, 0x5410); p1[k] = __byte_perm(lo.x, hi.x, 0x7632);
                                p2[k] = __byte_perm(lo.y, hi.y, 0x5410); p3[k] = __byte_perm(lo.y, hi.y, 0x7632);
                            }
                            dc[0] = make_float4(__uint_as_float(p0[0]), __uint_as_float(p0[1]), __uint_as_float(p0[2]), __uint_as_float(p0[3]));
                            dc[1] = make_float4(__uint_as_float(p1[0]), __uint_as_float(p1[1]), __uint_as_float(p1[2]), __uint_as_float(p1[3]));
                            dc[2] = make_float4(__uint_as_float(p2[0]), __uint_as_float(p2[1]), __uint_as_float(p2[2]), __uint_as_float(p2[3]));
                            dc[3] = make_float4(__uint_as_float(p3[0]), __uint_as_float(p3[1]), __uint_as_float(p3[2]), __uint_as_float(p3[3]));
                        }
                    }
                } else
                for (int first = 0; first < units; first += nthr * kUnitsPerThread) {
                    float v[kUnitsPerThread][kCB];
                    load_units<B16, FOLD, PATCH>(v, a, ii.geom, gr * a.cbg, first, wtid, nthr);
                    store_units<B16>(v, dst, a, first, wtid, nthr);
                }
                fence_proxy_async_smem();
                mbar_arrive(&a_full[as]);
            }
        }
    }
    if (warp >= 4 && (warp < 4 + kEpilogueWarps || a.helpers)) {
        // ---------------- epilogue: drain finished accumulator sets (lane = pixel)
        // Warps 4-7 drain every item.  The write-back of a block's LAST item cannot hide behind any later
        // MMAs, so there the eight warps 8-15 (producers that have finished staging, and the two spare
        // warps) join in: each lane quarter is then drained by three warps that take every third 32-pixel
        // block.  Their transposition tiles reuse the activation ring, which is idle by then.
        const int quarter = warp & 3;                       // tensor-memory lanes this warp may read
        const bool helper = warp >= 4 + kEpilogueWarps;
        const int share = helper ? 1 + ((warp - 8) >> 2) : 0;
        const size_t plane = (size_t)a.P * a.Q;
        const int chunks_per_tile = a.n_tile / 16;
        const int total_chunks = a.mt * chunks_per_tile;
        const int n_local = ((int)blockIdx.x < a.items) ? (a.items - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;
        bool alive = true;
        for (int li = helper ? n_local - 1 : 0; li >= 0 && li < n_local; ++li) {
            const int item = (int)blockIdx.x + li * (int)gridDim.x;
            const int buf = a.nbuf == 2 ? (li & 1) : 0;                              // nbuf is 1 or 2
            const uint32_t acc_phase = (uint32_t)(a.nbuf == 2 ? li >> 1 : li) & 1u;
            const bool split = a.helpers && li == n_local - 1;
            const ItemInfo ii = decode_item(a, item);
            const int nb = ii.nb;
            const bool add = a.ksplit > 1;                   // partial sums: add into the zeroed output
            // tcgen05.ld is warp-collective: take the decision for the whole warp
            // (warps 8-15 come late and only for the last item: they wait on a barrier of its own, whose
            // phase they cannot have missed)
            alive = __all_sync(0xffffffffu, alive && mbar_wait_bounded(helper ? tail_full : &acc_full[buf],
                                                                       helper ? 0u : acc_phase, abort_flag, a.max_polls));
            if (!alive) break;
            tc_fence_after_sync();
            const uint32_t lane_base = tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * acc_cols);
            if (a.swap) {
                // Lanes are filters, columns pixels: this thread holds adjacent pixels of ONE map.  A
                // warp-private shared-memory tile turns a 32-filter x 32-pixel block around so that each
                // store instruction again writes 32 adjacent pixels of one map.
                float* tile = helper ? reinterpret_cast<float*>(a_smem) + (size_t)(warp - 8) * 32 * kXposePitch
                                     : xpose + (size_t)(warp - 4) * 32 * kXposePitch;
                // Stacked taps: lanes 0-15 of the quarter hold 16 maps summed over the left-hand taps, lanes 16-31 the
                // same maps over the right-hand taps, one column to the right: those lanes write their row shifted
                // by one column (with the first column of the next block), and a map is the sum of two tile rows.
                constexpr bool stacked = STACK;         // (a template parameter: as a run-time flag it slowed the ordinary epilogue by 15 %)
                const int rpq = stacked ? 16 : a.n_tile / 4;    // maps per lane quarter: 32 (M = 128) or 16 (M = 64: lanes 0-15; stacked taps)
                const int blocks = a.tile_px / 32;
                auto load_block = [&](uint32_t (&v0)[16], uint32_t (&v1)[16], uint32_t (&vx)[1], int b) {
                    tmem_ld16(lane_base + (uint32_t)(b * 32), v0);
                    tmem_ld16(lane_base + (uint32_t)(b * 32 + 16), v1);
                    vx[0] = 0u;
                    if (stacked && b + 1 < blocks) tmem_ld1(lane_base + (uint32_t)(b * 32 + 32), vx);
                };
                auto store_block = [&](const uint32_t (&v0)[16], const uint32_t (&v1)[16], const uint32_t (&vx)[1], int b) {
                    __syncwarp();                                   // the previous block has been read out
                    float4* row = reinterpret_cast<float4*>(tile + lane * kXposePitch);
                    if (stacked) {
                        const bool up = lane >= 16;
                        auto sel = [&](uint32_t lo, uint32_t hi) { return __uint_as_float(up ? hi : lo); };
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            row[i] = make_float4(sel(v0[4 * i], v0[4 * i + 1]), sel(v0[4 * i + 1], v0[4 * i + 2]),
                                                 sel(v0[4 * i + 2], v0[4 * i + 3]), sel(v0[4 * i + 3], i < 3 ? v0[(4 * i + 4) & 15] : v1[0]));
                            row[4 + i] = make_float4(sel(v1[4 * i], v1[4 * i + 1]), sel(v1[4 * i + 1], v1[4 * i + 2]),
                                                     sel(v1[4 * i + 2], v1[4 * i + 3]), sel(v1[4 * i + 3], i < 3 ? v1[(4 * i + 4) & 15] : vx[0]));
                        }
                    } else if (lane < rpq) {                        // M = 64: only lanes 0-15 of a quarter hold rows
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            row[i] = make_float4(__uint_as_float(v0[4 * i]), __uint_as_float(v0[4 * i + 1]),
                                                 __uint_as_float(v0[4 * i + 2]), __uint_as_float(v0[4 * i + 3]));
                            row[4 + i] = make_float4(__uint_as_float(v1[4 * i]), __uint_as_float(v1[4 * i + 1]),
                                                     __uint_as_float(v1[4 * i + 2]), __uint_as_float(v1[4 * i + 3]));
                        }
                    }
                    __syncwarp();
                    // Each lane stores `vec` adjacent pixels of one map, so one instruction covers `vec` maps:
                    // per-warp store throughput is bounded by instructions in flight, not bytes (measured
                    // ~2.7 B/clk per warp with 4-byte lanes), hence the widest unit the alignment allows.
                    const int vec = a.vec;                          // 1, 2 or 4 (W, Q, P*Q multiples of vec)
                    const int lanes_per_row = 32 >> a.vec_shift;
                    const int row_sub = lane >> (5 - a.vec_shift), pg = lane & (lanes_per_row - 1);
                    int n, p, q;                                    // this lane's first pixel of the block
                    const bool ok = output_pixel<PATCH>(a, ii.geom, b * 32 + pg * vec, n, p, q);
                    float* o = a.y;
                    if (ok) o = a.y + (((size_t)n * a.K + nb * a.n_tile + quarter * rpq + row_sub) * a.P + p) * a.Q + q;
                    if (ok) {
                        const int kmax = min(rpq, a.K - nb * a.n_tile - quarter * rpq);   // maps of this quarter that exist
                        const float* src = tile + row_sub * kXposePitch + pg * vec;
                        if (vec == 4) {
#pragma unroll 4
                            for (int r = 0; r < 32; r += 4, o += 4 * plane, src += 4 * kXposePitch)
                                if (r + row_sub < kmax) {
                                    float4 t = *reinterpret_cast<const float4*>(src);
                                    if (stacked) {
                                        const float4 u = *reinterpret_cast<const float4*>(src + 16 * kXposePitch);
                                        t.x += u.x; t.y += u.y; t.z += u.z; t.w += u.w;
                                    }
                                    if (add) { atomicAdd(o, t.x); atomicAdd(o + 1, t.y); atomicAdd(o + 2, t.z); atomicAdd(o + 3, t.w); }
                                    else *reinterpret_cast<float4*>(o) = t;
                                }
                        } else if (vec == 2) {
#pragma unroll 8
                            for (int r = 0; r < 32; r += 2, o += 2 * plane, src += 2 * kXposePitch)
                                if (r + row_sub < kmax) {
                                    float2 t = *reinterpret_cast<const float2*>(src);
                                    if (stacked) {
                                        const float2 u = *reinterpret_cast<const float2*>(src + 16 * kXposePitch);
                                        t.x += u.x; t.y += u.y;
                                    }
                                    if (add) { atomicAdd(o, t.x); atomicAdd(o + 1, t.y); }
                                    else *reinterpret_cast<float2*>(o) = t;
                                }
                        } else {
#pragma unroll 8
                            for (int r = 0; r < 32; ++r, o += plane, src += kXposePitch)
                                if (r < kmax) {
                                    const float t = stacked ? src[0] + src[16 * kXposePitch] : src[0];
                                    if (add) atomicAdd(o, t); else *o = t;
                                }
                        }
                    }
                };
                uint32_t va0[16], va1[16], vb0[16], vb1[16], vax[1], vbx[1];
                const int b_step = split ? 3 : 1;
                int b = split ? share : 0;
                if (b < blocks) load_block(va0, va1, vax, b);
                while (b < blocks) {
                    tmem_ld_wait();
                    if (b + b_step < blocks) load_block(vb0, vb1, vbx, b + b_step);
                    store_block(va0, va1, vax, b);
                    if ((b += b_step) >= blocks) break;
                    tmem_ld_wait();
                    if (b + b_step < blocks) load_block(va0, va1, vax, b + b_step);
                    store_block(vb0, vb1, vbx, b);
                    b += b_step;
                }
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0 && !helper) mbar_arrive(&acc_empty[buf]);
                continue;
            }
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
                    int n, p, q;
                    ok = output_pixel<PATCH>(a, ii.geom, m * kTileM + quarter * 32 + lane, n, p, q);
                    if (ok) yb = a.y + ((size_t)n * a.K * a.P + p) * a.Q + q;
                }
                const int k0 = nb * a.n_tile + ch * 16;
                if (ok) {
                    float* o = yb + (size_t)k0 * plane;
#pragma unroll
                    for (int i = 0; i < 16; ++i, o += plane)
                        if (k0 + i < a.K) { if (add) atomicAdd(o, __uint_as_float(v[i])); else *o = __uint_as_float(v[i]); }
                }
            };
            // Two register buffers: the load of the next chunk is in flight while the current one is stored.
            uint32_t va[16], vb[16];
            int c = 0;
            load_chunk(va, c);
            while (c < total_chunks) {
                tmem_ld_wait();
                if (c + 1 < total_chunks) load_chunk(vb, c + 1);
                store_chunk(va, c);
                if (++c >= total_chunks) break;
                tmem_ld_wait();
                if (c + 1 < total_chunks) load_chunk(va, c + 1);
                store_chunk(vb, c);
                ++c;
            }
            // all of this warp's reads of the accumulator set are complete: hand it back to the MMA thread
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[buf]);
        }
    }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, a.tmem_cols);
    if (tid == 0 && *abort_flag) atomicExch(a.status, 1u);
    if (tid == 0 && blockIdx.x == 0) {
        unsigned long long t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        a.status[8] = (unsigned)(t - *t_entry);                  // ns from kernel entry to the block's end
    }
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
    return kStatusBytes + packed_floats(p) * sizeof(float);
}

bool b16_supported(const Shape& sh)
{
    return make_plan(sh, true).ok;
}

size_t b16_workspace_bytes(const Shape& sh)
{
    const Plan p = make_plan(sh, true);
    if (!p.ok) return kStatusBytes;
    return kStatusBytes + packed_floats(p) * sizeof(float);
}

namespace {
// Launch with programmatic stream serialization: the kernel may be scheduled while the preceding kernel on the
// stream drains; it calls grid_dep_wait() before it touches global memory.
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args... args)
{
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = env_int("CONV2D_B200_TF32_PDL", 1) != 0 ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// workspace_bytes: checked against the plan's need here, so that a call plans only once (the planner reads two
// dozen environment switches and costs ~2 us); SIZE_MAX = the caller has checked already.
conv2d_status_t launch_tensor_core(const void* x_any, const void* w_any, float* y, const Shape& sh, bool b16, bool fp16,
                                   void* workspace, size_t workspace_bytes, bool weights_packed, cudaStream_t stream)
{
    const float* x = static_cast<const float*>(x_any);   // 16-bit operands: re-read as such inside the kernel
    const float* w = static_cast<const float*>(w_any);
    const Plan p = make_plan(sh, b16);
    if (!p.ok) return CONV2D_ERR_UNSUPPORTED;
    if (workspace_bytes < kStatusBytes + packed_floats(p) * sizeof(float)) return CONV2D_ERR_WORKSPACE;
    unsigned* status = static_cast<unsigned*>(workspace);
    float* wp = reinterpret_cast<float*>(static_cast<unsigned char*>(workspace) + kStatusBytes);

    if (!weights_packed) {
        const long long total = (long long)packed_floats(p);
        const FoldedFilter ff{sh.C, sh.R, sh.S, p.fold_r, p.fold_s};
        const long long lanes = total / p.taps * (b16 ? 2 : 1);      // one thread per element of a tap's slice
        long long blocks = (lanes + 255) / 256;
        if (blocks > 148 * 16) blocks = 148 * 16;
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
                p.taps, p.n_tile, p.cblks, lanes, p.pair_taps);
        else
            repack_filters_kernel<float, 4><<<(unsigned)blocks, 256, 0, stream>>>(w, wp, status, sh.K, ff, p.taps,
                                                                                  p.n_tile, p.cblks, lanes, p.pair_taps);
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
                                     general_tc_kernel<false, false, true, true>,   general_tc_kernel<true, false, true, true>};
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
    a.pair_taps = p.pair_taps; a.s_slots = p.s_slots; a.s_step = p.pair_taps ? 2 : 1; a.item_stride = p.tile_px - p.ovl;
    a.div_HW = FastDiv(a.HW); a.div_W = FastDiv(sh.W); a.div_npix = FastDiv(p.npix);
    a.div_qn = FastDiv(p.npix / 4 > 0 ? p.npix / 4 : 1); a.div_patch_w = FastDiv(p.patch_w ? p.patch_w : 1);
    a.helpers = (p.swap && (size_t)p.a_stages * p.cbg * kCB * chunk_stride(p.npix) * 4 >= 2 * kXposeBytes &&
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
    if (p.ksplit > 1 &&
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
    if (launch_pdl(kernel, dim3((unsigned)p.grid), dim3(kThreads), p.smem_bytes, stream, a) != cudaSuccess) return CONV2D_ERR_CUDA;
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
    conv2d_status_t st = launch_general_tf32(x, w, y, sh, scratch, kNoAllocScratchBytes, /*weights_packed=*/false, stream);
    if (st != CONV2D_OK || !wait) return st;
    if (cudaStreamSynchronize(stream) != cudaSuccess) return CONV2D_ERR_CUDA;
    unsigned word = 0;
    if (cudaMemcpy(&word, scratch, sizeof word, cudaMemcpyDeviceToHost) != cudaSuccess) return CONV2D_ERR_CUDA;
    return word == 0 ? CONV2D_OK : CONV2D_ERR_DEVICE_TIMEOUT;
}

}  // namespace conv2d_b200
