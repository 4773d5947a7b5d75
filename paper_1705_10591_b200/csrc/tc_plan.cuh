// Tensor-core convolution, host side: tile and stage sizes, and the planner that picks operand roles, addressing
// mode, item size, filter residency and the split of the contraction for a shape.  Included by general_tf32.cu only.
#pragma once
#include <cstdlib>

#include "common.cuh"

namespace conv2d_b200 {
namespace {

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
constexpr int kXchgBlockFloats = 32 * 32;   // exchange area of a two-block cluster: one 32-filter x 32-pixel block of partial sums
// bytes of that area for `slots` 32-pixel blocks per lane quarter: blocks, then one barrier per (quarter, slot)
constexpr size_t xchg_area_bytes(int slots) { return (size_t)kEpilogueWarps * slots * (kXchgBlockFloats * 4 + 8); }

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
    int pair_compact; // 1 (with pair_taps): a lone last tap of a filter row is a 64-row slice issued as M = 64 (resident bank only)
    size_t cb_bytes;  // bytes of one channel block of the re-ordered bank (all taps of one filter block)
    int s_slots;      // shift-table entries per filter row: S, or ceil(S / 2) with stacked taps
    int ovl;          // pixels by which consecutive flat items overlap (4 with stacked taps, else 0)
    int ksplit;       // 2: the channel blocks of a tile are shared by two work items that add into y
    int cluster;      // 1 (with ksplit = 2): the two items run as a two-block cluster and exchange partial sums on chip
    int xchg_slots;   // ... 32-pixel blocks each of them receives
    int tmem_cols;    // power of two >= 32
    int supertiles;   // work-item rows over the flat pixel sequence
    int grid;
    size_t smem_bytes;
    double makespan;  // MMA work of the busiest block, in item pixels x taps x channel blocks (to compare patch widths)
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
Plan plan_with_patch_width(const Shape& sh, bool b16, int want_patch_w, bool allow_compact = true)
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
    // Compact stacking for banks that can stay in shared memory: pairs of taps as 128-row slices, the lone last tap of
    // an odd filter row as a 64-row slice that an M = 64 instruction adds onto the same accumulator lanes.  The bank
    // is then as large as the unstacked one, so a short contraction keeps its resident filters and still issues two
    // instructions per three taps instead of three at half rate (64 filters of 64 x 3 x 3 on 56 x 56 images).
    // Measured on that shape: the MMA thread's issue time per 256-pixel item falls from 9.4k to 7.4k cycles, but the
    // four write-back warps need 10.4k cycles for the item (8.9k unstacked: every map is the sum of two tile rows), and
    // with two accumulator sets the slower of the two sets the pace: 36.5 -> 39.4 us.  Off by default
    // (CONV2D_B200_TF32_PAIR_COMPACT = 1 turns it on) until the write-back is faster than the MMAs.
    p.pair_compact = 0;
    const size_t compact_cb_bytes = (size_t)r_eff * ((s_eff / 2) * 128 + (s_eff & 1) * 64) * kCB * 4;
    if (allow_compact && !p.pair_taps && p.swap && kp16 <= 64 && p.fold_r * p.fold_s == 1 && s_eff >= 2 && pair_mode != 0 &&
        !padded && (size_t)((c_eff + cbc - 1) / cbc) * compact_cb_bytes <= 152 * 1024 && env_int("CONV2D_B200_TF32_PAIR_COMPACT", 0) != 0) {
        p.pair_taps = 1;
        p.pair_compact = 1;
    }
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
        const int forced_wp = want_patch_w ? want_patch_w : env_int("CONV2D_B200_TF32_PATCH_W", 0);
        for (int wp = 32; wp <= 128; wp *= 2) {
            const int tw = (wp - (s_eff - 1)) / 4 * 4;
            if (tw < 4 || (forced_wp && wp != forced_wp)) continue;
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
    const int sms = sm_count();

    const int forced_mt = env_int("CONV2D_B200_TF32_MT", 0);      // benchmark ablations only
    p.cb_bytes = p.pair_compact ? compact_cb_bytes : (size_t)p.taps * chunk;
    const size_t wbytes = (size_t)p.cblks * p.cb_bytes;            // re-ordered filters of one filter block
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
            // (compact stacking issues one MMA per K step: at most 256 pixels per item)
            const long long one_round = ((total_pix + sms - 1) / sms + p.ovl + 31) / 32 * 32;
            if (one_round >= 64 && one_round <= (p.pair_compact ? 256 : 512)) res_px = (int)one_round;
        }
        {
            const int want = env_int("CONV2D_B200_TF32_TILE_PX", 0);
            if (p.swap && want >= 64 && want <= (p.pair_compact ? 256 : 512) && want % 32 == 0 && pixel_items(want) > 0) res_px = want;
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

    if (p.pair_compact && !p.resident) return plan_with_patch_width(sh, b16, want_patch_w, false);    // compact stacking needs the resident bank
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
                // With one accumulator set the MMAs of an item wait for the whole write-back of the item before it
                // (four warps, measured ~2000 cycles per 32-pixel block of 128 maps, ~1200 of 64); from the third round
                // of items on that outweighs the wider MMAs (64 x 64 x 56 x 56 -> 128 maps, 3 x 3: 480-pixel items
                // 69.1 us, 256-pixel items with two accumulator sets 64.6 us).
                if (nbuf == 1 && rounds >= 3)
                    cost += (double)(rounds - 2) * 0.75 * (px / 32.0) * (p.n_tile >= 128 ? 2000.0 : 1200.0);
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
        // equal stages: 6 taps as 3 + 3 instead of 5 + 1 (the short stage's MMAs would end long before the next
        // long stage has arrived)
        {
            const int per_block = (p.taps + p.tps - 1) / p.tps;
            p.tps = (p.taps + per_block - 1) / per_block;
        }
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
    if (p.pair_compact) p.px_groups = 1;
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
    // The split contraction as a two-block cluster: needs room for the exchange area behind the transposition tiles
    // (the filter ring gives up stages for it, down to two) and one item per block.
    p.cluster = 0;
    p.xchg_slots = 0;
    if (p.ksplit == 2 && p.swap && !p.patch_w && !p.pair_taps && p.fold_r * p.fold_s == 1 && p.n_tile == 128 && !p.resident &&
        items <= sms && env_int("CONV2D_B200_TF32_KSPLIT_CLUSTER", 1) != 0) {
        const int slots = (p.tile_px / 32 + 1) / 2;
        const size_t xb = xchg_area_bytes(slots);
        int bs = p.b_stages;
        while (bs > 2 && smem_need(p.a_stages, p.npix, p.n_tile, bs, p.tps, p.cbg) + extra + xb > kSmemLimit) --bs;
        if (smem_need(p.a_stages, p.npix, p.n_tile, bs, p.tps, p.cbg) + extra + xb <= kSmemLimit) {
            p.cluster = 1;
            p.xchg_slots = slots;
            p.b_stages = bs;
            p.smem_bytes = smem_need(p.a_stages, p.npix, p.n_tile, bs, p.tps, p.cbg) + extra + xb;
        }
    }
    int cols = p.nbuf * item_cols;
    p.tmem_cols = 32;
    while (p.tmem_cols < cols) p.tmem_cols <<= 1;
    p.makespan = (double)((items + sms - 1) / sms) * p.tile_px * p.taps * p.cblks;
    p.ok = true;
    return p;
}

// The patch width with the fewest staged pixels per output is the first choice.  A wider patch has a larger valid
// fraction (fewer MMA columns that only feed the next patch) and may need fewer rounds of items over the SMs: it is
// taken when the busiest block then has at least 5 % less MMA work (7 x 7 on 224 x 224, 64 -> 128 channels: 73 -> 61
// us with 64-column patches; 3 x 3 on 512 x 512: 101 -> 92 us; but 7 x 7 on 256 x 256: 196 us with 32 columns, 209 with 64,
// where both take two rounds of equal items).
Plan make_plan(const Shape& sh, bool b16 = false)
{
    Plan best = plan_with_patch_width(sh, b16, 0);
    if (!best.ok || !best.patch_w || env_int("CONV2D_B200_TF32_PATCH_W", 0) != 0) return best;
    const int first = best.patch_w;
    for (int wp = 32; wp <= 128; wp *= 2) {
        if (wp == first) continue;
        const Plan q = plan_with_patch_width(sh, b16, wp);
        if (q.ok && q.patch_w == wp && q.makespan < 0.95 * best.makespan) best = q;
    }
    return best;
}

size_t packed_floats(const Plan& p)
{
    return (size_t)p.n_blocks * p.cblks * (p.cb_bytes / 4);
}

}  // namespace
}  // namespace conv2d_b200
