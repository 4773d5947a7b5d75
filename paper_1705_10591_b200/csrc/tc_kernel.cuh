// Tensor-core convolution: the persistent kernel (filter copies, MMA issue, producers, epilogue) and its device
// helpers.  The design is described at the top of general_tf32.cu.  Included by general_tf32.cu only.
#pragma once
#include "tc_plan.cuh"
#include "ptx.cuh"
#include "fastdiv.cuh"

namespace conv2d_b200 {
namespace {


using namespace ptx;

// Tuning builds (-DCONV2D_B200_TC_DIAGNOSTICS) make the MMA-issuing thread of block 0 count its cycles and leave
// them in status words 2-9.  The product build contains none of it: that thread's instruction stream is what
// bounds the heavy shapes, and a timer read with a memory clobber around every wait is not free.
#ifdef CONV2D_B200_TC_DIAGNOSTICS
constexpr bool kDiag = true;
#else
constexpr bool kDiag = false;
#endif
// Cycle counter read that the compiler may not move across memory operations or barriers (0 in product builds).
__device__ __forceinline__ long long clock_now()
{
    long long t = 0;
    if (kDiag) asm volatile("mov.u64 %0, %%clock64;" : "=l"(t) :: "memory");
    return t;
}
__device__ __forceinline__ unsigned long long wall_ns()
{
    unsigned long long t = 0;
    if (kDiag) asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

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
    int pair_compact;       // stacked taps, resident bank: the odd last tap of a filter row is a 64-row slice of its own,
                            // issued as an M = 64 MMA onto the same accumulator lanes (no zero-padded upper half)
    int cb_bytes;           // resident filters: bytes of one channel block of the bank (all taps)
    int item_stride;        // flat addressing: pixels between the starts of consecutive items (tile_px minus the overlap)
    int ksplit;             // items per output tile (split of the contraction): 1 or 2
    int xchg_slots;         // cluster instances: 32-pixel blocks each block of a pair receives from its peer
    int xchg_bytes;         // ... and the bytes of the exchange area (rows + barriers) behind the transposition tiles
    unsigned max_polls;     // bound of every barrier wait
    int test_drop_stage;    // test hook: the filter copy with this ordinal is armed but never issued (-1: none)
    int early_x;            // 1: this call's filter re-ordering kernel directly precedes on the stream, so the image is
                            // final already and the producers need not wait for that kernel
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

// CLUSTER: the two work items of a split contraction (ksplit = 2) run as a two-block cluster, one item per block.
// Each block stores every other 32-pixel block of the tile: it sends its partial sums of the peer's blocks into the
// peer's shared memory (distributed shared memory, plain stores) and adds what the peer sent to its own
// accumulators before the ordinary write-back.  No zero-fill of y, no atomic adds, and a + b = b + a keeps the
// result independent of timing.
template <bool B16, bool FOLD, bool PATCH, bool STACK, bool CLUSTER = false>
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
    const size_t b_region_bytes = a.resident ? (size_t)a.cblks * a.cb_bytes : (size_t)a.b_stages * b_stage_bytes;
    float* xpose = reinterpret_cast<float*>(b_smem + b_region_bytes);            // only present (and used) when a.swap
    unsigned char* after_xpose = b_smem + b_region_bytes + (a.swap ? kXposeBytes : 0);
    float* xchg = reinterpret_cast<float*>(after_xpose);     // CLUSTER: [4 quarters][xchg_slots][8 column groups][32 lanes][4 floats] partial sums from the peer
    uint64_t* xbar = reinterpret_cast<uint64_t*>(after_xpose + (size_t)kEpilogueWarps * a.xchg_slots * kXchgBlockFloats * 4);   // [4][xchg_slots]
    uint64_t* bars = reinterpret_cast<uint64_t*>(after_xpose + (CLUSTER ? a.xchg_bytes : 0));
    uint64_t* a_full = bars;                               // [kMaxAStages]
    uint64_t* a_empty = a_full + kMaxAStages;              // [kMaxAStages]
    uint64_t* b_full = a_empty + kMaxAStages;              // [kMaxBStages]
    uint64_t* b_empty = b_full + kMaxBStages;              // [kMaxBStages]
    uint64_t* acc_full = b_empty + kMaxBStages;            // [2]
    uint64_t* acc_empty = acc_full + 2;                    // [2]
    uint64_t* tail_full = acc_empty + 2;                   // [1] the block's last item is complete (for warps 8-15)
    uint64_t* drain_bar = tail_full + 1;                   // [1] time-out path only: the MMAs issued so far have completed
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(drain_bar + 1);
    volatile uint32_t* abort_flag = tmem_slot + 1;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    volatile unsigned long long* t_entry = reinterpret_cast<volatile unsigned long long*>(tmem_slot + 2);
    uint32_t* tap_shift = tmem_slot + 4;                   // [taps] r * row_pitch + s of every tap, in staged pixels
    // (bit 31: the slot is a lone tap held as a 64-row slice, see pair_compact)
    for (int t = tid; t < a.taps; t += kThreads)
        tap_shift[t] = (uint32_t)((t / a.s_slots) * a.row_pitch + (t % a.s_slots) * a.s_step) |
                       ((a.pair_compact && (a.S & 1) && t % a.s_slots == a.s_slots - 1) ? 0x80000000u : 0u);
    if (kDiag && tid == 0) *t_entry = wall_ns();

    if (tid == 0) {
        for (int i = 0; i < a.a_stages; ++i) { mbar_init(&a_full[i], kProducers / a.pgroups); mbar_init(&a_empty[i], 1); }
        for (int i = 0; i < a.b_stages; ++i) { mbar_init(&b_full[i], 1); mbar_init(&b_empty[i], 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(&acc_full[i], 1); mbar_init(&acc_empty[i], kEpilogueWarps); }
        mbar_init(tail_full, 1);
        mbar_init(drain_bar, 1);
        if (CLUSTER)
            for (int i = 0; i < kEpilogueWarps * a.xchg_slots; ++i) mbar_init(&xbar[i], 32);
        *abort_flag = 0;
        fence_mbar_init();
    }
    __syncthreads();
    if (CLUSTER) cluster_sync_all();        // the peer's barriers exist before anything can arrive on them
    if (warp == 1) { tmem_alloc(tmem_slot, a.tmem_cols); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = *tmem_slot;
    // Everything above touched only this block's shared and tensor memory; it may overlap the tail of the
    // preceding kernel on the stream (the filter re-ordering of this call, or the previous call).  From here
    // on global memory is read and written: every role waits for the preceding kernel first, except that the
    // producers go ahead when that kernel is this call's own filter re-ordering.  It was launched the ordinary way,
    // so everything before it on the stream had finished when it started, it does not touch the image, and the
    // image is read only: the first activation stages are then in flight while the filters are still being written.
    grid_dep_launch();
    if (!(a.early_x && producer_index(warp) >= 0)) grid_dep_wait();

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
                const uint32_t piece = (uint32_t)a.cb_bytes;
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
            // (the start-address field of a descriptor holds bits 4-17 of the shared-memory address; the address of a
            // block that is not the first of its cluster has bits above those set, which must not leak into LBO)
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
            if (kDiag && blockIdx.x == 0) a.status[6] = (unsigned)(wall_ns() - *t_entry);   // ns from kernel entry to the start of the MMA loop
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
                    uint32_t a_lo_block = a_lo_fixed | ((smem_u32(a_smem + (size_t)as * a_stage_bytes) >> 4) & 0x3FFFu);
                    for (int g = 0; g < a.cbg && alive; ++g, a_lo_block += a_block_bytes >> 4) {
                        if (gr * a.cbg + g >= a.cblks) break;
                        uint32_t row_shift = 0;                                  // r * row pitch, in pixels (= 16-byte units)
                        int sx = 0, sc = 0;
                        for (int t0 = 0; t0 < a.taps; t0 += a.tps) {
                            const int nt = min(a.tps, a.taps - t0);
                            uint32_t b_lo;
                            if (a.resident) {
                                b_lo = b_lo_fixed | ((smem_u32(b_smem + (size_t)(gr * a.cbg + g) * a.cb_bytes) >> 4) & 0x3FFFu);
                            } else {
                                if (!mbar_wait_bounded(&b_full[bs], b_phase, abort_flag, a.max_polls)) { alive = false; break; }
                                tc_fence_after_sync();
                                b_lo = b_lo_fixed | ((smem_u32(b_smem + (size_t)bs * b_stage_bytes) >> 4) & 0x3FFFu);
                            }
                            if (a.swap && a.px_groups == 1) {
                                // M operand = the 128 filters of this stage, N operand = n_mma staged pixels.
                                // One MMA pair per tap carries less tensor-pipe work than this one thread needs to
                                // issue it with loop and address arithmetic around it (~230 cycles per MMA that
                                // way), so a tap is one block of straight-line code and its shift comes from a
                                // table, fetched one tap ahead.
                                const uint32_t* shift = tap_shift + t0;
                                uint32_t cur = shift[0];
                                if (STACK && a.pair_compact) {
                                    // pairs of taps as M = 128 slices, a lone last tap as an M = 64 slice of half the size
                                    // (its chunk stride and K step are half as long too) onto the same accumulator lanes
                                    const uint32_t idesc64 = B16 ? idesc_b16(64u, n_cols, a.fp16 != 0) : idesc_tf32(64u, n_cols);
                                    for (int t = 0; t < nt; ++t) {
                                        const uint32_t a_lo = a_lo_block + (cur & 0x7FFFFFFFu);
                                        const bool lone = (cur >> 31) != 0u;
                                        cur = shift[t + 1 < nt ? t + 1 : t];
                                        if (lone) {
                                            issue_tap<B16, 1>(d0, a_lo, b_lo - (64u << 16), a_kstep, b_kstep >> 1, n_mma, desc_hi, idesc64, accumulate);
                                            b_lo += b_chunk_bytes >> 5;
                                        } else {
                                            issue_tap<B16, 1>(d0, a_lo, b_lo, a_kstep, b_kstep, n_mma, desc_hi, idesc, accumulate);
                                            b_lo += b_chunk_bytes >> 4;
                                        }
                                        accumulate = 1;
                                    }
                                } else
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
            if (!alive) {
                // A wait ran out: MMAs issued before that may still be reading shared memory and writing tensor
                // memory.  Let them finish (bounded) before the block frees its tensor memory and exits.
                mma_commit(drain_bar);
                uint32_t dummy = 0;
                mbar_wait_bounded(drain_bar, 0u, &dummy, 1u << 16);
            }
            if (kDiag && blockIdx.x == 0) {
                a.status[2] = (unsigned)wait_a;
                a.status[3] = (unsigned)wait_acc;
                a.status[4] = (unsigned)(clock_now() - t_begin);
                a.status[5] = (unsigned)n_items;
                a.status[9] = (unsigned)issue_cycles;
                a.status[7] = (unsigned)(wall_ns() - *t_entry);  // ns from kernel entry to the last MMA issued
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
            const bool add = !CLUSTER && a.ksplit > 1;       // partial sums: add into the zeroed output
            // tcgen05.ld is warp-collective: take the decision for the whole warp
            // (warps 8-15 come late and only for the last item: they wait on a barrier of its own, whose
            // phase they cannot have missed)
            const long long t_wait0 = clock_now();
            alive = __all_sync(0xffffffffu, alive && mbar_wait_bounded(helper ? tail_full : &acc_full[buf],
                                                                       helper ? 0u : acc_phase, abort_flag, a.max_polls));
            if (!alive) break;
            tc_fence_after_sync();
            const long long t_busy0 = clock_now();
            if (kDiag && blockIdx.x == 0 && warp == 4 && lane == 0) a.status[10] += (unsigned)(t_busy0 - t_wait0);   // waited for accumulators
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
                if (CLUSTER) {
                    const uint32_t rank = cluster_ctarank(), peer = rank ^ 1u;
                    // rows and barriers belong to a (lane quarter, block) pair; with the helper warps a quarter is
                    // drained by three warps, block b going to warp (b / 2) mod 3 of the quarter on both sides
                    float* my_rows = xchg + (size_t)quarter * a.xchg_slots * kXchgBlockFloats;
                    uint64_t* my_bars = xbar + quarter * a.xchg_slots;
                    const int nshare = a.helpers ? 3 : 1;
                    uint32_t v0[16], v1[16], vx[1];
                    vx[0] = 0u;
                    // the blocks the peer stores: this block's partial sums go into the peer's shared memory as
                    // [4-column group][lane][16 bytes], so that one store instruction of the warp writes 512 contiguous
                    // bytes over the cluster network (a row per lane, i.e. 16-byte pieces 144 bytes apart, took 2150 cycles
                    // per 32-pixel block, this layout 1290)
                    const long long t_x0 = clock_now();
                    long long t_xwait = 0;
                    for (int b = (int)peer; b < blocks; b += 2) {
                        if ((b >> 1) % nshare != share) continue;
                        tmem_ld16(lane_base + (uint32_t)(b * 32), v0);
                        tmem_ld16(lane_base + (uint32_t)(b * 32 + 16), v1);
                        tmem_ld_wait();
                        const int slot = b >> 1;
                        const uint32_t dst = map_to_cta(smem_u32(my_rows + (size_t)slot * kXchgBlockFloats + lane * 4), peer);
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            st_cluster_v4(dst + 512u * i, __uint_as_float(v0[4 * i]), __uint_as_float(v0[4 * i + 1]),
                                          __uint_as_float(v0[4 * i + 2]), __uint_as_float(v0[4 * i + 3]));
                            st_cluster_v4(dst + 2048u + 512u * i, __uint_as_float(v1[4 * i]), __uint_as_float(v1[4 * i + 1]),
                                          __uint_as_float(v1[4 * i + 2]), __uint_as_float(v1[4 * i + 3]));
                        }
                    }
                    // The arrivals come after the stores of all blocks (measured: the same time as arriving block by
                    // block, ~1290 cycles per block either way: the remote stores themselves, ~150 cycles per 512-byte
                    // instruction, are the cost; one arrival per warp behind a cluster-scope fence measured slower).
                    for (int b = (int)peer; b < blocks; b += 2) {
                        if ((b >> 1) % nshare != share) continue;
                        mbar_arrive_remote(map_to_cta(smem_u32(&my_bars[b >> 1]), peer));
                    }
                    const long long t_x1 = clock_now();
                    // this block's own blocks: accumulators + the peer's partial sums, then the ordinary write-back
                    for (int b = (int)rank; b < blocks; b += 2) {
                        if ((b >> 1) % nshare != share) continue;
                        tmem_ld16(lane_base + (uint32_t)(b * 32), v0);
                        tmem_ld16(lane_base + (uint32_t)(b * 32 + 16), v1);
                        tmem_ld_wait();
                        const int slot = b >> 1;
                        const long long t_w0 = clock_now();
                        alive = __all_sync(0xffffffffu, mbar_wait_bounded_cluster(&my_bars[slot], 0u, abort_flag, a.max_polls));
                        t_xwait += clock_now() - t_w0;
                        if (!alive) break;
                        const float4* row = reinterpret_cast<const float4*>(my_rows + (size_t)slot * kXchgBlockFloats) + lane;
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const float4 t = row[32 * i], u = row[128 + 32 * i];
                            v0[4 * i] = __float_as_uint(__uint_as_float(v0[4 * i]) + t.x);
                            v0[4 * i + 1] = __float_as_uint(__uint_as_float(v0[4 * i + 1]) + t.y);
                            v0[4 * i + 2] = __float_as_uint(__uint_as_float(v0[4 * i + 2]) + t.z);
                            v0[4 * i + 3] = __float_as_uint(__uint_as_float(v0[4 * i + 3]) + t.w);
                            v1[4 * i] = __float_as_uint(__uint_as_float(v1[4 * i]) + u.x);
                            v1[4 * i + 1] = __float_as_uint(__uint_as_float(v1[4 * i + 1]) + u.y);
                            v1[4 * i + 2] = __float_as_uint(__uint_as_float(v1[4 * i + 2]) + u.z);
                            v1[4 * i + 3] = __float_as_uint(__uint_as_float(v1[4 * i + 3]) + u.w);
                        }
                        store_block(v0, v1, vx, b);
                    }
                    if (!alive) break;
                    if (kDiag && blockIdx.x == 0 && warp == 4 && lane == 0) {     // cycles: sending, waiting for the peer, whole exchange
                        a.status[13] = (unsigned)(t_x1 - t_x0);
                        a.status[14] = (unsigned)t_xwait;
                        a.status[15] = (unsigned)(clock_now() - t_x0);
                    }
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0 && !helper) mbar_arrive(&acc_empty[buf]);
                    continue;
                }
                uint32_t va0[16], va1[16], vb0[16], vb1[16], vax[1], vbx[1];
                const int b_step = split ? 3 : 1;
                int b = split ? share : 0;
                if (b < blocks) load_block(va0, va1, vax, b);
                long long t_ld = 0;       // (diagnostics build: cycles spent waiting for tensor-memory loads)
                while (b < blocks) {
                    long long t0 = clock_now();
                    tmem_ld_wait();
                    t_ld += clock_now() - t0;
                    if (b + b_step < blocks) load_block(vb0, vb1, vbx, b + b_step);
                    store_block(va0, va1, vax, b);
                    if ((b += b_step) >= blocks) break;
                    t0 = clock_now();
                    tmem_ld_wait();
                    t_ld += clock_now() - t0;
                    if (b + b_step < blocks) load_block(va0, va1, vax, b + b_step);
                    store_block(vb0, vb1, vbx, b);
                    b += b_step;
                }
                if (kDiag && blockIdx.x == 0 && warp == 4 && lane == 0) a.status[12] += (unsigned)t_ld;
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0 && !helper) mbar_arrive(&acc_empty[buf]);
                if (kDiag && blockIdx.x == 0 && warp == 4 && lane == 0) a.status[11] += (unsigned)(clock_now() - t_busy0);   // drained one item
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
    // (a block must not exit while its peer may still write into its shared memory or arrive on its barriers)
    if (CLUSTER) cluster_sync_all();
    if (warp == 1) tmem_dealloc(tmem, a.tmem_cols);
    if (tid == 0 && *abort_flag) atomicExch(a.status, 1u);
    if (kDiag && tid == 0 && blockIdx.x == 0) a.status[8] = (unsigned)(wall_ns() - *t_entry);   // ns from kernel entry to the block's end
}

}  // namespace
}  // namespace conv2d_b200
