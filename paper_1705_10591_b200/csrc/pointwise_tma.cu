// General case with 1 x 1 filters on the tcgen05 tensor cores (fp32 inputs as TF32, or bf16 / fp16 inputs), every
// operand and the output moved by tiled TMA
// copies (the staging and the prefetch of Algorithm 2, lines 4-5 and 8-9, done by the copy engine; its write-back,
// line 20, as well).
//
// With one tap per filter the convolution of image n is the matrix product
//     Y[n] (K x HW) = Wmat (K x C) * X[n] (C x HW),
// and both operands already lie in memory the way the tensor core can read them, so nothing has to be turned
// around by threads:
//   * Filters, the M operand: w[k][c] has the channels contiguous = K-major.  A tensor-map copy with a 32-channel
//     (128-byte) inner box and 128-byte swizzle writes exactly the 8-row x 128-byte atoms the MMA reads; the whole
//     bank of a filter block (up to 128 filters x 256 channels) stays in shared memory for the life of the block
//     (Section 3.2: the filters are small, keep them on chip).
//   * Pixels, the N operand: NCHW has the pixels of a channel contiguous = MN-major, which kind::tf32 accepts in one
//     layout only: 128-byte rows (32 pixels of one channel) whose 32-byte chunks are swizzled over groups of 4
//     channel rows, as a tensor-map copy with SWIZZLE_128B_ATOM_32B writes them.  One box of 32 pixels x 32 channels
//     serves four K steps of 8 channels; an MMA covers up to 8 such boxes (N <= 256) that lie 32 * 128 bytes apart.
//     A stage of the mbarrier ring holds 32 channels of all pixels of a work item.
//   * Output: accumulators (lanes = filters, columns = pixels) go tensor memory -> registers -> a swizzled
//     32-filter x 32-pixel shared-memory tile per warp -> one tensor-map store per tile.  Out-of-range rows and
//     pixels are clipped by the copy engine, so ragged images and filter counts need no predicates.
// (16-bit operands: 64 pixels or channels per 128-byte row, K steps of 16, the ordinary 128-byte swizzle on both operands.)
// The tensor core reads fp32 bits as TF32 by dropping the low 13 mantissa bits, so on this path both operands are
// truncated, not rounded: |error| <= (2^-10 + 2^-10 + 2^-20) * sum|x*w| plus fp32 accumulation over at most 256
// channels, (C + 1) * 2^-24 * sum|x*w|: below 1.97e-3 * sum|x*w|, inside the 2e-3 bound of CONV2D_ALGO_TF32.
//
// Persistent blocks, one per SM: warp 0 (one thread) issues the loads, warp 1 (one thread) the MMAs, warps 2-9
// drain the accumulators, two per tensor-memory lane quarter.  Two accumulator sets: the write-back of item i runs
// under the loads and MMAs of item i + 1, which is what an operation bound by memory traffic needs.
// Work items are runs of `a_item` 32-pixel atoms of the flat atom sequence (image-major; an image has
// ceil(HW / 32) atoms, the last one may be ragged and is zero-filled on load and clipped on store).
// Every wait is bounded; on expiry the block stops, frees its tensor memory and raises the status word.
#include <algorithm>
#include <cstdio>
#include <cuda.h>

#include "common.cuh"
#include "fastdiv.cuh"
#include "ptx.cuh"

namespace conv2d_b200 {
namespace {

using namespace ptx;

constexpr int kPwThreads = 320;           // warp 0: loads, warp 1: MMAs, warps 2-9: write-back
constexpr int kPwEpiWarps = 8;
constexpr int kPwMaxStages = 8;
constexpr int kAccCols = 256;             // tensor-memory columns of one accumulator set
constexpr int kMaxChunks = 8;             // 128-byte channel chunks of the resident filter bank (at most 128 KB)

// Sizes that depend on the operand type: fp32 (read by the tensor core as TF32) or a 16-bit float.  A 128-byte row
// holds 32 or 64 elements; a stage holds four K steps (of 8 or 16 channels) for all pixels of a work item.
template <bool B16>
struct Geom {
    static constexpr int kElem = B16 ? 2 : 4;
    static constexpr int kAtomPx = 128 / kElem;            // pixels per 128-byte row of a swizzle atom
    static constexpr int kKStep = B16 ? 16 : 8;            // channels per MMA
    static constexpr int kStageCh = 4 * kKStep;            // channels per activation stage = per 128-byte filter row
    static constexpr int kAtomBytes = 128 * kStageCh;      // one box of kAtomPx pixels x kStageCh channels
    static constexpr int kMaxAtoms = kAccCols / kAtomPx;   // atoms per work item: N <= 256 columns per MMA
};
constexpr size_t kPwSmemLimit = 227 * 1024;
constexpr size_t kPwBookBytes = 512;      // barriers, tensor-memory slot, abort flag
constexpr double kPwPairBias = 1.03;      // planner: the two-SM form is taken when its estimate is at least 3 % shorter
constexpr int kPwMaxStreamChannels = 8192;  // streamed filters: keeps the fp32 accumulation term of the error bound small

// Tensor maps over the image as (pixel in atom, channel, atom, image) whose boxes hold 1 .. 8 atoms: box i + 1 atoms.
struct XMaps { CUtensorMap m[8]; };

struct PwArgs {
    unsigned* status;
    int K;
    int fp16;            // 16-bit operands only: 1 = IEEE half, 0 = bf16
    int apb;             // atoms per image: ceil(HW / pixels per atom)
    int total_atoms;     // N * apb
    int a_item;          // atoms per work item
    int tiles;           // work items along the pixels
    int n_blocks;        // filter blocks of m_rows filters
    int m_rows;          // rows of the M operand: 64 (at most 64 filters) or 128
    int items;           // tiles * n_blocks, numbered filter block-major
    int cchunks;         // channel chunks of one stage each: ceil(C / channels per stage)
    int ksplit;          // 1, or 2: the channel chunks of a tile are shared out to two work items that both add into a zeroed y
    int cpart;           // channel chunks per work item: ceil(cchunks / ksplit)
    int ksteps;          // K steps: ceil(C / channels per MMA)
    int stages;          // activation ring depth
    int stream_a;        // 1: too many channels for a resident bank; every ring stage carries its filter chunk too
    int multi;           // 1: H*W is a whole number of atoms: one copy brings all atoms of an item that lie in one image
    int wide;            // pairs only: an item spans two MMA widths of pixels and uses both accumulator sets at once, so
                         // that a filter chunk serves twice the pixels (no write-back under the next item's MMAs then)
    unsigned max_polls;  // bound of every barrier wait
    int test_drop_stage; // test hook: the activation stage with this ordinal is armed but never copied (-1: none)
    FastDiv div_apb, div_tiles, div_nb;
};

// The copy, allocation, MMA and commit instructions of the one-SM and of the two-SM (cta_group::2) form.
template <bool PAIR>
struct Ops {
    // `bar`: shared::cluster address of the barrier that collects the bytes (a barrier of the pair's first block, PAIR)
    static __device__ __forceinline__ void load_2d(void* dst, const void* map, int c0, int c1, uint32_t bar)
    {
        if (PAIR) tma_load_2d_pair(dst, map, c0, c1, bar); else tma_load_2d(dst, map, c0, c1, bar);
    }
    static __device__ __forceinline__ void load_3d(void* dst, const void* map, int c0, int c1, int c2, uint32_t bar)
    {
        if (PAIR) tma_load_3d_pair(dst, map, c0, c1, c2, bar); else tma_load_3d(dst, map, c0, c1, c2, bar);
    }
    static __device__ __forceinline__ void load_4d(void* dst, const void* map, int c0, int c1, int c2, int c3, uint32_t bar)
    {
        if (PAIR) tma_load_4d_pair(dst, map, c0, c1, c2, c3, bar); else tma_load_4d(dst, map, c0, c1, c2, c3, bar);
    }
    static __device__ __forceinline__ void alloc(uint32_t* slot, uint32_t cols)
    {
        if (PAIR) { tmem_alloc_pair(slot, cols); tmem_relinquish_pair(); } else { tmem_alloc(slot, cols); tmem_relinquish(); }
    }
    static __device__ __forceinline__ void dealloc(uint32_t taddr, uint32_t cols)
    {
        if (PAIR) tmem_dealloc_pair(taddr, cols); else tmem_dealloc(taddr, cols);
    }
    template <bool B16>
    static __device__ __forceinline__ void mma(uint32_t d, uint64_t ad, uint64_t bd, uint32_t idesc, bool accumulate)
    {
        if (PAIR) { if (B16) mma_b16_pair(d, ad, bd, idesc, accumulate); else mma_tf32_pair(d, ad, bd, idesc, accumulate); }
        else { if (B16) mma_b16(d, ad, bd, idesc, accumulate); else mma_tf32(d, ad, bd, idesc, accumulate); }
    }
    // arrives on `bar` (of both blocks of a pair) when the MMAs issued so far have completed
    static __device__ __forceinline__ void commit(uint64_t* bar) { if (PAIR) mma_commit_pair_both(bar); else mma_commit(bar); }
    static __device__ __forceinline__ void commit_local(uint64_t* bar) { if (PAIR) mma_commit_pair(bar); else mma_commit(bar); }
};

// PAIR = false: one block per work item (a pixel tile x one block of `m_rows` filters).
// PAIR = true (more than 128 filters): the two blocks of a cluster work as a pair on 256 filters x `a_item` atoms of
// pixels with two-SM MMAs (cta_group::2, M = 256).  Block r of the pair holds filter block 2 * pair + r (its 128 rows
// of the M operand) and the r-th half of the item's pixels (its half of the N operand), so every byte of the image is
// fetched once per 256 filters instead of once per 128, and each SM's tensor core reads half of the pixel operand
// from its own shared memory.  The first block issues the MMAs; its `full` barriers collect the bytes of both
// blocks' copies, its commits arrive on the `empty` / `acc_full` barriers of both blocks, and the write-back warps
// of both blocks (each drains its own 128 accumulator lanes) arrive on its `acc_empty` barriers.  A pair's items
// always span `a_item` atoms: atoms past the end of the batch are zero-filled by the loads and skipped by the stores.
template <bool B16, bool PAIR>
__global__ void __launch_bounds__(kPwThreads, 1)
pointwise_tma_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_x,
                     const __grid_constant__ CUtensorMap map_y, const __grid_constant__ XMaps maps_x, const PwArgs a)
{
    using G = Geom<B16>;
    using Op = Ops<PAIR>;
    constexpr int kAtomPx = G::kAtomPx, kStageCh = G::kStageCh, kAtomBytes = G::kAtomBytes;
    constexpr uint32_t kBlocks = PAIR ? 2u : 1u;                              // blocks that work on one item
    extern __shared__ unsigned char smem_raw[];
    // swizzle atoms must start on 1024 bytes
    unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    const bool stream_a = a.stream_a != 0;
    const int my_atoms_max = PAIR ? a.a_item >> 1 : a.a_item;                 // atoms this block loads per stage
    const uint32_t a_chunk_bytes = (uint32_t)a.m_rows * 128u;                 // filters x 32 channels
    const uint32_t b_off = stream_a ? a_chunk_bytes : 0u;                     // a stage: [its filter chunk,] the pixel boxes
    const uint32_t b_stage_bytes = b_off + (uint32_t)my_atoms_max * kAtomBytes;
    unsigned char* a_smem = smem;
    unsigned char* b_smem = a_smem + (stream_a ? (size_t)0 : (size_t)a.cpart * a_chunk_bytes);
    unsigned char* o_smem = b_smem + (size_t)a.stages * b_stage_bytes;      // [kPwEpiWarps][32 rows x 128 bytes]
    uint64_t* bars = reinterpret_cast<uint64_t*>(o_smem + (size_t)kPwEpiWarps * 4096);
    uint64_t* a_full = bars;                       // [kMaxChunks] 32-channel chunk i of the current filter block has landed (*)
    uint64_t* a_empty = a_full + kMaxChunks;       // [1] all MMAs that read the bank have completed
    uint64_t* b_full = a_empty + 1;                // [kPwMaxStages] (*)
    uint64_t* b_empty = b_full + kPwMaxStages;     // [kPwMaxStages]
    uint64_t* acc_full = b_empty + kPwMaxStages;   // [2]
    uint64_t* acc_empty = acc_full + 2;            // [2] (*)        (*) of a pair: waited on in its first block only
    uint64_t* drain_bar = acc_empty + 2;           // [1] time-out path: the MMAs issued so far have completed
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(drain_bar + 1);
    volatile uint32_t* abort_flag = tmem_slot + 1;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t rank = PAIR ? cluster_ctarank() : 0u;
    const bool first_block = rank == 0;                                       // issues the MMAs of the item
    const int worker = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;       // block, or pair of blocks
    const int n_workers = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;
    if (tid == 0) {
        prefetch_tensormap(&map_w);
        prefetch_tensormap(&map_x);
        prefetch_tensormap(&map_y);
        for (int i = 0; i < (stream_a ? 0 : a.cpart); ++i) mbar_init(&a_full[i], 1);
        mbar_init(a_empty, 1);
        for (int i = 0; i < a.stages; ++i) { mbar_init(&b_full[i], 1); mbar_init(&b_empty[i], 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(&acc_full[i], 1); mbar_init(&acc_empty[i], kBlocks * kPwEpiWarps); }
        mbar_init(drain_bar, 1);
        *abort_flag = 0;
        fence_mbar_init();
    }
    __syncthreads();
    if (PAIR) cluster_sync_all();       // the peer's barriers exist before a copy or a commit can signal them
    if (warp == 1) Op::alloc(tmem_slot, 2 * kAccCols);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = *tmem_slot;
    // Everything above touched only this block's (pair's) shared and tensor memory and may overlap the tail of the
    // preceding kernel on the stream; global memory is read and written from here on.
    grid_dep_launch();
    grid_dep_wait();
    if (blockIdx.x == 0 && tid == 0) *a.status = 0u;       // (a block that gives up raises it at its very end)

    // item -> (bank = (filter block or pair of filter blocks) * ksplit + part of the channels, first atom): bank-major,
    // so that a block rarely changes its resident bank; with streamed filters pixel tile-major, so that the blocks
    // that read the same pixels do so at the same time and all but the first find them in L2
    auto decode = [&](int item, int& bank, int& first) {
        int tile;
        if (stream_a) tile = a.div_nb.divmod(item, bank);
        else bank = a.div_tiles.divmod(item, tile);
        first = tile * a.a_item;
    };
    // bank -> filter unit, first channel chunk and number of chunks of its part of the contraction
    auto split = [&](int bank, int& unit, int& c_lo, int& c_n) {
        unit = a.ksplit == 2 ? bank >> 1 : bank;
        c_lo = a.ksplit == 2 ? (bank & 1) * a.cpart : 0;
        c_n = min(a.cpart, a.cchunks - c_lo);
    };
    // first filter row of this block for a unit
    auto filter_row = [&](int unit) { return (PAIR ? 2 * unit + (int)rank : unit) * a.m_rows; };

    if (warp == 0) {
        // ---------------- loads (one thread per block): this block's filter rows and its (half of the) pixels
        if (lane == 0) {
            const uint32_t a_full_addr = PAIR ? map_to_cta(smem_u32(a_full), 0) : smem_u32(a_full);   // the first block's barriers
            const uint32_t b_full_addr = PAIR ? map_to_cta(smem_u32(b_full), 0) : smem_u32(b_full);
            int cur_bank = -1, slot = 0, issued = 0;
            uint32_t ph = 0, a_loads = 0;
            bool alive = true;
            for (int item = worker; item < a.items && alive; item += n_workers) {
                int bank, first, unit, c_lo, c_n;
                decode(item, bank, first);
                split(bank, unit, c_lo, c_n);
                const int k_row = filter_row(unit);
                // a lone block loads the atoms that exist; a block of a pair always its half of the item (past the batch: zeros)
                const int my_atoms = PAIR ? my_atoms_max : min(a.a_item, a.total_atoms - first);
                const int my_first = first + (PAIR ? (int)rank * my_atoms_max : 0);
                const uint32_t stage_tx = kBlocks * (b_off + (uint32_t)my_atoms * kAtomBytes);
                const bool new_bank = !stream_a && bank != cur_bank;
                if (new_bank) {
                    // another bank: wait until the MMAs on the old one are done
                    if (a_loads && !mbar_wait_bounded(a_empty, (a_loads - 1u) & 1u, abort_flag, a.max_polls)) { alive = false; break; }
                    cur_bank = bank;
                    ++a_loads;
                }
                for (int st = 0; st < c_n; ++st) {
                    const int ch = (c_lo + st) * kStageCh;       // first channel of this stage
                    if (new_bank) {
                        // chunk st of the bank goes out just ahead of the activation stage that needs it, so the
                        // first MMA waits for 16 KB of filters, not for the whole bank
                        if (first_block) mbar_arrive_expect_tx(&a_full[st], kBlocks * a_chunk_bytes);
                        Op::load_2d(a_smem + (size_t)st * a_chunk_bytes, &map_w, ch, k_row, a_full_addr + 8u * (uint32_t)st);
                    }
                    if (!mbar_wait_bounded(&b_empty[slot], ph ^ 1u, abort_flag, a.max_polls)) { alive = false; break; }
                    unsigned char* stage = b_smem + (size_t)slot * b_stage_bytes;
                    const uint32_t bar = b_full_addr + 8u * (uint32_t)slot;
                    if (first_block) mbar_arrive_expect_tx(&b_full[slot], stage_tx);
                    if (stream_a) Op::load_2d(stage, &map_w, ch, k_row, bar);
                    if (!(first_block && issued == a.test_drop_stage)) {     // (test hook: the first block's pixels never arrive)
                        unsigned char* dst = stage + b_off;
                        int blk;
                        int n = a.div_apb.divmod(my_first, blk);
                        if (a.multi) {
                            // one copy per image the atoms touch
                            for (int left = my_atoms; left > 0; ++n, blk = 0) {
                                const int cnt = min(left, a.apb - blk);
                                Op::load_4d(dst, &maps_x.m[cnt - 1], 0, ch, blk, n, bar);
                                dst += (size_t)cnt * kAtomBytes;
                                left -= cnt;
                            }
                        } else
                            for (int i = 0; i < my_atoms; ++i, dst += kAtomBytes) {
                                Op::load_3d(dst, &map_x, blk * kAtomPx, ch, n, bar);
                                if (++blk == a.apb) { blk = 0; ++n; }
                            }
                    }
                    ++issued;
                    if (++slot == a.stages) { slot = 0; ph ^= 1u; }
                }
            }
            if (*abort_flag && first_block) {
                // let copies already in flight (of both blocks of a pair: they signal these barriers) land before the
                // block's shared memory is released
                uint32_t dummy = 0;
                for (int cb = 0; cb < (stream_a ? 0 : a.cpart) && a_loads; ++cb)
                    mbar_wait_bounded(&a_full[cb], (a_loads - 1u) & 1u, &dummy, 1u << 14);
                const int pending = issued < a.stages ? issued : a.stages;
                for (int i = 0; i < pending; ++i) {
                    const int it = issued - 1 - i;
                    mbar_wait_bounded(&b_full[it % a.stages], (uint32_t)(it / a.stages) & 1u, &dummy, 1u << 14);
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issue (one thread; of a pair: of its first block)
        if (lane == 0 && first_block) {
            const uint32_t a_base = smem_u32(a_smem), b_base = smem_u32(b_smem);
            int cur_bank = -1, slot = 0, buf = 0;
            uint32_t ph = 0, a_waits = 0, acc_phase[2] = {0u, 0u};
            bool alive = true;
            for (int item = worker; item < a.items && alive; item += n_workers) {
                int bank, first, unit, c_lo, c_n;
                decode(item, bank, first);
                split(bank, unit, c_lo, c_n);
                const bool new_bank = !stream_a && bank != cur_bank;
                cur_bank = bank;
                // (of a pair: both blocks' write-back warps arrive here, the peer's with cluster-scope release)
                if (!(PAIR ? mbar_wait_bounded_cluster(&acc_empty[buf], acc_phase[buf] ^ 1u, abort_flag, a.max_polls)
                           : mbar_wait_bounded(&acc_empty[buf], acc_phase[buf] ^ 1u, abort_flag, a.max_polls))) { alive = false; break; }
                tc_fence_after_sync();
                const int groups = (PAIR && a.wide) ? 2 : 1;                 // MMA widths per item
                const uint32_t n_cols = (uint32_t)((PAIR ? a.a_item / groups : min(a.a_item, a.total_atoms - first)) * kAtomPx);
                const uint32_t m = PAIR ? 256u : (uint32_t)a.m_rows;
                const uint32_t idesc = (B16 ? idesc_b16(m, n_cols, a.fp16 != 0) : idesc_tf32(m, n_cols)) | kIdescBMajorMN;
                const uint32_t d = tmem + (uint32_t)(buf * kAccCols);
                for (int st = 0; st < c_n && alive; ++st) {
                    if (new_bank && !mbar_wait_bounded(&a_full[st], a_waits & 1u, abort_flag, a.max_polls)) { alive = false; break; }
                    if (!mbar_wait_bounded(&b_full[slot], ph, abort_flag, a.max_polls)) { alive = false; break; }
                    tc_fence_after_sync();
                    const uint32_t stage = b_base + (uint32_t)slot * b_stage_bytes;
                    const uint32_t a_chunk = stream_a ? stage : a_base + (uint32_t)st * a_chunk_bytes;
                    const uint32_t b_stage = stage + b_off;
                    const int ks = min(4, a.ksteps - (c_lo + st) * 4);
                    for (int g = 0; g < groups; ++g) {
                        // group g: this block's atoms [g * q, (g + 1) * q) of the stage, accumulator set g
                        const uint32_t b_grp = b_stage + (uint32_t)g * (uint32_t)(my_atoms_max / groups) * kAtomBytes;
                        for (int kk = 0; kk < ks; ++kk) {
                            // filters: 32 bytes further inside the 128-byte rows; pixels: the next 8 (fp32) or 16 (16-bit) channel rows
                            const uint64_t a_desc = smem_desc_sw128(a_chunk + (uint32_t)kk * 32u, 16u, 1024u);
                            const uint64_t b_desc = B16 ? smem_desc_sw128(b_grp + (uint32_t)kk * 2048u, (uint32_t)kStageCh * 128u, 1024u)
                                                        : smem_desc_mn_sw128_32b(b_grp + (uint32_t)kk * 1024u, (uint32_t)kStageCh * 128u, 512u);
                            Op::template mma<B16>(d + (uint32_t)(g * kAccCols), a_desc, b_desc, idesc, st > 0 || kk > 0);
                        }
                    }
                    Op::commit(&b_empty[slot]);
                    if (++slot == a.stages) { slot = 0; ph ^= 1u; }
                }
                if (!alive) break;
                if (new_bank) ++a_waits;
                Op::commit(&acc_full[buf]);
                // the next item of this block uses another filter block: tell the loaders when this bank is free
                const int next = item + n_workers;
                if (!stream_a && next < a.items && a.div_tiles.div(next) != bank) Op::commit(a_empty);
                acc_phase[buf] ^= 1u;
                if (!(PAIR && a.wide)) buf ^= 1;         // (a wide item uses both sets: one logical buffer)
            }
            if (!alive) {
                Op::commit_local(drain_bar);
                uint32_t dummy = 0;
                mbar_wait_bounded(drain_bar, 0u, &dummy, 1u << 16);
            }
        }
    } else {
        // ---------------- write-back: tensor memory -> registers -> swizzled tile -> tensor-map store
        // (of a pair: both blocks, each its own 128 filters and all pixels of the item)
        const int ew = warp - 2;
        const int quarter = warp & 3;                       // tensor-memory lanes this warp may read
        const int half = ew >> 2;                           // the two warps of a quarter take alternate 32-pixel blocks
        unsigned char* tile = o_smem + (size_t)ew * 4096;
        const int rows_q = a.m_rows / 4;                    // filters per lane quarter: 32, or 16 (M = 64: lanes 0-15)
        const uint32_t acc_empty_first = PAIR ? map_to_cta(smem_u32(acc_empty), 0) : 0u;
        bool alive = true;
        int li = 0;
        for (int item = worker; item < a.items; item += n_workers, ++li) {
            int bank, first, unit, c_lo, c_n;
            decode(item, bank, first);
            split(bank, unit, c_lo, c_n);
            const bool wide = PAIR && a.wide;
            const int buf = wide ? 0 : li & 1;
            const uint32_t acc_phase = (uint32_t)(wide ? li : li >> 1) & 1u;
            alive = __all_sync(0xffffffffu, alive && mbar_wait_bounded(&acc_full[buf], acc_phase, abort_flag, a.max_polls));
            if (!alive) break;
            tc_fence_after_sync();
            const uint32_t lane_base = tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * kAccCols);
            const int k0 = filter_row(unit) + quarter * rows_q;
            constexpr int kBpa = kAtomPx / 32;                  // 32-column blocks per atom
            // Accumulator column -> atom of the item.  One MMA width holds the atoms of block 0 of a pair, then those of
            // block 1; a wide item has two widths (accumulator sets 0 and 1), each with half of either block's atoms.
            const int q_atoms = PAIR ? my_atoms_max / (wide ? 2 : 1) : a.a_item;     // atoms of one block in one width
            const int width_blocks = (PAIR ? 2 : 1) * q_atoms * kBpa;               // 32-column blocks of one width
            if (k0 < a.K)
                for (int i = half; i < (wide ? 2 : 1) * width_blocks; i += 2) {
                    const int g = i >= width_blocks ? 1 : 0, ib = i - g * width_blocks;    // width, block inside it
                    const int hb = ib / (q_atoms * kBpa), jb = ib - hb * (q_atoms * kBpa); // block of the pair, block inside its part
                    const int atom = first + hb * my_atoms_max + g * q_atoms + jb / kBpa;
                    if (atom >= a.total_atoms) continue;            // (past the batch: zero-filled on load, never stored)
                    uint32_t v[32];
                    tmem_ld32(lane_base + (uint32_t)(g * kAccCols + ib * 32), v);
                    tmem_ld_wait();
                    if (lane == 0) bulk_wait_group_read<0>();       // the previous store has read the tile
                    __syncwarp();
                    if (lane < rows_q) {
                        // row = this lane's filter, 32 pixels = eight 16-byte chunks, chunk c stored at c ^ (row & 7)
                        unsigned char* row = tile + lane * 128;
#pragma unroll
                        for (int c = 0; c < 8; ++c)
                            *reinterpret_cast<uint4*>(row + ((c ^ (lane & 7)) << 4)) = make_uint4(v[4 * c], v[4 * c + 1], v[4 * c + 2], v[4 * c + 3]);
                    }
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        int blk;
                        const int n = a.div_apb.divmod(atom, blk);
                        // (split contraction: both parts add into y, which the launcher zeroed; a + b = b + a)
                        if (a.ksplit == 2) tma_reduce_add_3d(&map_y, blk * kAtomPx + (jb % kBpa) * 32, k0, n, tile);
                        else tma_store_3d(&map_y, blk * kAtomPx + (jb % kBpa) * 32, k0, n, tile);
                        bulk_commit_group();
                    }
                }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) {
                if (first_block) mbar_arrive(&acc_empty[buf]);
                else mbar_arrive_remote(acc_empty_first + 8u * (uint32_t)buf);
            }
        }
        if (lane == 0) bulk_wait_group<0>();                 // this thread's stores are complete
    }

    tc_fence_before_sync();
    __syncthreads();
    if (PAIR) cluster_sync_all();       // neither block leaves while the peer may still signal its barriers or read its operands
    if (warp == 1) Op::dealloc(tmem, 2 * kAccCols);
    if (tid == 0 && *abort_flag) atomicExch(a.status, 1u);
}


// Streamed filters, fp32 only: the filters rounded to the nearest TF32 value, into the workspace, so that only the
// image is truncated by the tensor core and the error bound holds for any channel count.  Also clears the status
// block, like the re-ordering kernels of the other tensor-core path.
__global__ void round_filters_tf32_kernel(const float4* __restrict__ w, float4* __restrict__ wp, long long n4,
                                          unsigned* __restrict__ status)
{
    grid_dep_launch();      // the convolution kernel may set itself up while this one runs
    if (blockIdx.x == 0 && threadIdx.x < kStatusBytes / sizeof(unsigned)) status[threadIdx.x] = 0u;
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += stride) {
        const float4 v = w[i];
        wp[i] = make_float4(to_tf32_rna(v.x), to_tf32_rna(v.y), to_tf32_rna(v.z), to_tf32_rna(v.w));
    }
}

// ---------------------------------------------------------------- host side
using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                   const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver's tensor-map encoder, looked up through the runtime so that the library does not link against the
// driver (it must load on machines without one).
EncodeTiledFn encode_tiled_fn()
{
    static EncodeTiledFn fn = []() -> EncodeTiledFn {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q = cudaDriverEntryPointSymbolNotFound;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            return nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

// Tensor of `rank` dimensions (innermost first), zeros for out-of-range elements.  `swizzle`: 128-byte rows
// with 16-byte chunks swizzled (K-major operands, output tiles) or with 32-byte chunks (the MN-major TF32 operand).
bool encode_map(CUtensorMap* map, CUtensorMapDataType type, const void* base, int rank, const cuuint64_t* dims,
                const cuuint64_t* strides_bytes, const cuuint32_t* box, CUtensorMapSwizzle swizzle)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint32_t ones[4] = {1, 1, 1, 1};
    return fn(map, type, (cuuint32_t)rank, const_cast<void*>(base), dims, strides_bytes, box, ones,
              CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct PwPlan {
    bool ok;
    int m_rows, n_blocks, apb, a_item, tiles, cchunks, stages, grid;
    int ksplit, cpart;     // split of the contraction over two work items (1: none), channel chunks per item
    bool stream_a;         // the filter bank does not fit: filter chunks travel through the ring with the pixels
    bool round_filters;    // ... and (fp32) are first rounded to TF32 into the workspace
    bool pair;             // two-SM MMAs: work items are (pixel tile, pair of 128-filter blocks), one per two-block cluster
    bool wide;             // ... whose items span two MMA widths of pixels (both accumulator sets at once)
    int n_units;           // filter blocks, or pairs of them
    long long total_atoms;
    long long items;
    double cost;           // planner's estimate of the kernel time in SM cycles (compares the one-SM and the two-SM form)
    size_t smem_bytes;
};

// Plan for the one-SM (`pair` = false) or the two-SM form.
template <bool B16>
PwPlan make_pw_variant(const Shape& sh, bool pair)
{
    using G = Geom<B16>;
    PwPlan p{};
    p.ok = false;
    p.pair = pair;
    p.m_rows = (sh.K <= 64 && !pair) ? 64 : 128;
    p.n_blocks = (sh.K + p.m_rows - 1) / p.m_rows;
    if (pair && p.n_blocks < 2) return p;
    p.n_units = pair ? (p.n_blocks + 1) / 2 : p.n_blocks;
    const long long HW = (long long)sh.H * sh.W;
    p.apb = (int)((HW + G::kAtomPx - 1) / G::kAtomPx);
    p.total_atoms = (long long)sh.N * p.apb;
    if (p.total_atoms > 0x3fffffffLL) return p;
    p.cchunks = (sh.C + G::kStageCh - 1) / G::kStageCh;
    const int sms = sm_count();
    const int workers = pair ? sms / 2 : sms;            // blocks, or pairs of blocks
    if (workers < 1) return p;
    // Atoms per item and split of the contraction.
    // One-SM form: the fewest rounds of items over the SMs, counted in atoms, plus half an atom of fixed cost per
    // item; ties go to the larger item (wider MMAs).  64 x 32 x 32 pixels = 2048 atoms of 32: 7 per item = 293 items =
    // two rounds of 7, where 8 per item would be two rounds of 8.
    // Two-SM form (an even number of atoms, half for each block): the widest MMAs that still leave an item for at
    // least half of the pairs; measured, narrower items only pay when most of the machine would otherwise idle.
    // Very long contractions (48 channel chunks or more: 1536 fp32 channels) on few pixels leave most SMs without
    // an item however small the items are; there the channel chunks of a tile may be shared out to two items that
    // both add into a zeroed y.  An item's time then counts as max(atoms, 3) (MMAs narrower than three atoms are as
    // short as their issue) and halves with the split, which costs 0.75 atoms (the zero-fill, adds instead of
    // stores).  Measured: 32 x 2048 x 7 x 8, 512 filters 31.6 -> 25.1 us, 128 filters 31.3 -> 22.3; with 512 or 1024
    // channels the split never paid (32 x 512 x 14 x 14, 128 filters: 11.2 -> 14.4 us).
    // CONV2D_B200_TMA_KSPLIT: 0 never split, 1 where the estimate says so, 2 wherever there are two chunks.
    const int forced = env_int("CONV2D_B200_TMA_ATOMS", 0);
    const int want_ks = env_int("CONV2D_B200_TMA_KSPLIT", 1);
    const bool deep = p.cchunks >= 48;
    const int ks_lo = (want_ks == 2 && p.cchunks >= 2) ? 2 : 1;
    const int ks_hi = (want_ks == 2 && p.cchunks >= 2) || (want_ks == 1 && deep) ? 2 : 1;
    p.a_item = 0;
    p.ksplit = 1;
    double best = 0;
    // Wide items of a pair (twice the atoms, both accumulator sets for one item): a streamed filter chunk then serves
    // twice the pixels, but the write-back no longer runs under the next item's MMAs.  Measured, that pays only for
    // long contractions (32 chunks or more: 1024 fp32 channels) and only where the wide items need no more rounds
    // over the pairs, counted in pixels, than the ordinary ones (16 x 1024 x 14 x 14, 2048 filters: 43.4 -> 36.6 us;
    // 64 x 1024 x 16 x 16, 1024 filters: 74.4 -> 66.6; 64 x 512 x 32 x 32, 512 filters: 70.7 -> 79.9, not taken).
    // CONV2D_B200_TMA_WIDE: 0 never, 1 so, 2 wherever a pair runs.
    const int want_wide = env_int("CONV2D_B200_TMA_WIDE", 1);
    {
        const long long tiles_w = (p.total_atoms + 2 * G::kMaxAtoms - 1) / (2 * G::kMaxAtoms);
        const long long tiles_n = (p.total_atoms + G::kMaxAtoms - 1) / G::kMaxAtoms;
        const long long rounds_w = (tiles_w * p.n_units + workers - 1) / workers, rounds_n = (tiles_n * p.n_units + workers - 1) / workers;
        p.wide = pair && !forced && (want_wide == 2 || (want_wide == 1 && p.cchunks >= 32 && 2 * rounds_w <= rounds_n));
    }
    if (p.wide) {
        p.a_item = 2 * G::kMaxAtoms;
        p.ksplit = 1;
    }
    for (int ks = ks_lo; ks <= ks_hi && !p.wide; ++ks) {
        int at_pair = 0;
        for (int at = G::kMaxAtoms; at >= 1; --at) {
            if (pair && (at & 1)) continue;
            if (forced && at != (forced < G::kMaxAtoms ? forced : G::kMaxAtoms)) continue;
            const long long tiles = (p.total_atoms + at - 1) / at;
            const long long items = tiles * p.n_units * ks;
            if (pair) {
                at_pair = at;
                if (2 * items >= workers) break;
                continue;
            }
            const long long rounds = (items + workers - 1) / workers;
            const double unit = 32.0 / G::kAtomPx;                       // an fp32 atom; a 16-bit atom counts double
            const double cost = (double)rounds * ((deep || ks == 2 ? std::max((double)at, 3.0 * unit) : (double)at) + 0.5 * unit) / ks +
                                (ks == 2 ? 0.75 * unit : 0.0);
            if (p.a_item == 0 || cost < best - 1e-9) { best = cost; p.a_item = at; p.ksplit = ks; }
        }
        if (pair && at_pair) {
            const long long tiles = (p.total_atoms + at_pair - 1) / at_pair;
            const long long rounds = (tiles * p.n_units * ks + workers - 1) / workers;
            const double cost = (double)rounds * (at_pair + 2.0) / ks + (ks == 2 ? 0.75 : 0.0);
            if (p.a_item == 0 || cost < best - 1e-9) { best = cost; p.a_item = at_pair; p.ksplit = ks; }
        }
    }
    if (p.a_item == 0) return p;
    p.cpart = (p.cchunks + p.ksplit - 1) / p.ksplit;
    p.stream_a = p.cpart > kMaxChunks;
    if (p.stream_a && env_int("CONV2D_B200_TMA_STREAM", 1) == 0) return p;
    p.round_filters = p.stream_a && !B16;
    p.tiles = (int)((p.total_atoms + p.a_item - 1) / p.a_item);
    p.items = (long long)p.tiles * p.n_units * p.ksplit;
    if (p.items > 0x7fffffffLL) return p;
    const size_t bank = (size_t)p.m_rows * 128;           // one channel chunk of a filter block
    const size_t fixed = (p.stream_a ? 0 : (size_t)p.cpart * bank) + (size_t)kPwEpiWarps * 4096 + kPwBookBytes + 1024;
    const size_t stage = (p.stream_a ? bank : 0) + (size_t)(pair ? p.a_item / 2 : p.a_item) * G::kAtomBytes;
    if (fixed + 2 * stage > kPwSmemLimit) return p;
    p.stages = (int)((kPwSmemLimit - fixed) / stage);
    if (p.stages > kPwMaxStages) p.stages = kPwMaxStages;
    {
        const int cap = env_int("CONV2D_B200_TMA_STAGES", 0);      // tuning: a shallower ring
        if (cap >= 2 && cap < p.stages) p.stages = cap;
    }
    p.smem_bytes = fixed + (size_t)p.stages * stage;
    // more than half of an SM's shared memory, so that two of these blocks, which both want all 512 tensor-memory
    // columns, never share an SM
    if (p.smem_bytes < 116 * 1024) p.smem_bytes = 116 * 1024;
    p.grid = (int)(p.items < workers ? p.items : workers) * (pair ? 2 : 1);
    // Estimated time in SM cycles, used only to choose between the two forms (constants fitted to measurements on
    // B200): the longest of (a) the busiest block's items, a stage taking the longest of its MMAs (at least 120
    // cycles each), its bytes at 40 B/clk and the copy latency spread over the ring, (b) all stages' bytes through
    // L2 at 7 TB/s, (c) the image, read once per filter block (pair) when it does not stay in L2 between the
    // filter block-major passes of a resident bank, and the output through HBM.
    {
        const double rounds = (double)((p.items + workers - 1) / workers);
        const double mma = 4.0 * std::max((double)p.a_item * 16.0 * G::kAtomPx / 32.0, 120.0);
        const double stage_time = std::max({mma, (double)stage / 40.0, 2500.0 / std::max(p.stages - 1, 1)});
        const double crit = rounds * (p.cpart * stage_time + 2500.0);
        const double l2 = (double)p.items * (pair ? 2 : 1) * p.cpart * (double)stage / 3700.0;
        const double x_bytes = (double)sh.N * sh.C * (double)HW * G::kElem, y_bytes = (double)sh.N * sh.K * (double)HW * 4.0;
        const double passes = (!p.stream_a && x_bytes > 100e6) ? p.n_units : 1;
        const double hbm = (y_bytes * (p.ksplit == 2 ? 2.0 : 1.0) + x_bytes * passes) / 3400.0;
        p.cost = std::max({crit, l2, hbm});
    }
    p.ok = true;
    return p;
}

template <bool B16>
PwPlan make_pw_plan(const Shape& sh)
{
    using G = Geom<B16>;
    PwPlan none{};
    none.ok = false;
    if (sh.R != 1 || sh.S != 1 || sh.pad_h || sh.pad_w) return none;
    const long long HW = (long long)sh.H * sh.W;
    // tensor-map strides are multiples of 16 bytes
    constexpr int kPer16 = 16 / G::kElem;
    if (HW % kPer16 != 0 || sh.C % kPer16 != 0 || sh.C > kPwMaxStreamChannels) return none;
    if (env_int("CONV2D_B200_TF32_TMA", 1) == 0) return none;
    const PwPlan one = make_pw_variant<B16>(sh, false);
    // CONV2D_B200_TMA_PAIR: 0 never, 1 where the planner expects it to be faster, 2 wherever it exists
    const int want = env_int("CONV2D_B200_TMA_PAIR", 1);
    if (want == 0 || sh.K <= 128) return one;
    const PwPlan two = make_pw_variant<B16>(sh, true);
    if (!two.ok) return one;
    if (!one.ok || want == 2) return two;
    return two.cost * kPwPairBias <= one.cost ? two : one;
}

template <bool B16>
int describe_pw(const Shape& sh, char* text, size_t text_bytes)
{
    using G = Geom<B16>;
    const PwPlan p = make_pw_plan<B16>(sh);
    if (!p.ok) return -1;
    const double px = (double)sh.N * sh.H * sh.W;
    const double cols = (double)p.total_atoms * G::kAtomPx;
    const double cols_issued = (double)p.tiles * p.a_item * G::kAtomPx;   // (a pair's last item is computed in full)
    const double issued = 2.0 * p.m_rows * (p.pair ? 2 * p.n_units : p.n_blocks) * (p.pair ? cols_issued : cols) *
                          ((sh.C + G::kKStep - 1) / G::kKStep * G::kKStep);
    return snprintf(text, text_bytes,
                    "tensor_core=1 kernel=pointwise_tma addressing=atoms filters_as=M two_sm=%d m_rows=%d tile_px=%d acc_sets=%d items=%lld "
                    "grid=%d stages=%d ksplit=%d resident_filters=%d filters_rounded_first=%d smem_bytes=%zu mma_useful_px=%.4f "
                    "mma_useful_flops=%.4f",
                    p.pair ? 1 : 0, p.pair ? 256 : p.m_rows, p.a_item * G::kAtomPx, p.wide ? 1 : 2, p.items, p.grid, p.stages, p.ksplit, p.stream_a ? 0 : 1,
                    p.round_filters ? 1 : 0, p.smem_bytes,
                    px / (p.pair ? cols_issued : cols), 2.0 * px * sh.K * sh.C / issued);
}

template <bool B16>
conv2d_status_t launch_pw(const void* x, const void* w, float* y, const Shape& sh, bool fp16,
                          void* workspace, size_t workspace_bytes, bool weights_packed, cudaStream_t stream)
{
    using G = Geom<B16>;
    const PwPlan p = make_pw_plan<B16>(sh);
    if (!p.ok) return CONV2D_ERR_UNSUPPORTED;
    const size_t rounded_bytes = p.round_filters ? (size_t)sh.K * sh.C * sizeof(float) : 0;
    if (!workspace || workspace_bytes < kStatusBytes + rounded_bytes) return CONV2D_ERR_WORKSPACE;
    if (p.ksplit == 2) {
        // both parts of the contraction add into y
        if (cudaMemsetAsync(y, 0, (size_t)sh.N * sh.K * sh.H * sh.W * sizeof(float), stream) != cudaSuccess) return CONV2D_ERR_CUDA;
    }
    if (p.round_filters) {
        float* wp = reinterpret_cast<float*>(static_cast<unsigned char*>(workspace) + kStatusBytes);
        if ((reinterpret_cast<uintptr_t>(w) | reinterpret_cast<uintptr_t>(wp)) & 15u) return CONV2D_ERR_UNSUPPORTED;
        if (!weights_packed) {
            const long long n4 = (long long)sh.K * sh.C / 4;
            long long blocks = (n4 + 255) / 256;
            if (blocks > sm_count() * 8LL) blocks = sm_count() * 8LL;
            // (launched the ordinary way: it starts only when the previous kernel on the stream, which may still be
            // reading the workspace, has finished)
            round_filters_tf32_kernel<<<(unsigned)blocks, 256, 0, stream>>>(static_cast<const float4*>(w), reinterpret_cast<float4*>(wp),
                                                                            n4, static_cast<unsigned*>(workspace));
            count_launch();
        }
        w = wp;
    }
    const cuuint64_t HW = (cuuint64_t)sh.H * sh.W;
    const cuuint64_t es = G::kElem;
    const CUtensorMapDataType in_type = !B16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32
                                      : (fp16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16);
    CUtensorMap map_w, map_x, map_y;
    {
        const cuuint64_t dims[2] = {(cuuint64_t)sh.C, (cuuint64_t)sh.K};
        const cuuint64_t strides[1] = {(cuuint64_t)sh.C * es};
        const cuuint32_t box[2] = {(cuuint32_t)G::kStageCh, (cuuint32_t)p.m_rows};
        if (!encode_map(&map_w, in_type, w, 2, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B)) return CONV2D_ERR_UNSUPPORTED;
    }
    {
        // pixels contiguous: the MN-major operand; 4-byte elements need the 32-byte-atom flavour of the 128-byte swizzle
        const cuuint64_t dims[3] = {HW, (cuuint64_t)sh.C, (cuuint64_t)sh.N};
        const cuuint64_t strides[2] = {HW * es, HW * es * (cuuint64_t)sh.C};
        const cuuint32_t box[3] = {(cuuint32_t)G::kAtomPx, (cuuint32_t)G::kStageCh, 1};
        if (!encode_map(&map_x, in_type, x, 3, dims, strides, box,
                        B16 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B))
            return CONV2D_ERR_UNSUPPORTED;
    }
    XMaps maps_x{};
    const bool multi = HW % G::kAtomPx == 0 && env_int("CONV2D_B200_TMA_MULTI", 1) != 0;
    if (multi) {
        // the image as (pixel in atom, channel, atom, image): a box of i + 1 atoms lands as i + 1 consecutive
        // [channel][pixel] blocks, which is how the MMA descriptor walks along the pixels
        const cuuint64_t dims[4] = {(cuuint64_t)G::kAtomPx, (cuuint64_t)sh.C, HW / G::kAtomPx, (cuuint64_t)sh.N};
        const cuuint64_t strides[3] = {HW * es, 128, HW * es * (cuuint64_t)sh.C};
        for (int i = 0; i < G::kMaxAtoms; ++i) {
            const cuuint32_t box[4] = {(cuuint32_t)G::kAtomPx, (cuuint32_t)G::kStageCh, (cuuint32_t)(i + 1), 1};
            if (!encode_map(&maps_x.m[i], in_type, x, 4, dims, strides, box,
                            B16 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B))
                return CONV2D_ERR_UNSUPPORTED;
        }
    }
    {
        const cuuint64_t dims[3] = {HW, (cuuint64_t)sh.K, (cuuint64_t)sh.N};
        const cuuint64_t strides[2] = {HW * 4, HW * 4 * (cuuint64_t)sh.K};
        const cuuint32_t box[3] = {32u, (cuuint32_t)(p.m_rows / 4), 1};
        if (!encode_map(&map_y, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, y, 3, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B))
            return CONV2D_ERR_UNSUPPORTED;
    }
    static size_t smem_done[64] = {}, smem_done_pair[64] = {};
    if ((p.pair ? raise_smem_limit(reinterpret_cast<const void*>(pointwise_tma_kernel<B16, true>), p.smem_bytes, smem_done_pair)
                : raise_smem_limit(reinterpret_cast<const void*>(pointwise_tma_kernel<B16, false>), p.smem_bytes, smem_done)) != cudaSuccess)
        return CONV2D_ERR_CUDA;
    PwArgs a{};
    a.status = static_cast<unsigned*>(workspace);
    a.K = sh.K;
    a.fp16 = fp16 ? 1 : 0;
    a.apb = p.apb; a.total_atoms = (int)p.total_atoms; a.a_item = p.a_item; a.tiles = p.tiles;
    a.n_blocks = p.n_blocks; a.m_rows = p.m_rows; a.items = (int)p.items;
    a.cchunks = p.cchunks; a.ksteps = (sh.C + G::kKStep - 1) / G::kKStep; a.stages = p.stages;
    a.stream_a = p.stream_a ? 1 : 0;
    a.wide = p.wide ? 1 : 0;
    a.ksplit = p.ksplit; a.cpart = p.cpart;
    a.multi = multi ? 1 : 0;
    a.max_polls = (unsigned)env_int("CONV2D_B200_TF32_MAX_POLLS", 1 << 22);
    a.test_drop_stage = env_int("CONV2D_B200_TF32_TEST_DROP_STAGE", -1);
    a.div_apb = FastDiv(p.apb); a.div_tiles = FastDiv(p.tiles); a.div_nb = FastDiv(p.n_units * p.ksplit);
    if (env_int("CONV2D_B200_TF32_VERBOSE", 0) != 0)
        fprintf(stderr, "conv2d plan: pointwise_tma%s%s%s m_rows %d n_blocks %d atoms/item %d tiles %d stages %d grid %d smem %zu\n",
                B16 ? " (16-bit)" : "", p.stream_a ? " (streamed filters)" : "", p.pair ? " (two-SM)" : "", p.m_rows, p.n_blocks, p.a_item, p.tiles, p.stages, p.grid, p.smem_bytes);
    if (p.pair) {
        // no more pairs than the device runs at once: the items are dealt out to the pairs of the grid in turn
        static int max_pairs[64] = {};
        const int slot = (int)((p.smem_bytes >> 12) & 63);
        if (max_pairs[slot] == 0) {
            cudaLaunchConfig_t cfg{};
            cfg.gridDim = dim3((unsigned)(sm_count() / 2 * 2));
            cfg.blockDim = dim3(kPwThreads);
            cfg.dynamicSmemBytes = p.smem_bytes;
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeClusterDimension;
            attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
            cfg.attrs = attr;
            cfg.numAttrs = 1;
            int n = 0;
            if (cudaOccupancyMaxActiveClusters(&n, pointwise_tma_kernel<B16, true>, &cfg) != cudaSuccess || n < 1) {
                (void)cudaGetLastError();
                n = sm_count() / 2;
            }
            max_pairs[slot] = n;
        }
        const int pairs = p.grid / 2 < max_pairs[slot] ? p.grid / 2 : max_pairs[slot];
        if (launch_pdl_cluster(pointwise_tma_kernel<B16, true>, dim3((unsigned)(2 * pairs)), dim3(kPwThreads), p.smem_bytes, stream, 2u,
                               map_w, map_x, map_y, maps_x, a) != cudaSuccess)
            return CONV2D_ERR_CUDA;
    } else if (launch_pdl(pointwise_tma_kernel<B16, false>, dim3((unsigned)p.grid), dim3(kPwThreads), p.smem_bytes, stream,
                          map_w, map_x, map_y, maps_x, a) != cudaSuccess)
        return CONV2D_ERR_CUDA;
    count_launch();
    return cudaGetLastError() == cudaSuccess ? CONV2D_OK : CONV2D_ERR_CUDA;
}

}  // namespace

bool pointwise_tma_supported(const Shape& sh, bool b16)
{
    return b16 ? make_pw_plan<true>(sh).ok : make_pw_plan<false>(sh).ok;
}

int describe_pointwise_tma_plan(const Shape& sh, bool b16, char* text, size_t text_bytes)
{
    return b16 ? describe_pw<true>(sh, text, text_bytes) : describe_pw<false>(sh, text, text_bytes);
}

// Workspace bytes the kernel needs beyond the status block (the rounded filters), 0 if none or not supported.
size_t pointwise_tma_workspace_extra(const Shape& sh, bool b16)
{
    if (b16) return 0;
    const PwPlan p = make_pw_plan<false>(sh);
    return p.ok && p.round_filters ? (size_t)sh.K * sh.C * sizeof(float) : 0;
}

conv2d_status_t launch_pointwise_tma(const void* x, const void* w, float* y, const Shape& sh, bool b16, bool fp16,
                                     void* workspace, size_t workspace_bytes, bool weights_packed, cudaStream_t stream)
{
    return b16 ? launch_pw<true>(x, w, y, sh, fp16, workspace, workspace_bytes, weights_packed, stream)
               : launch_pw<false>(x, w, y, sh, false, workspace, workspace_bytes, weights_packed, stream);
}

}  // namespace conv2d_b200
