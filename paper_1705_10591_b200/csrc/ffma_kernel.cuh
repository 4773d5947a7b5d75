// fp32 general-case kernel (Section 4, Algorithm 2) and its launchers, as templates.  Included by the translation units
// general_ffma_r*.cu, one per filter size, so that the instances compile in parallel; general_ffma.cu dispatches.
//
// Kept from the paper's design:
//   * grid = (blocks of filters) x (image blocks); a thread block covers the same image block
//     over all C channels for kTileK adjacent filters (Section 4.1);
//   * channels are staged kCB at a time in shared memory: the image block with its right/bottom
//     halo as it lies in memory, the filters transposed so that adjacent filters are adjacent
//     words (Section 4.2, Fig. 6);
//   * a thread accumulates kThrK filters x kThrQ horizontally adjacent outputs in registers,
//     keeps one input row segment of kThrQ+S-1 pixels in registers and reuses it for the S
//     horizontal taps (Section 4.2); filter values are read as 128-bit units, image pixels are
//     broadcast to the threads that differ only in their filter group.
//   * the next channel block is fetched while the current one is multiplied (Algorithm 2's prefetch): here
//     by asynchronous copies (cp.async) into a second image buffer and a raw filter buffer, so no thread
//     holds the prefetched data in registers.
// Changed for B200: register tile 8 x 8 with 128-bit shared-memory reads on both operands and packed
// two-filter FMAs; the filters arrive as they lie in memory ([filter][channel][tap], 16-byte pieces) and are
// turned around shared memory -> shared memory once per channel block;
// the output is written with 128-bit stores per filter row segment where alignment allows.
#pragma once
#include "common.cuh"

namespace conv2d_b200 {
namespace {


constexpr int kTileK = 64;    // filters per thread block (the paper's F_TB)
constexpr int kThrK = 8;      // filters per thread (F_T)
constexpr int kGroups = kTileK / kThrK;   // filter groups of a block: adjacent threads, adjacent filter units

// Image tile of a block: TH output rows of SEGS segments of TQ adjacent outputs (a thread's W_T); the block has
// kGroups x SEGS x TH threads.  32 x 8 outputs in segments of 8 is the default; the other shapes exist because a
// 26 x 26 map fills only 66 % of 32 x 8 tiles (and a 12 x 12 map 28 %): the launcher takes the shape that wastes least.
template <int TQ, int SEGS, int TH>
struct Tile {
    static constexpr int kTQ = TQ, kSegs = SEGS, kTH = TH, kTW = TQ * SEGS;
    static constexpr int kThreads = kGroups * SEGS * TH;
    static constexpr int kMinBlocks = kThreads <= 256 ? 2 : 1;
    // widest shared-memory read / global store unit (floats) that every segment start is aligned to
    static constexpr int kVec = TQ % 4 == 0 ? 4 : (TQ % 2 == 0 ? 2 : 1);
};

template <int R, int S, int CB, int TW, int TH>
struct Smem {
    static constexpr int kRows = TH + R - 1;
    static constexpr int kPitch = (TW + S - 1 + 3 + 3) / 4 * 4;   // room for whole 128-bit reads past the halo
    static constexpr int kRaw = CB * R * S;                      // floats of one filter in a channel block, as in memory
    static constexpr int kRawPitch = (kRaw + 3) / 4 * 4;
    float img[2][CB][kRows][kPitch];    // double buffer: channel block i + 1 lands while block i is multiplied
    float raw[kTileK][kRawPitch];       // filters of the coming block as they lie in memory
    float flt[CB][R * S][kTileK + 4];   // +4: transposed filter stores spread over banks, 128-bit reads stay aligned
};

// Asynchronous global -> shared copy of `bytes` (4, 8 or 16); only the first src_bytes are read, the rest is zero.
template <int BYTES>
__device__ __forceinline__ void cp_async(void* dst_smem, const void* src, int src_bytes)
{
    const unsigned d = (unsigned)__cvta_generic_to_shared(dst_smem);
    asm volatile("cp.async.ca.shared.global [%0], [%1], %2, %3;" ::"r"(d), "l"(src), "n"(BYTES), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }

// XV / WV: floats per asynchronous copy of the image rows / of the filters (4, 2 or 1, by alignment).
template <int R, int S, int CB, typename T, int XV, int WV>
__global__ void __launch_bounds__(T::kThreads, T::kMinBlocks)
general_ffma_kernel(const float* __restrict__ x, const float* __restrict__ w, float* __restrict__ y,
                    int C, int H, int W, int K, int P, int Q, int tiles_q, int vec_st)
{
    constexpr int TW = T::kTW, TH = T::kTH, kThrQ = T::kTQ, kThreads = T::kThreads, VR = T::kVec;
    using SM = Smem<R, S, CB, TW, TH>;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    SM& sm = *reinterpret_cast<SM*>(smem_raw);

    const int tid = threadIdx.x;
    const int tx = tid % kGroups;                     // filter group: adjacent threads, adjacent filter units
    const int ty = tid / kGroups;                     // output segment
    const int seg_row = ty / T::kSegs;
    const int seg_col = (ty % T::kSegs) * kThrQ;

    const int k0 = blockIdx.y * kTileK;
    const int tq = blockIdx.x % tiles_q, tp = blockIdx.x / tiles_q;
    const int p0 = tp * TH, q0 = tq * TW;
    const int n = blockIdx.z;
    const float* xin = x + (size_t)n * C * H * W;

    // Accumulators as (filter 2i, filter 2i+1) pairs: B200 reaches its fp32 FMA peak only with the two-wide
    // packed instruction (fma.rn.f32x2); the pixel is duplicated, the two filter taps are adjacent in shFlt.
    float2 acc[kThrK / 2][kThrQ];
#pragma unroll
    for (int i = 0; i < kThrK / 2; ++i)
#pragma unroll
        for (int j = 0; j < kThrQ; ++j) acc[i][j] = make_float2(0.f, 0.f);

    constexpr int NV = (kThrQ + S - 1 + VR - 1) / VR; // reads of VR floats per input row segment

    // Issues the copies of the channel block that starts at c0: image rows with their halo into img[buf], the
    // filters' runs of CB x R x S floats into raw.  Pieces outside the tensors are filled with zeros.
    auto issue = [&](int c0, int buf) {
        constexpr int kPieces = SM::kPitch / XV;
        for (int idx = tid; idx < CB * SM::kRows * kPieces; idx += kThreads) {
            const int v = idx % kPieces;
            const int row = (idx / kPieces) % SM::kRows;
            const int cc = idx / (kPieces * SM::kRows);
            const int c = c0 + cc, h = p0 + row, col = q0 + v * XV;
            const bool in = c < C && h < H && col < W;
            const int left = in ? min(XV, W - col) * 4 : 0;
            const float* src = in ? xin + ((size_t)c * H + h) * W + col : x;
            cp_async<4 * XV>(&sm.img[buf][cc][row][v * XV], src, left);
        }
        constexpr int kRuns = SM::kRaw / WV;
        const int live = (C - c0) * (R * S);                    // floats of a filter's run that exist
        for (int idx = tid; idx < kTileK * kRuns; idx += kThreads) {
            const int v = idx % kRuns, kk = idx / kRuns;
            const int e = v * WV;
            const bool in = k0 + kk < K && e < live;
            const int left = in ? min(WV, live - e) * 4 : 0;
            const float* src = in ? w + ((size_t)(k0 + kk) * C + c0) * (R * S) + e : w;
            cp_async<4 * WV>(&sm.raw[kk][e], src, left);
        }
        cp_async_commit();
    };

    issue(0, 0);
    for (int c0 = 0, it = 0; c0 < C; c0 += CB, ++it) {
        const int buf = it & 1;
        cp_async_wait_all();
        __syncthreads();                 // this block has landed; everyone is done with the previous one
        // filters: [filter][channel][tap] -> [channel][tap][filter]
        for (int idx = tid; idx < kTileK * SM::kRaw; idx += kThreads) {
            const int e = idx % SM::kRaw, kk = idx / SM::kRaw;
            sm.flt[e / (R * S)][e % (R * S)][kk] = sm.raw[kk][e];
        }
        __syncthreads();
        if (c0 + CB < C) issue(c0 + CB, buf ^ 1);      // the next block arrives under the multiplications below

#pragma unroll 1
        for (int cc = 0; cc < CB; ++cc) {
#pragma unroll
            for (int r = 0; r < R; ++r) {
                float2 img[VR * NV];                             // (x, x)
                const float* srow = &sm.img[buf][cc][seg_row + r][seg_col];
#pragma unroll
                for (int v = 0; v < NV; ++v) {
                    if (VR == 4) {
                        const float4 t = reinterpret_cast<const float4*>(srow)[v];
                        img[4 * v + 0] = make_float2(t.x, t.x); img[4 * v + 1] = make_float2(t.y, t.y);
                        img[4 * v + 2] = make_float2(t.z, t.z); img[4 * v + 3] = make_float2(t.w, t.w);
                    } else if (VR == 2) {
                        const float2 t = reinterpret_cast<const float2*>(srow)[v];
                        img[2 * v + 0] = make_float2(t.x, t.x); img[2 * v + 1] = make_float2(t.y, t.y);
                    } else {
                        const float t = srow[v];
                        img[v] = make_float2(t, t);
                    }
                }
#pragma unroll
                for (int s = 0; s < S; ++s) {
                    float2 flt[kThrK / 2];                       // taps of filters (2i, 2i+1)
                    const float4* fs = reinterpret_cast<const float4*>(&sm.flt[cc][r * S + s][tx * kThrK]);
#pragma unroll
                    for (int v = 0; v < kThrK / 4; ++v) {
                        const float4 t = fs[v];
                        flt[2 * v + 0] = make_float2(t.x, t.y); flt[2 * v + 1] = make_float2(t.z, t.w);
                    }
#pragma unroll
                    for (int i = 0; i < kThrK / 2; ++i)
#pragma unroll
                        for (int j = 0; j < kThrQ; ++j) acc[i][j] = __ffma2_rn(img[s + j], flt[i], acc[i][j]);
                }
            }
        }
    }

    // ---- write the register tile ----
    const int p = p0 + seg_row, q = q0 + seg_col;
    if (p >= P || q >= Q) return;
#pragma unroll
    for (int i = 0; i < kThrK; ++i) {
        const int k = k0 + tx * kThrK + i;
        if (k >= K) break;
        float* o = y + (((size_t)n * K + k) * P + p) * Q + q;
        float row[kThrQ];
#pragma unroll
        for (int j = 0; j < kThrQ; ++j) row[j] = (i & 1) ? acc[i / 2][j].y : acc[i / 2][j].x;
        if (VR == 4 && vec_st == 4 && q + kThrQ <= Q) {
#pragma unroll
            for (int v = 0; v < kThrQ / 4; ++v)
                *reinterpret_cast<float4*>(o + 4 * v) = make_float4(row[4 * v], row[4 * v + 1], row[4 * v + 2], row[4 * v + 3]);
        } else if (VR >= 2 && vec_st >= 2 && q + kThrQ <= Q) {
#pragma unroll
            for (int v = 0; v < kThrQ / 2; ++v)
                *reinterpret_cast<float2*>(o + 2 * v) = make_float2(row[2 * v], row[2 * v + 1]);
        } else {
#pragma unroll
            for (int j = 0; j < kThrQ; ++j)
                if (q + j < Q) o[j] = row[j];
        }
    }
}

template <int R, int S, int CB, typename T, int XV, int WV>
conv2d_status_t launch_tile_v(const float* x, const float* w, float* y, const Shape& sh, cudaStream_t stream)
{
    auto kern = general_ffma_kernel<R, S, CB, T, XV, WV>;
    const size_t smem = sizeof(Smem<R, S, CB, T::kTW, T::kTH>);
    static size_t smem_done[64] = {};
    if (smem > 48 * 1024 && raise_smem_limit(reinterpret_cast<const void*>(kern), smem, smem_done) != cudaSuccess)
        return CONV2D_ERR_CUDA;
    const int tiles_q = (sh.Q + T::kTW - 1) / T::kTW, tiles_p = (sh.P + T::kTH - 1) / T::kTH;
    dim3 grid(tiles_q * tiles_p, (sh.K + kTileK - 1) / kTileK, sh.N);
    // widest store unit the output rows allow (floats)
    const int vec_st = (sh.Q % 4 == 0 && reinterpret_cast<uintptr_t>(y) % 16 == 0) ? 4
                     : (sh.Q % 2 == 0 && reinterpret_cast<uintptr_t>(y) % 8 == 0) ? 2 : 1;
    kern<<<grid, T::kThreads, smem, stream>>>(x, w, y, sh.C, sh.H, sh.W, sh.K, sh.P, sh.Q, tiles_q, vec_st);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? CONV2D_OK : CONV2D_ERR_CUDA;
}

// Width of the asynchronous copies: whole 16-byte pieces where every piece starts on 16 bytes (image: W a multiple
// of 4; filters: C*R*S and CB*R*S multiples of 4), else 8- or 4-byte pieces.
template <int R, int S, int CB, typename T>
conv2d_status_t launch_tile(const float* x, const float* w, float* y, const Shape& sh, cudaStream_t stream)
{
    constexpr int kRaw = CB * R * S;
    const bool x4 = sh.W % 4 == 0 && reinterpret_cast<uintptr_t>(x) % 16 == 0;
    const long long crs = (long long)sh.C * R * S;
    const int wv = (kRaw % 4 == 0 && crs % 4 == 0 && reinterpret_cast<uintptr_t>(w) % 16 == 0) ? 4
                 : (kRaw % 2 == 0 && crs % 2 == 0 && reinterpret_cast<uintptr_t>(w) % 8 == 0) ? 2 : 1;
    if (x4) {
        if (wv == 4) return launch_tile_v<R, S, CB, T, 4, (kRaw % 4 == 0 ? 4 : 1)>(x, w, y, sh, stream);
        if (wv == 2) return launch_tile_v<R, S, CB, T, 4, (kRaw % 2 == 0 ? 2 : 1)>(x, w, y, sh, stream);
        return launch_tile_v<R, S, CB, T, 4, 1>(x, w, y, sh, stream);
    }
    if (wv == 4) return launch_tile_v<R, S, CB, T, 1, (kRaw % 4 == 0 ? 4 : 1)>(x, w, y, sh, stream);
    if (wv == 2) return launch_tile_v<R, S, CB, T, 1, (kRaw % 2 == 0 ? 2 : 1)>(x, w, y, sh, stream);
    return launch_tile_v<R, S, CB, T, 1, 1>(x, w, y, sh, stream);
}

// Share of a tile shape's outputs that exist, for a P x Q map; 0 where the shape cannot serve the map: the 16-byte
// copies of the image rows start at the tile's first column, so a width that is not a multiple of 4 must cover the
// whole map width with one tile.
template <typename T>
double tile_fill(const Shape& sh)
{
    if (T::kTW % 4 != 0 && sh.Q > T::kTW) return 0.0;
    const int tq = (sh.Q + T::kTW - 1) / T::kTW, tp = (sh.P + T::kTH - 1) / T::kTH;
    return (double)sh.P * sh.Q / ((double)tq * T::kTW * tp * T::kTH);
}

template <int R, int S, int CB>
conv2d_status_t launch_instance(const float* x, const float* w, float* y, const Shape& sh, cudaStream_t stream)
{
    using T0 = Tile<8, 4, 8>;      // 32 x 8 outputs, 256 threads
    using T1 = Tile<8, 2, 16>;     // 16 x 16
    using T2 = Tile<10, 3, 10>;    // 30 x 10, 240 threads
    using T4 = Tile<9, 3, 9>;      // 27 x 9, 216 threads
    using T5 = Tile<9, 6, 5>;      // 54 x 5, 240 threads
    using T6 = Tile<6, 2, 12>;     // 12 x 12, 192 threads
    const int forced = env_int("CONV2D_B200_FFMA_TILE", -1);
    int best = 0;
    double fill = tile_fill<T0>(sh) * 1.02;          // the default wins ties: 128-bit reads and stores
    auto consider = [&](int id, double f) { if (f > fill + 1e-9) { fill = f; best = id; } };
    consider(1, tile_fill<T1>(sh) * 1.02);
    consider(2, tile_fill<T2>(sh));
    consider(4, tile_fill<T4>(sh));
    consider(5, tile_fill<T5>(sh));
    consider(6, tile_fill<T6>(sh));
    if (forced >= 0 && forced <= 6) {
        const double f[7] = {1.0, 1.0, tile_fill<T2>(sh), 0.0, tile_fill<T4>(sh), tile_fill<T5>(sh), tile_fill<T6>(sh)};
        if (f[forced] > 0.0) best = forced;
    }
    switch (best) {
    case 1: return launch_tile<R, S, CB, T1>(x, w, y, sh, stream);
    case 2: return launch_tile<R, S, CB, T2>(x, w, y, sh, stream);
    case 4: return launch_tile<R, S, CB, T4>(x, w, y, sh, stream);
    case 5: return launch_tile<R, S, CB, T5>(x, w, y, sh, stream);
    case 6: return launch_tile<R, S, CB, T6>(x, w, y, sh, stream);
    default: return launch_tile<R, S, CB, T0>(x, w, y, sh, stream);
    }
}

}  // namespace
}  // namespace conv2d_b200
