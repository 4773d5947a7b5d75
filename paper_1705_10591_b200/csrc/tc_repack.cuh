// Tensor-core convolution: kernels that re-order the filters, once per call, into the exact shared-memory image
// the MMA instructions read (see the layout comment below).  Included by general_tf32.cu only.
#pragma once
#include "tc_plan.cuh"
#include "ptx.cuh"

namespace conv2d_b200 {
namespace {

using namespace ptx;

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
// stacked = 2 (compact): the same, but where S is odd the lone last tap of a filter row is a slice of 64 rows in
// natural filter order and half the size, so a channel block takes R * (floor(S / 2) * 128 + (S odd) * 64) rows.
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
        if (stacked == 2) {
            // compact bank of one filter block: per filter row `pairs` slices of 128 rows, then the lone tap's 64 rows
            const int pairs = ff.S / 2, odd = ff.S & 1;
            const size_t row_elems = (size_t)(pairs * n_tile + odd * (n_tile / 2)) * kChunks * EPC;
            T* base = wp + (size_t)cb * ff.R * row_elems;
            const bool chan = vc < ff.C;
            for (int r = 0; r < ff.R; ++r, base += row_elems) {
                for (int u = 0; u < pairs; ++u) {
                    T v = T(0);
                    if (k < K && chan) {
                        v = __ldg(src + (vc * ff.R + r) * ff.S + 2 * u + upper);
                        if (sizeof(T) == 4) v = (T)to_tf32_rna((float)v);
                    }
                    base[((size_t)(u * kChunks + chunk) * n_tile + f) * EPC + e] = v;
                }
                if (odd && f < n_tile / 2) {           // natural order: row f is filter f
                    T v = T(0);
                    if (f < K && chan) {
                        v = __ldg(w + ((size_t)f * ff.C * ff.R + (size_t)vc * ff.R + r) * ff.S + ff.S - 1);
                        if (sizeof(T) == 4) v = (T)to_tf32_rna((float)v);
                    }
                    base[(size_t)pairs * kChunks * n_tile * EPC + ((size_t)chunk * (n_tile / 2) + f) * EPC + e] = v;
                }
            }
            continue;
        }
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

}  // namespace
}  // namespace conv2d_b200
