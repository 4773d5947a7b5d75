// Special case: one input channel, many filters (Section 3, Algorithm 1).
//
// Kept from the paper's design:
//   * the image is cut into blocks whose halo lies only to the right and below (Section 3.1);
//   * a thread block walks down its block row by row; horizontal sharing of input pixels goes
//     through shared memory, vertical sharing through a per-thread register window of
//     (R-1+rows per step) x (S+n-1) pixels that slides down (Section 3.2);
//   * every thread owns n horizontally adjacent outputs and reads, computes and writes them as
//     one unit (Section 3.2; here n = 4, a 128-bit unit, instead of the 64-bit unit of Kepler);
//   * all threads of a warp use the same filter tap at the same time, so the filter value is a
//     broadcast operand (Section 3.3).
// Changed for B200: the whole input tile (with halo) is staged once per block instead of one row
// per step with two barriers, because input is ~3 % of the bytes moved and 228 KB of shared memory
// per SM holds several such tiles; two output rows are produced per step so that each filter tap
// fetched feeds 8 FMAs; output stores are 128-bit streaming stores (the output is 97 % of the
// traffic and is never read back).
#include "common.cuh"
#include "ptx.cuh"

namespace conv2d_b200 {

// Raised by a kernel whose bounded wait expired; read and cleared by conv2d_get_status.
__device__ unsigned g_device_timeout;

__constant__ float c_filters[kConstFilterFloats];

namespace {

constexpr int kThreads = 128;
constexpr int kVec = 4;                       // outputs per thread per row (the paper's n)
constexpr int kTileW = kThreads * kVec;       // 512 output columns per block
constexpr int kPitch = kTileW + 8;            // staged columns per row (halo S-1 <= 8), floats
constexpr int kPitch4 = kPitch / 4;

__device__ __forceinline__ void store4(float* p, float4 v) { __stcs(reinterpret_cast<float4*>(p), v); }

// Stores the n = 4 adjacent outputs of one thread at columns q0..q0+3 of a row of Q outputs with the
// widest unit the row alignment allows: `unit` = 4 when Q % 4 == 0 (every row 16-byte aligned),
// 2 when Q % 2 == 0, else 1.  q0 is a multiple of 4.
__device__ __forceinline__ void store_outputs(float* o, float a0, float a1, float a2, float a3, int q0, int Q, int unit)
{
    if (unit == 4 && q0 + 3 < Q) {
        store4(o, make_float4(a0, a1, a2, a3));
    } else if (unit >= 2) {
        if (q0 + 1 < Q) __stcs(reinterpret_cast<float2*>(o), make_float2(a0, a1));
        if (q0 + 3 < Q) __stcs(reinterpret_cast<float2*>(o + 2), make_float2(a2, a3));
    } else {
        if (q0 + 0 < Q) __stcs(o + 0, a0);
        if (q0 + 1 < Q) __stcs(o + 1, a1);
        if (q0 + 2 < Q) __stcs(o + 2, a2);
        if (q0 + 3 < Q) __stcs(o + 3, a3);
    }
}

// WSRC: 0 = filter taps read from the constant bank, 1 = from a shared-memory copy (128-bit broadcast loads).
template <int R, int S, int TR, int WSRC>
__global__ void __launch_bounds__(kThreads)
single_channel_kernel(const float* __restrict__ x, const float* __restrict__ w, float* __restrict__ y,
                      int H, int W, int K, int P, int Q, int tile_h, int vec_ld, int vec_st)
{
    constexpr int NV = (S + kVec - 1 + 3) / 4;          // float4 loads per window row
    constexpr int WC = 4 * NV;                          // window columns held (>= S + n - 1)
    constexpr int WR = R - 1 + TR;                      // window rows held
    constexpr int RS = R * S;
    constexpr int RSP = (RS + 3) / 4 * 4;               // taps per filter, padded to a 128-bit multiple

    extern __shared__ float4 smem4[];
    float4* tile4 = smem4;
    const int tid = threadIdx.x;
    const int col0 = blockIdx.x * kTileW;
    const int row0 = blockIdx.y * tile_h;
    const int n = blockIdx.z;
    const int th = min(tile_h, P - row0);               // output rows of this block
    const int rows_in = th + R - 1;                     // staged input rows
    const float* xin = x + (size_t)n * H * W;

    // ---- stage the input tile (each needed pixel fetched once per block) ----
    for (int idx = tid; idx < rows_in * kPitch4; idx += kThreads) {
        const int row = idx / kPitch4, c4 = idx - row * kPitch4;
        const int col = col0 + 4 * c4;
        const float* src = xin + (size_t)(row0 + row) * W + col;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (vec_ld && col + 3 < W) {
            v = __ldg(reinterpret_cast<const float4*>(src));
        } else {
            if (col + 0 < W) v.x = __ldg(src + 0);
            if (col + 1 < W) v.y = __ldg(src + 1);
            if (col + 2 < W) v.z = __ldg(src + 2);
            if (col + 3 < W) v.w = __ldg(src + 3);
        }
        tile4[idx] = v;
    }
    float* wsm = reinterpret_cast<float*>(smem4 + (size_t)(tile_h + R - 1) * kPitch4);
    if (WSRC == 1) {
        for (int idx = tid; idx < K * RSP; idx += kThreads) {
            const int f = idx / RSP, t = idx - f * RSP;
            wsm[idx] = (t < RS) ? __ldg(w + (size_t)f * RS + t) : 0.f;
        }
    }
    __syncthreads();

    const int q0 = col0 + kVec * tid;
    if (q0 >= Q) return;                                 // no barrier after this point

    float win[WR][WC];
#pragma unroll
    for (int r = 0; r < R - 1; ++r)
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            const float4 t = tile4[r * kPitch4 + tid + v];
            win[r][4 * v + 0] = t.x; win[r][4 * v + 1] = t.y; win[r][4 * v + 2] = t.z; win[r][4 * v + 3] = t.w;
        }

    const size_t plane = (size_t)P * Q;
    for (int p = 0; p < th; p += TR) {
        // newest TR rows of the window
#pragma unroll
        for (int tr = 0; tr < TR; ++tr) {
            const int row = p + R - 1 + tr;
#pragma unroll
            for (int v = 0; v < NV; ++v) {
                float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
                if (row < rows_in) t = tile4[row * kPitch4 + tid + v];
                win[R - 1 + tr][4 * v + 0] = t.x; win[R - 1 + tr][4 * v + 1] = t.y;
                win[R - 1 + tr][4 * v + 2] = t.z; win[R - 1 + tr][4 * v + 3] = t.w;
            }
        }

        float* yout = y + ((size_t)n * K * P + (size_t)(row0 + p)) * Q + q0;
#pragma unroll 1
        for (int f = 0; f < K; ++f, yout += plane) {
            float wr[RSP];
            if (WSRC == 1) {
                const float4* wf = reinterpret_cast<const float4*>(wsm + f * RSP);
#pragma unroll
                for (int v = 0; v < RSP / 4; ++v) {
                    const float4 t = wf[v];
                    wr[4 * v + 0] = t.x; wr[4 * v + 1] = t.y; wr[4 * v + 2] = t.z; wr[4 * v + 3] = t.w;
                }
            } else {
#pragma unroll
                for (int t = 0; t < RS; ++t) wr[t] = c_filters[f * RS + t];
            }
            float acc[TR][kVec];
#pragma unroll
            for (int tr = 0; tr < TR; ++tr)
#pragma unroll
                for (int j = 0; j < kVec; ++j) acc[tr][j] = 0.f;
#pragma unroll
            for (int r = 0; r < R; ++r)
#pragma unroll
                for (int s = 0; s < S; ++s)
#pragma unroll
                    for (int tr = 0; tr < TR; ++tr)
#pragma unroll
                        for (int j = 0; j < kVec; ++j)
                            acc[tr][j] = fmaf(win[tr + r][s + j], wr[r * S + s], acc[tr][j]);
#pragma unroll
            for (int tr = 0; tr < TR; ++tr) {
                if (p + tr < th) {
                    float* o = yout + (size_t)tr * Q;
                    if (vec_st && q0 + 3 < Q) {
                        store4(o, make_float4(acc[tr][0], acc[tr][1], acc[tr][2], acc[tr][3]));
                    } else {
#pragma unroll
                        for (int j = 0; j < kVec; ++j)
                            if (q0 + j < Q) __stcs(o + j, acc[tr][j]);
                    }
                }
            }
        }
        // slide the window down by TR rows
#pragma unroll
        for (int r = 0; r < R - 1; ++r)
#pragma unroll
            for (int c = 0; c < WC; ++c) win[r][c] = win[r + TR][c];
    }
}

// Per-thread unit ablation (the matched / unmatched experiment of Section 5.1): the same row-walking
// scheme with a per-thread unit of UNIT adjacent outputs (1 = float, 2 = float2, 4 = float4) read, computed
// and written as one piece.  On Kepler the unit had to match the 8-byte bank; on B200 banks are 4 bytes
// wide, so any difference comes from instruction count and store width.  Benchmark use only
// (CONV2D_B200_SC_UNIT); scalar FMA, one output row per step, taps in shared memory.
template <int R, int S, int UNIT>
__global__ void __launch_bounds__(kThreads)
single_channel_unit_kernel(const float* __restrict__ x, const float* __restrict__ w, float* __restrict__ y,
                           int H, int W, int K, int P, int Q, int tile_h, int vec_st)
{
    constexpr int TW = kThreads * UNIT;                 // output columns per block
    constexpr int PITCH = TW + 8;                       // staged floats per row
    constexpr int WC = S + UNIT - 1;                    // window columns
    constexpr int RS = R * S;
    extern __shared__ float4 smem4[];
    float* tile = reinterpret_cast<float*>(smem4);
    const int tid = threadIdx.x;
    const int col0 = blockIdx.x * TW, row0 = blockIdx.y * tile_h, n = blockIdx.z;
    const int th = min(tile_h, P - row0);
    const int rows_in = th + R - 1;
    const float* xin = x + (size_t)n * H * W;
    for (int idx = tid; idx < rows_in * PITCH; idx += kThreads) {
        const int row = idx / PITCH, c = idx - row * PITCH;
        const int col = col0 + c;
        tile[idx] = (col < W) ? __ldg(xin + (size_t)(row0 + row) * W + col) : 0.f;
    }
    float* wsm = tile + (size_t)(tile_h + R - 1) * PITCH;
    for (int idx = tid; idx < K * RS; idx += kThreads) wsm[idx] = __ldg(w + idx);
    __syncthreads();
    const int q0 = col0 + UNIT * tid;
    if (q0 >= Q) return;
    float win[R][WC];
#pragma unroll
    for (int r = 0; r < R - 1; ++r)
#pragma unroll
        for (int c = 0; c < WC; ++c) win[r][c] = tile[r * PITCH + UNIT * tid + c];
    const size_t plane = (size_t)P * Q;
    for (int p = 0; p < th; ++p) {
#pragma unroll
        for (int c = 0; c < WC; ++c) win[R - 1][c] = tile[(p + R - 1) * PITCH + UNIT * tid + c];
        float* yout = y + ((size_t)n * K * P + (size_t)(row0 + p)) * Q + q0;
#pragma unroll 1
        for (int f = 0; f < K; ++f, yout += plane) {
            float acc[UNIT];
#pragma unroll
            for (int j = 0; j < UNIT; ++j) acc[j] = 0.f;
#pragma unroll
            for (int r = 0; r < R; ++r)
#pragma unroll
                for (int s2 = 0; s2 < S; ++s2) {
                    const float wv = wsm[f * RS + r * S + s2];
#pragma unroll
                    for (int j = 0; j < UNIT; ++j) acc[j] = fmaf(win[r][s2 + j], wv, acc[j]);
                }
            if (vec_st && q0 + UNIT <= Q) {
                if (UNIT == 4) store4(yout, make_float4(acc[0], acc[1 % UNIT], acc[2 % UNIT], acc[3 % UNIT]));
                else if (UNIT == 2) __stcs(reinterpret_cast<float2*>(yout), make_float2(acc[0], acc[1 % UNIT]));
                else __stcs(yout, acc[0]);
            } else {
#pragma unroll
                for (int j = 0; j < UNIT; ++j)
                    if (q0 + j < Q) __stcs(yout + j, acc[j]);
            }
        }
#pragma unroll
        for (int r = 0; r < R - 1; ++r)
#pragma unroll
            for (int c = 0; c < WC; ++c) win[r][c] = win[r + 1][c];
    }
}

template <int R, int S, int UNIT>
conv2d_status_t launch_unit(const float* x, const float* w, float* y, const Shape& sh, int tile_h, cudaStream_t stream)
{
    constexpr int TW = kThreads * UNIT;
    const size_t smem = ((size_t)(tile_h + R - 1) * (TW + 8) + (size_t)sh.K * R * S) * sizeof(float);
    if (smem > 200 * 1024) return CONV2D_ERR_UNSUPPORTED;
    auto kern = single_channel_unit_kernel<R, S, UNIT>;
    static size_t smem_done[64] = {};
    if (raise_smem_limit(reinterpret_cast<const void*>(kern), smem, smem_done) != cudaSuccess) return CONV2D_ERR_CUDA;
    dim3 grid((sh.Q + TW - 1) / TW, (sh.P + tile_h - 1) / tile_h, sh.N);
    const int vec_st = (sh.Q % UNIT == 0) && (reinterpret_cast<uintptr_t>(y) % 16 == 0);
    kern<<<grid, kThreads, smem, stream>>>(x, w, y, sh.H, sh.W, sh.K, sh.P, sh.Q, tile_h, vec_st);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? CONV2D_OK : CONV2D_ERR_CUDA;
}

// Packed-FMA variant.  B200 issues fp32 FMAs at full rate only as two-wide packed instructions
// (fma.rn.f32x2): a scalar-FMA loop tops out near 82 % of the fp32 peak, a packed one near 99 %,
// and the packed form leaves issue slots for the loads, stores and address arithmetic.  The two
// lanes of a packed FMA are two adjacent FILTERS applied to the same pixel: the pixel window is
// held as (x, x) pairs (built once per row step, reused by all filters) and the taps of filters
// 2i and 2i+1 are interleaved in shared memory so that one 128-bit broadcast load brings two taps
// for both filters.  Everything else is as in the kernel above.
template <int R, int S, int TR>
__global__ void __launch_bounds__(kThreads)
single_channel_packed_kernel(const float* __restrict__ x, const float* __restrict__ w, float* __restrict__ y,
                             int H, int W, int K, int P, int Q, int tile_h, int vec_ld, int vec_st)
{
    constexpr int NV = (S + kVec - 1 + 3) / 4;          // float4 loads per window row
    constexpr int WC = 4 * NV;
    constexpr int WR = R - 1 + TR;
    constexpr int RS = R * S;
    constexpr int RS2 = (RS + 1) / 2;                   // 128-bit units per filter pair (two taps each)

    extern __shared__ float4 smem4[];
    float4* tile4 = smem4;
    const int tid = threadIdx.x;
    const int col0 = blockIdx.x * kTileW;
    const int row0 = blockIdx.y * tile_h;
    const int n = blockIdx.z;
    const int th = min(tile_h, P - row0);
    const int rows_in = th + R - 1;
    const float* xin = x + (size_t)n * H * W;

    for (int idx = tid; idx < rows_in * kPitch4; idx += kThreads) {
        const int row = idx / kPitch4, c4 = idx - row * kPitch4;
        const int col = col0 + 4 * c4;
        const float* src = xin + (size_t)(row0 + row) * W + col;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (vec_ld && col + 3 < W) {
            v = __ldg(reinterpret_cast<const float4*>(src));
        } else {
            if (col + 0 < W) v.x = __ldg(src + 0);
            if (col + 1 < W) v.y = __ldg(src + 1);
            if (col + 2 < W) v.z = __ldg(src + 2);
            if (col + 3 < W) v.w = __ldg(src + 3);
        }
        tile4[idx] = v;
    }
    // taps of filter pair i: [i][unit u] = (w[2i][2u], w[2i+1][2u], w[2i][2u+1], w[2i+1][2u+1]); zero past K or RS
    float4* wsm4 = smem4 + (size_t)(tile_h + R - 1) * kPitch4;
    const int pairs = (K + 1) / 2;
    for (int idx = tid; idx < pairs * RS2; idx += kThreads) {
        const int i = idx / RS2, u = idx - i * RS2;
        const int f0 = 2 * i, f1 = 2 * i + 1, t0 = 2 * u, t1 = 2 * u + 1;
        float4 v;
        v.x = __ldg(w + (size_t)f0 * RS + t0);
        v.y = (f1 < K) ? __ldg(w + (size_t)f1 * RS + t0) : 0.f;
        v.z = (t1 < RS) ? __ldg(w + (size_t)f0 * RS + t1) : 0.f;
        v.w = (t1 < RS && f1 < K) ? __ldg(w + (size_t)f1 * RS + t1) : 0.f;
        wsm4[idx] = v;
    }
    __syncthreads();

    const int q0 = col0 + kVec * tid;
    if (q0 >= Q) return;

    float2 win[WR][WC];                                   // (x, x) pairs
#pragma unroll
    for (int r = 0; r < R - 1; ++r)
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            const float4 t = tile4[r * kPitch4 + tid + v];
            win[r][4 * v + 0] = make_float2(t.x, t.x); win[r][4 * v + 1] = make_float2(t.y, t.y);
            win[r][4 * v + 2] = make_float2(t.z, t.z); win[r][4 * v + 3] = make_float2(t.w, t.w);
        }

    const size_t plane = (size_t)P * Q;
    const bool vec_ok = vec_st && (q0 + 3 < Q);
    for (int p = 0; p < th; p += TR) {
#pragma unroll
        for (int tr = 0; tr < TR; ++tr) {
            const int row = p + R - 1 + tr;
#pragma unroll
            for (int v = 0; v < NV; ++v) {
                float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
                if (row < rows_in) t = tile4[row * kPitch4 + tid + v];
                win[R - 1 + tr][4 * v + 0] = make_float2(t.x, t.x); win[R - 1 + tr][4 * v + 1] = make_float2(t.y, t.y);
                win[R - 1 + tr][4 * v + 2] = make_float2(t.z, t.z); win[R - 1 + tr][4 * v + 3] = make_float2(t.w, t.w);
            }
        }
        bool row_ok[TR];
#pragma unroll
        for (int tr = 0; tr < TR; ++tr) row_ok[tr] = (p + tr < th);

        float* yout = y + ((size_t)n * K * P + (size_t)(row0 + p)) * Q + q0;
        const float4* wf = wsm4;
#pragma unroll 1
        for (int i = 0; i < pairs; ++i, yout += 2 * plane, wf += RS2) {
            float2 acc[TR][kVec];
#pragma unroll
            for (int tr = 0; tr < TR; ++tr)
#pragma unroll
                for (int j = 0; j < kVec; ++j) acc[tr][j] = make_float2(0.f, 0.f);
#pragma unroll
            for (int u = 0; u < RS2; ++u) {
                const float4 w2 = wf[u];
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int t = 2 * u + h;
                    if (t < RS) {
                        const int r = t / S, s2 = t % S;
                        const float2 wv = h == 0 ? make_float2(w2.x, w2.y) : make_float2(w2.z, w2.w);
#pragma unroll
                        for (int tr = 0; tr < TR; ++tr)
#pragma unroll
                            for (int j = 0; j < kVec; ++j)
                                acc[tr][j] = __ffma2_rn(win[tr + r][s2 + j], wv, acc[tr][j]);
                    }
                }
            }
            const bool second = (2 * i + 1 < K);
#pragma unroll
            for (int tr = 0; tr < TR; ++tr) {
                if (row_ok[tr]) {
                    float* o = yout + (size_t)tr * Q;
                    if (vec_ok) {
                        store4(o, make_float4(acc[tr][0].x, acc[tr][1].x, acc[tr][2].x, acc[tr][3].x));
                        if (second) store4(o + plane, make_float4(acc[tr][0].y, acc[tr][1].y, acc[tr][2].y, acc[tr][3].y));
                    } else {
#pragma unroll
                        for (int j = 0; j < kVec; ++j)
                            if (q0 + j < Q) {
                                __stcs(o + j, acc[tr][j].x);
                                if (second) __stcs(o + plane + j, acc[tr][j].y);
                            }
                    }
                }
            }
        }
#pragma unroll
        for (int r = 0; r < R - 1; ++r)
#pragma unroll
            for (int c = 0; c < WC; ++c) win[r][c] = win[r + TR][c];
    }
}

template <int R, int S, int TR>
conv2d_status_t launch_packed(const float* x, const float* w, float* y, const Shape& sh, int tile_h, cudaStream_t stream)
{
    constexpr int RS2 = (R * S + 1) / 2;
    const size_t smem = (size_t)(tile_h + R - 1) * kPitch * sizeof(float) + (size_t)((sh.K + 1) / 2) * RS2 * sizeof(float4);
    auto kern = single_channel_packed_kernel<R, S, TR>;
    static size_t smem_done[64] = {};
    if (smem > 48 * 1024 && raise_smem_limit(reinterpret_cast<const void*>(kern), smem, smem_done) != cudaSuccess)
        return CONV2D_ERR_CUDA;
    dim3 grid((sh.Q + kTileW - 1) / kTileW, (sh.P + tile_h - 1) / tile_h, sh.N);
    const int vec_ld = (sh.W % 4 == 0) && (reinterpret_cast<uintptr_t>(x) % 16 == 0);
    const int vec_st = (sh.Q % 4 == 0) && (reinterpret_cast<uintptr_t>(y) % 16 == 0);
    kern<<<grid, kThreads, smem, stream>>>(x, w, y, sh.H, sh.W, sh.K, sh.P, sh.Q, tile_h, vec_ld, vec_st);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? CONV2D_OK : CONV2D_ERR_CUDA;
}

template <int R, int S, int TR, int WSRC>
conv2d_status_t launch_instance(const float* x, const float* w, float* y, const Shape& sh, int tile_h, cudaStream_t stream)
{
    constexpr int RSP = (R * S + 3) / 4 * 4;
    size_t smem = (size_t)(tile_h + R - 1) * kPitch * sizeof(float);
    if (WSRC == 1) smem += (size_t)sh.K * RSP * sizeof(float);
    auto kern = single_channel_kernel<R, S, TR, WSRC>;
    static size_t smem_done[64] = {};
    if (smem > 48 * 1024 && raise_smem_limit(reinterpret_cast<const void*>(kern), smem, smem_done) != cudaSuccess)
        return CONV2D_ERR_CUDA;
    dim3 grid((sh.Q + kTileW - 1) / kTileW, (sh.P + tile_h - 1) / tile_h, sh.N);
    const int vec_ld = (sh.W % 4 == 0) && (reinterpret_cast<uintptr_t>(x) % 16 == 0);
    const int vec_st = (sh.Q % 4 == 0) && (reinterpret_cast<uintptr_t>(y) % 16 == 0);
    kern<<<grid, kThreads, smem, stream>>>(x, w, y, sh.H, sh.W, sh.K, sh.P, sh.Q, tile_h, vec_ld, vec_st);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? CONV2D_OK : CONV2D_ERR_CUDA;
}

// Wide persistent variant for large images.
//
// Measured on B200: the output (97 % of the bytes) reaches HBM at 6.1-6.8 TB/s only when the pieces
// written close together in time form long contiguous runs (a thread block writing 8-16 KB of one
// output row at a time, its warps in step); 128-thread blocks writing 512-byte pieces into K planes
// reach 4.5-5.2 TB/s however cheap the arithmetic.  So here one 512-thread block owns kRowsW = 2048
// adjacent output columns and walks over row bands of `band_h` output rows; blocks are persistent and
// take bands round-robin, so the blocks running at any moment cover adjacent rows.  The input band
// (with halo) is brought in by 1-D bulk (TMA) copies, one per image row, into a double buffer guarded
// by mbarriers: the copy of the next band runs under the FMA loop of the current one (the prefetch of
// Algorithm 1, done by the copy engine instead of registers).  Arithmetic as in the packed kernel.
constexpr int kRowsThreads = 512;
constexpr int kRowsW = kRowsThreads * kVec;            // 2048 output columns per block
constexpr int kRowsPitch = kRowsW + 8;                 // staged floats per row
constexpr int kRowsPitch4 = kRowsPitch / 4;

template <int R, int S, int TR>
__global__ void __launch_bounds__(kRowsThreads, 1)
single_channel_rows_kernel(const float* __restrict__ x, const float* __restrict__ w, float* __restrict__ y,
                           int N, int H, int W, int K, int P, int Q, int band_h, int col_tiles, int items, int unit,
                           unsigned max_polls, int test_short_item)
{
    constexpr int NV = (S + kVec - 1 + 3) / 4;
    constexpr int WC = 4 * NV;
    constexpr int WR = R - 1 + TR;
    constexpr int RS = R * S;
    constexpr int RS2 = (RS + 1) / 2;

    extern __shared__ float4 smem4[];
    const int stage_f4 = (band_h + R - 1) * kRowsPitch4;
    float4* tiles4 = smem4;                                          // [2][band_h+R-1][kRowsPitch4]
    float4* wsm4 = smem4 + 2 * (size_t)stage_f4;
    const int pairs = (K + 1) / 2;
    uint64_t* full = reinterpret_cast<uint64_t*>(wsm4 + (size_t)pairs * RS2);   // [2]
    volatile uint32_t* abort_flag = reinterpret_cast<uint32_t*>(full + 2);

    const int tid = threadIdx.x;
    if (tid == 0) {
        ptx::mbar_init(&full[0], 1);
        ptx::mbar_init(&full[1], 1);
        *abort_flag = 0;
        ptx::fence_mbar_init();
    }
    for (int idx = tid; idx < pairs * RS2; idx += kRowsThreads) {
        const int i = idx / RS2, u = idx - i * RS2;
        const int f0 = 2 * i, f1 = 2 * i + 1, t0 = 2 * u, t1 = 2 * u + 1;
        float4 v;
        v.x = __ldg(w + (size_t)f0 * RS + t0);
        v.y = (f1 < K) ? __ldg(w + (size_t)f1 * RS + t0) : 0.f;
        v.z = (t1 < RS) ? __ldg(w + (size_t)f0 * RS + t1) : 0.f;
        v.w = (t1 < RS && f1 < K) ? __ldg(w + (size_t)f1 * RS + t1) : 0.f;
        wsm4[idx] = v;
    }
    __syncthreads();

    const int bands = (P + band_h - 1) / band_h;
    // item -> (image, band, column tile); the column tile varies fastest
    uint32_t issued[2] = {0u, 0u};                        // copies armed per stage (thread 0)
    auto issue = [&](int item, int stage) {               // thread 0 only
        const int ct = item % col_tiles;
        const int band = (item / col_tiles) % bands;
        const int n = item / (col_tiles * bands);
        const int row0 = band * band_h, col0 = ct * kRowsW;
        const int rows_in = min(band_h, P - row0) + R - 1;
        const int cols = min(kRowsPitch, W - col0);                   // multiple of 4 (W % 4 == 0)
        const uint32_t row_bytes = (uint32_t)cols * 4u;
        if (*abort_flag) return;                                      // a wait has run out: no further copies
        ++issued[stage];
        // (test hook: one item is armed for one row more than is copied, so that its wait runs out)
        ptx::mbar_arrive_expect_tx(&full[stage], row_bytes * (uint32_t)(rows_in + (item == test_short_item ? 1 : 0)));
        const float* src = x + ((size_t)n * H + row0) * W + col0;
        float4* dst = tiles4 + (size_t)stage * stage_f4;
        for (int r = 0; r < rows_in; ++r)
            ptx::bulk_g2s(dst + (size_t)r * kRowsPitch4, src + (size_t)r * W, row_bytes, &full[stage]);
    };

    int it = blockIdx.x;
    if (tid == 0 && it < items) issue(it, 0);
    const size_t plane = (size_t)P * Q;
    bool alive = true;
    for (int local = 0; it < items; it += gridDim.x, ++local) {
        const int stage = local & 1;
        __syncthreads();                                              // everyone is done reading the other buffer
        if (tid == 0 && it + (int)gridDim.x < items) issue(it + gridDim.x, stage ^ 1);
        if (alive && !ptx::mbar_wait_bounded(&full[stage], (uint32_t)(local >> 1) & 1u, abort_flag, max_polls)) alive = false;
        if (!alive) continue;                                         // keep meeting the barriers, do no work

        const int ct = it % col_tiles;
        const int band = (it / col_tiles) % bands;
        const int n = it / (col_tiles * bands);
        const int row0 = band * band_h, col0 = ct * kRowsW;
        const int th = min(band_h, P - row0);
        const int rows_in = th + R - 1;
        const int q0 = col0 + kVec * tid;
        if (q0 >= Q) continue;
        const float4* tile4 = tiles4 + (size_t)stage * stage_f4;

        float2 win[WR][WC];
#pragma unroll
        for (int r = 0; r < R - 1; ++r)
#pragma unroll
            for (int v = 0; v < NV; ++v) {
                const float4 t = tile4[r * kRowsPitch4 + tid + v];
                win[r][4 * v + 0] = make_float2(t.x, t.x); win[r][4 * v + 1] = make_float2(t.y, t.y);
                win[r][4 * v + 2] = make_float2(t.z, t.z); win[r][4 * v + 3] = make_float2(t.w, t.w);
            }
        for (int p = 0; p < th; p += TR) {
#pragma unroll
            for (int tr = 0; tr < TR; ++tr) {
                const int row = p + R - 1 + tr;
#pragma unroll
                for (int v = 0; v < NV; ++v) {
                    float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (row < rows_in) t = tile4[row * kRowsPitch4 + tid + v];
                    win[R - 1 + tr][4 * v + 0] = make_float2(t.x, t.x); win[R - 1 + tr][4 * v + 1] = make_float2(t.y, t.y);
                    win[R - 1 + tr][4 * v + 2] = make_float2(t.z, t.z); win[R - 1 + tr][4 * v + 3] = make_float2(t.w, t.w);
                }
            }
            bool row_ok[TR];
#pragma unroll
            for (int tr = 0; tr < TR; ++tr) row_ok[tr] = (p + tr < th);

            float* yout = y + ((size_t)n * K * P + (size_t)(row0 + p)) * Q + q0;
            const float4* wf = wsm4;
#pragma unroll 1
            for (int i = 0; i < pairs; ++i, yout += 2 * plane, wf += RS2) {
                float2 acc[TR][kVec];
#pragma unroll
                for (int tr = 0; tr < TR; ++tr)
#pragma unroll
                    for (int j = 0; j < kVec; ++j) acc[tr][j] = make_float2(0.f, 0.f);
#pragma unroll
                for (int u = 0; u < RS2; ++u) {
                    const float4 w2 = wf[u];
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const int t = 2 * u + h;
                        if (t < RS) {
                            const int r = t / S, s2 = t % S;
                            const float2 wv = h == 0 ? make_float2(w2.x, w2.y) : make_float2(w2.z, w2.w);
#pragma unroll
                            for (int tr = 0; tr < TR; ++tr)
#pragma unroll
                                for (int j = 0; j < kVec; ++j)
                                    acc[tr][j] = __ffma2_rn(win[tr + r][s2 + j], wv, acc[tr][j]);
                        }
                    }
                }
                const bool second = (2 * i + 1 < K);
#pragma unroll
                for (int tr = 0; tr < TR; ++tr) {
                    if (row_ok[tr]) {
                        float* o = yout + (size_t)tr * Q;
                        store_outputs(o, acc[tr][0].x, acc[tr][1].x, acc[tr][2].x, acc[tr][3].x, q0, Q, unit);
                        if (second)
                            store_outputs(o + plane, acc[tr][0].y, acc[tr][1].y, acc[tr][2].y, acc[tr][3].y, q0, Q, unit);
                    }
                }
            }
#pragma unroll
            for (int r = 0; r < R - 1; ++r)
#pragma unroll
                for (int c = 0; c < WC; ++c) win[r][c] = win[r + TR][c];
        }
    }
    __syncthreads();
    if (tid == 0 && *abort_flag) {
        // The last copy armed on each stage may still be in flight into this block's shared memory: give it a
        // bounded time to land (a copy that completed long ago answers at the first poll).
        uint32_t dummy = 0;
        for (int st = 0; st < 2; ++st)
            if (issued[st]) ptx::mbar_wait_bounded(&full[st], (issued[st] - 1u) & 1u, &dummy, 1u << 12);
        atomicExch(&g_device_timeout, 1u);
    }
}

template <int R, int S, int TR>
conv2d_status_t launch_rows(const float* x, const float* w, float* y, const Shape& sh, int band_h, cudaStream_t stream)
{
    constexpr int RS2 = (R * S + 1) / 2;
    const size_t smem = 2 * (size_t)(band_h + R - 1) * kRowsPitch * sizeof(float)
                      + (size_t)((sh.K + 1) / 2) * RS2 * sizeof(float4) + 64;
    if (smem > 227 * 1024) return CONV2D_ERR_UNSUPPORTED;
    auto kern = single_channel_rows_kernel<R, S, TR>;
    static size_t smem_done[64] = {};
    if (raise_smem_limit(reinterpret_cast<const void*>(kern), smem, smem_done) != cudaSuccess)
        return CONV2D_ERR_CUDA;
    const int col_tiles = (sh.Q + kRowsW - 1) / kRowsW;
    const long long items = (long long)sh.N * ((sh.P + band_h - 1) / band_h) * col_tiles;
    if (items > 0x7fffffffLL) return CONV2D_ERR_UNSUPPORTED;
    const int sms = sm_count();
    const int grid = (int)(items < sms ? items : sms);
    const int unit = (reinterpret_cast<uintptr_t>(y) % 16 != 0) ? 1 : (sh.Q % 4 == 0 ? 4 : (sh.Q % 2 == 0 ? 2 : 1));
    // Failure-detection test hooks (host-side injection only): a short wait bound and one item whose barrier
    // expects a row that is never copied, so that the wait expires and the time-out path can be checked.
    kern<<<grid, kRowsThreads, smem, stream>>>(x, w, y, sh.N, sh.H, sh.W, sh.K, sh.P, sh.Q, band_h, col_tiles, (int)items, unit,
                                               (unsigned)env_int("CONV2D_B200_SC_MAX_POLLS", 1 << 22),
                                               env_int("CONV2D_B200_SC_TEST_SHORT_ITEM", -1));
    count_launch();
    return cudaGetLastError() == cudaSuccess ? CONV2D_OK : CONV2D_ERR_CUDA;
}

// Wide persistent variant for rows that are only 8-byte aligned (Q = 2 mod 4, e.g. 3 x 3 or 7 x 7 taps on
// an image whose width is a multiple of 4).  Output row p starts 2*(p mod 2) floats past a 16-byte
// boundary.  Measured: writing such rows as two 64-bit pieces per thread (16 bytes apart across lanes)
// halves the store efficiency, and a plain float2-per-thread kernel beat the kernel above by 25-40 %.
// Here the rows are split into two classes by parity, one work item per class: for odd rows every
// thread's four outputs start two columns earlier, so that ALL stores are aligned 128-bit stores again
// (the two outputs that hang over the left image edge are masked).  A class walks down its band two
// rows at a time, one output row per step; both classes stage the same input band (input is a few
// per cent of the traffic).
constexpr int kShiftPitch = kRowsW + 16;               // staged floats per row: 4 before the tile, halo after
constexpr int kShiftPitch2 = kShiftPitch / 2;

template <int R, int S>
__global__ void __launch_bounds__(kRowsThreads, 1)
single_channel_rows_shift_kernel(const float* __restrict__ x, const float* __restrict__ w, float* __restrict__ y,
                                 int N, int H, int W, int K, int P, int Q, int band_h, int col_tiles, int items,
                                 unsigned max_polls, int test_short_item)
{
    constexpr int WC = (S + kVec - 1 + 1) / 2 * 2;      // window columns, even
    constexpr int RS = R * S;
    constexpr int RS2 = (RS + 1) / 2;

    extern __shared__ float4 smem4[];
    const int stage_f = (band_h + R - 1) * kShiftPitch;              // floats per stage
    float* tiles = reinterpret_cast<float*>(smem4);                  // [2][band_h+R-1][kShiftPitch]
    float4* wsm4 = smem4 + (2 * (size_t)stage_f) / 4;
    const int pairs = (K + 1) / 2;
    uint64_t* full = reinterpret_cast<uint64_t*>(wsm4 + (size_t)pairs * RS2);   // [2]
    volatile uint32_t* abort_flag = reinterpret_cast<uint32_t*>(full + 2);

    const int tid = threadIdx.x;
    if (tid == 0) {
        ptx::mbar_init(&full[0], 1);
        ptx::mbar_init(&full[1], 1);
        *abort_flag = 0;
        ptx::fence_mbar_init();
    }
    for (int idx = tid; idx < pairs * RS2; idx += kRowsThreads) {
        const int i = idx / RS2, u = idx - i * RS2;
        const int f0 = 2 * i, f1 = 2 * i + 1, t0 = 2 * u, t1 = 2 * u + 1;
        float4 v;
        v.x = __ldg(w + (size_t)f0 * RS + t0);
        v.y = (f1 < K) ? __ldg(w + (size_t)f1 * RS + t0) : 0.f;
        v.z = (t1 < RS) ? __ldg(w + (size_t)f0 * RS + t1) : 0.f;
        v.w = (t1 < RS && f1 < K) ? __ldg(w + (size_t)f1 * RS + t1) : 0.f;
        wsm4[idx] = v;
    }
    __syncthreads();

    const int bands = (P + band_h - 1) / band_h;
    // item -> (image, band, column tile, row class); the class varies fastest, then the column tile.
    // Staged column c of a row holds image column col0 - 4 + c.
    uint32_t issued[2] = {0u, 0u};                        // copies armed per stage (thread 0)
    auto issue = [&](int item, int stage) {               // thread 0 only
        const int rest = item >> 1;
        const int ct = rest % col_tiles;
        const int band = (rest / col_tiles) % bands;
        const int n = rest / (col_tiles * bands);
        const int row0 = band * band_h, col0 = ct * kRowsW;
        const int rows_in = min(band_h, P - row0) + R - 1;
        const int src_col = col0 >= 4 ? col0 - 4 : 0;
        const int dst_off = src_col - (col0 - 4);                     // 0 or 4 floats
        const int cols = min(kShiftPitch - dst_off, W - src_col);     // multiple of 4 (W % 4 == 0)
        const uint32_t row_bytes = (uint32_t)cols * 4u;
        if (*abort_flag) return;                                      // a wait has run out: no further copies
        ++issued[stage];
        // (test hook: one item is armed for one row more than is copied, so that its wait runs out)
        ptx::mbar_arrive_expect_tx(&full[stage], row_bytes * (uint32_t)(rows_in + (item == test_short_item ? 1 : 0)));
        const float* src = x + ((size_t)n * H + row0) * W + src_col;
        float* dst = tiles + (size_t)stage * stage_f + dst_off;
        for (int r = 0; r < rows_in; ++r)
            ptx::bulk_g2s(dst + (size_t)r * kShiftPitch, src + (size_t)r * W, row_bytes, &full[stage]);
    };

    int it = blockIdx.x;
    if (tid == 0 && it < items) issue(it, 0);
    const size_t plane = (size_t)P * Q;
    bool alive = true;
    for (int local = 0; it < items; it += gridDim.x, ++local) {
        const int stage = local & 1;
        __syncthreads();                                              // everyone is done reading the other buffer
        if (tid == 0 && it + (int)gridDim.x < items) issue(it + gridDim.x, stage ^ 1);
        if (alive && !ptx::mbar_wait_bounded(&full[stage], (uint32_t)(local >> 1) & 1u, abort_flag, max_polls)) alive = false;
        if (!alive) continue;                                         // keep meeting the barriers, do no work

        const int cls = it & 1;                                       // parity of the output rows of this item
        const int rest = it >> 1;
        const int ct = rest % col_tiles;
        const int band = (rest / col_tiles) % bands;
        const int n = rest / (col_tiles * bands);
        const int row0 = band * band_h, col0 = ct * kRowsW;           // band_h is even, so row0 is even
        const int th = min(band_h, P - row0);
        const int rows_in = th + R - 1;
        const int shift = 2 * cls;                                    // odd rows: start two columns earlier
        const int q0 = col0 + kVec * tid - shift;
        if (q0 >= Q || cls >= th) continue;
        // this thread's window starts at staged column 4*tid + 4 - shift (even: 64-bit loads)
        const float2* tile2 = reinterpret_cast<const float2*>(tiles + (size_t)stage * stage_f) + (4 * tid + 4 - shift) / 2;

        float2 win[R][WC];                                            // (x, x) pairs
        auto load_row = [&](int wr, int row) {
#pragma unroll
            for (int v = 0; v < WC / 2; ++v) {
                float2 t = make_float2(0.f, 0.f);
                if (row < rows_in) t = tile2[row * kShiftPitch2 + v];
                win[wr][2 * v] = make_float2(t.x, t.x);
                win[wr][2 * v + 1] = make_float2(t.y, t.y);
            }
        };
#pragma unroll
        for (int r = 0; r < R - 1; ++r) load_row(r, cls + r);
        const bool vec_ok = (q0 >= 0) && (q0 + 3 < Q);
        for (int p = cls; p < th; p += 2) {
            load_row(R - 1, p + R - 1);
            float* yout = y + ((size_t)n * K * P + (size_t)(row0 + p)) * Q + q0;
            const float4* wf = wsm4;
#pragma unroll 1
            for (int i = 0; i < pairs; ++i, yout += 2 * plane, wf += RS2) {
                float2 acc[kVec];
#pragma unroll
                for (int j = 0; j < kVec; ++j) acc[j] = make_float2(0.f, 0.f);
#pragma unroll
                for (int u = 0; u < RS2; ++u) {
                    const float4 w2 = wf[u];
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const int t = 2 * u + h;
                        if (t < RS) {
                            const int r = t / S, s2 = t % S;
                            const float2 wv = h == 0 ? make_float2(w2.x, w2.y) : make_float2(w2.z, w2.w);
#pragma unroll
                            for (int j = 0; j < kVec; ++j) acc[j] = __ffma2_rn(win[r][s2 + j], wv, acc[j]);
                        }
                    }
                }
                const bool second = (2 * i + 1 < K);
                if (vec_ok) {
                    store4(yout, make_float4(acc[0].x, acc[1].x, acc[2].x, acc[3].x));
                    if (second) store4(yout + plane, make_float4(acc[0].y, acc[1].y, acc[2].y, acc[3].y));
                } else {
#pragma unroll
                    for (int j = 0; j < kVec; ++j)
                        if (q0 + j >= 0 && q0 + j < Q) {
                            __stcs(yout + j, acc[j].x);
                            if (second) __stcs(yout + plane + j, acc[j].y);
                        }
                }
            }
            // slide down two rows: rows p+2 .. p+R-1 stay, row p+R is new (row p+R+1 is loaded next step)
#pragma unroll
            for (int r = 0; r + 2 < R; ++r)
#pragma unroll
                for (int c = 0; c < WC; ++c) win[r][c] = win[r + 2][c];
            if (R >= 2) load_row(R - 2, p + R);
        }
    }
    __syncthreads();
    if (tid == 0 && *abort_flag) {
        // as in the kernel above: wait (bounded) for the last copy armed on each stage
        uint32_t dummy = 0;
        for (int st = 0; st < 2; ++st)
            if (issued[st]) ptx::mbar_wait_bounded(&full[st], (issued[st] - 1u) & 1u, &dummy, 1u << 12);
        atomicExch(&g_device_timeout, 1u);
    }
}

template <int R, int S>
conv2d_status_t launch_rows_shift(const float* x, const float* w, float* y, const Shape& sh, int band_h, cudaStream_t stream)
{
    constexpr int RS2 = (R * S + 1) / 2;
    band_h &= ~1;                                           // the row classes need an even band height
    if (band_h < 2) band_h = 2;
    auto need = [&](int bh) {
        return 2 * (size_t)(bh + R - 1) * kShiftPitch * sizeof(float) + (size_t)((sh.K + 1) / 2) * RS2 * sizeof(float4) + 64;
    };
    while (band_h > 2 && need(band_h) > 227 * 1024) band_h -= 2;
    const size_t smem = need(band_h);
    if (smem > 227 * 1024) return CONV2D_ERR_UNSUPPORTED;
    auto kern = single_channel_rows_shift_kernel<R, S>;
    static size_t smem_done[64] = {};
    if (raise_smem_limit(reinterpret_cast<const void*>(kern), smem, smem_done) != cudaSuccess)
        return CONV2D_ERR_CUDA;
    const int col_tiles = (sh.Q + 2 + kRowsW - 1) / kRowsW;    // odd rows start two columns to the left
    const long long items = 2LL * sh.N * ((sh.P + band_h - 1) / band_h) * col_tiles;
    if (items > 0x7fffffffLL) return CONV2D_ERR_UNSUPPORTED;
    const int sms = sm_count();
    const int grid = (int)(items < sms ? items : sms);
    kern<<<grid, kRowsThreads, smem, stream>>>(x, w, y, sh.N, sh.H, sh.W, sh.K, sh.P, sh.Q, band_h, col_tiles, (int)items,
                                               (unsigned)env_int("CONV2D_B200_SC_MAX_POLLS", 1 << 22),
                                               env_int("CONV2D_B200_SC_TEST_SHORT_ITEM", -1));
    count_launch();
    return cudaGetLastError() == cudaSuccess ? CONV2D_OK : CONV2D_ERR_CUDA;
}

// The shifted kernel pays for its aligned stores with one output row per step, which suits the memory-bound
// 3 x 3 case (measured 0.652 -> 0.463 ms on 4096 x 4096, 32 filters); the FMA-bound 7 x 7 case measured
// slightly slower with it and stays on the kernel above.
template <int R, int S>
conv2d_status_t try_rows_shift(const float*, const float*, float*, const Shape&, int, cudaStream_t) { return CONV2D_ERR_UNSUPPORTED; }
template <>
conv2d_status_t try_rows_shift<3, 3>(const float* x, const float* w, float* y, const Shape& sh, int band_h, cudaStream_t stream)
{
    return launch_rows_shift<3, 3>(x, w, y, sh, band_h, stream);
}

template <int R, int S>
conv2d_status_t dispatch_rs(const float* x, const float* w, float* y, const Shape& sh, cudaStream_t stream)
{
    // Tuning knobs (benchmark ablations only): tile height, rows per step, packed/scalar FMA, tap source.
    int tile_h = env_int("CONV2D_B200_SC_TILE_H", 0);
    if (tile_h <= 0) {
        // 8 rows per block unless that leaves the machine short of blocks (small images): then fewer rows,
        // down to 2, aiming at four blocks per SM
        tile_h = 8;
        const long long col_tiles = (sh.Q + kTileW - 1) / kTileW;
        while (tile_h > 2 && col_tiles * ((sh.P + tile_h - 1) / tile_h) * sh.N < 4 * sm_count()) tile_h >>= 1;
    }
    if (tile_h < 1) tile_h = 1;
    if (tile_h > 64) tile_h = 64;
    if (tile_h > sh.P) tile_h = sh.P;
    const int tr = env_int("CONV2D_B200_SC_ROWS", R >= 7 ? 1 : 2);
    constexpr int RS2 = (R * S + 1) / 2;
    const int unit = env_int("CONV2D_B200_SC_UNIT", 0);      // per-thread unit ablation (benchmark only)
    if (unit == 1 || unit == 2 || unit == 4) {
        const conv2d_status_t st = unit == 1 ? launch_unit<R, S, 1>(x, w, y, sh, tile_h, stream)
                                 : unit == 2 ? launch_unit<R, S, 2>(x, w, y, sh, tile_h, stream)
                                             : launch_unit<R, S, 4>(x, w, y, sh, tile_h, stream);
        if (st != CONV2D_ERR_UNSUPPORTED) return st;
    }
    // Large images: the wide persistent kernels (they need 16-byte aligned input rows for the bulk copies).
    const bool rows_ok = sh.W % 4 == 0 && reinterpret_cast<uintptr_t>(x) % 16 == 0;
    if (rows_ok && env_int("CONV2D_B200_SC_WIDE", 1) != 0) {
        // Rows per work item: 8, or another height (4..16, as far as the double buffer fits) when that fills the last
        // round of work items over the SMs clearly better (2048 x 2048, 1 x 1: 256 items of 8 rows are 1.73 rounds
        // on 148 SMs, 146 items of 14 rows one round).  Every row below 8 costs a little (more halo rows, more
        // per-item set-up), hence the 1.5 % per row.
        // (Heights are multiples of the rows a step produces: an odd height would compute its last row twice.)
        auto pick_band = [&](int step, int item_factor, size_t pitch_bytes) {
            const int sms = sm_count();
            const long long col_tiles = (sh.Q + kRowsW - 1) / kRowsW;
            const size_t filter_bytes = (size_t)((sh.K + 1) / 2) * RS2 * sizeof(float4) + 64;
            int best = 8;
            double best_score = 0, score8 = 0;
            for (int bh = 16; bh >= 4; bh -= step) {
                if (bh % step || 2 * (size_t)(bh + R - 1) * pitch_bytes + filter_bytes > 227 * 1024) continue;
                const long long items = (long long)item_factor * sh.N * ((sh.P + bh - 1) / bh) * col_tiles;
                const long long rounds = (items + sms - 1) / sms;
                const double score = (double)items / (double)(rounds * sms) * (1.0 - 0.015 * (8 - bh > 0 ? 8 - bh : 0));
                if (bh == 8) score8 = score;
                if (score > best_score) { best_score = score; best = bh; }
            }
            return score8 >= best_score - 0.02 ? 8 : best;       // 8 rows unless another height is clearly better
        };
        const int forced_band = env_int("CONV2D_B200_SC_BAND_H", 0);
        int band_h = forced_band > 0 ? forced_band : pick_band((tr == 1 || R >= 7) ? 1 : 2, 1, kRowsPitch * sizeof(float));
        if (band_h < 1) band_h = 1;
        if (band_h > 16) band_h = 16;
        // Rows that are only 8-byte aligned: the variant that shifts odd rows by two columns.  Its aligned
        // 128-bit stores beat the tile kernel's 64-bit pairs already on mid-size images (3 x 3, 32 filters,
        // 1024 x 1024: 75 -> 41 us; 512 x 512: 26 -> 20 us), although half of its 2048 columns are idle there.
        if (sh.Q >= 384 && sh.Q % 4 == 2 && ((long long)sh.P * sh.Q) % 4 == 0 && reinterpret_cast<uintptr_t>(y) % 16 == 0 &&
            env_int("CONV2D_B200_SC_SHIFT", 1) != 0) {
            const conv2d_status_t st = try_rows_shift<R, S>(x, w, y, sh, forced_band > 0 ? band_h : pick_band(2, 2, kShiftPitch * sizeof(float)), stream);
            if (st != CONV2D_ERR_UNSUPPORTED) return st;
        }
        if (sh.Q >= env_int("CONV2D_B200_SC_WIDE_MINQ", 1024)) {
            const conv2d_status_t st = (tr == 1 || R >= 7) ? launch_rows<R, S, 1>(x, w, y, sh, band_h, stream)
                                                           : launch_rows<R, S, 2>(x, w, y, sh, band_h, stream);
            if (st != CONV2D_ERR_UNSUPPORTED) return st;
        }
    }
    if (env_int("CONV2D_B200_SC_PACKED", 1) != 0 &&
        (size_t)((sh.K + 1) / 2) * RS2 * sizeof(float4) <= 96 * 1024) {
        return (tr == 1 || R >= 7) ? launch_packed<R, S, 1>(x, w, y, sh, tile_h, stream)
                                   : launch_packed<R, S, 2>(x, w, y, sh, tile_h, stream);
    }
    constexpr int RSP = (R * S + 3) / 4 * 4;
    int wsrc = env_int("CONV2D_B200_SC_WSRC", 1);
    if ((size_t)sh.K * RSP * sizeof(float) > 64 * 1024) wsrc = 0;       // too many taps for the shared copy
    if (wsrc == 0) {
        if ((size_t)sh.K * R * S > (size_t)kConstFilterFloats) return launch_direct_fallback(x, w, y, sh, stream);
        if (cudaMemcpyToSymbolAsync(c_filters, w, (size_t)sh.K * R * S * sizeof(float), 0,
                                    cudaMemcpyDeviceToDevice, stream) != cudaSuccess)
            return CONV2D_ERR_CUDA;
        return tr == 1 ? launch_instance<R, S, 1, 0>(x, w, y, sh, tile_h, stream)
                       : launch_instance<R, S, 2, 0>(x, w, y, sh, tile_h, stream);
    }
    return tr == 1 ? launch_instance<R, S, 1, 1>(x, w, y, sh, tile_h, stream)
                   : launch_instance<R, S, 2, 1>(x, w, y, sh, tile_h, stream);
}

}  // namespace

cudaError_t consume_device_timeout(bool* raised)
{
    unsigned flag = 0;
    cudaError_t e = cudaMemcpyFromSymbol(&flag, g_device_timeout, sizeof flag);
    if (e != cudaSuccess) return e;
    *raised = flag != 0;
    if (flag != 0) {
        const unsigned zero = 0;
        e = cudaMemcpyToSymbol(g_device_timeout, &zero, sizeof zero);
    }
    return e;
}

conv2d_status_t launch_single_channel(const float* x, const float* w, float* y, const Shape& sh, cudaStream_t stream)
{
    if (sh.R == 1 && sh.S == 1) return dispatch_rs<1, 1>(x, w, y, sh, stream);
    if (sh.R == 3 && sh.S == 3) return dispatch_rs<3, 3>(x, w, y, sh, stream);
    if (sh.R == 5 && sh.S == 5) return dispatch_rs<5, 5>(x, w, y, sh, stream);
    if (sh.R == 7 && sh.S == 7) return dispatch_rs<7, 7>(x, w, y, sh, stream);
    return launch_direct_fallback(x, w, y, sh, stream);
}

}  // namespace conv2d_b200
