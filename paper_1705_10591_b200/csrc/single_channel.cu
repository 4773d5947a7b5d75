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

namespace conv2d_b200 {

__constant__ float c_filters[kConstFilterFloats];

namespace {

constexpr int kThreads = 128;
constexpr int kVec = 4;                       // outputs per thread per row (the paper's n)
constexpr int kTileW = kThreads * kVec;       // 512 output columns per block
constexpr int kPitch = kTileW + 8;            // staged columns per row (halo S-1 <= 8), floats
constexpr int kPitch4 = kPitch / 4;

__device__ __forceinline__ void store4(float* p, float4 v) { __stcs(reinterpret_cast<float4*>(p), v); }

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

template <int R, int S, int TR, int WSRC>
conv2d_status_t launch_instance(const float* x, const float* w, float* y, const Shape& sh, int tile_h, cudaStream_t stream)
{
    constexpr int RSP = (R * S + 3) / 4 * 4;
    size_t smem = (size_t)(tile_h + R - 1) * kPitch * sizeof(float);
    if (WSRC == 1) smem += (size_t)sh.K * RSP * sizeof(float);
    auto kern = single_channel_kernel<R, S, TR, WSRC>;
    if (smem > 48 * 1024) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return CONV2D_ERR_CUDA;
    }
    dim3 grid((sh.Q + kTileW - 1) / kTileW, (sh.P + tile_h - 1) / tile_h, sh.N);
    const int vec_ld = (sh.W % 4 == 0) && (reinterpret_cast<uintptr_t>(x) % 16 == 0);
    const int vec_st = (sh.Q % 4 == 0) && (reinterpret_cast<uintptr_t>(y) % 16 == 0);
    kern<<<grid, kThreads, smem, stream>>>(x, w, y, sh.H, sh.W, sh.K, sh.P, sh.Q, tile_h, vec_ld, vec_st);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? CONV2D_OK : CONV2D_ERR_CUDA;
}

int env_int(const char* name, int dflt)
{
    const char* v = getenv(name);
    return (v && *v) ? atoi(v) : dflt;
}

template <int R, int S>
conv2d_status_t dispatch_rs(const float* x, const float* w, float* y, const Shape& sh, cudaStream_t stream)
{
    // Tuning knobs (benchmark ablations only): tile height, rows per step, tap source.
    int tile_h = env_int("CONV2D_B200_SC_TILE_H", 16);
    if (tile_h < 1) tile_h = 1;
    if (tile_h > 64) tile_h = 64;
    if (tile_h > sh.P) tile_h = sh.P;
    const int tr = env_int("CONV2D_B200_SC_ROWS", 2);
    constexpr int RSP = (R * S + 3) / 4 * 4;
    int wsrc = env_int("CONV2D_B200_SC_WSRC", 1);
    if ((size_t)sh.K * RSP * sizeof(float) > 64 * 1024) wsrc = 0;       // too many taps for the shared copy
    if (wsrc == 0) {
        if ((size_t)sh.K * R * S > (size_t)kConstFilterFloats) return CONV2D_ERR_UNSUPPORTED;
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

conv2d_status_t launch_single_channel(const float* x, const float* w, float* y, const Shape& sh, cudaStream_t stream)
{
    if (sh.R == 1 && sh.S == 1) return dispatch_rs<1, 1>(x, w, y, sh, stream);
    if (sh.R == 3 && sh.S == 3) return dispatch_rs<3, 3>(x, w, y, sh, stream);
    if (sh.R == 5 && sh.S == 5) return dispatch_rs<5, 5>(x, w, y, sh, stream);
    if (sh.R == 7 && sh.S == 7) return dispatch_rs<7, 7>(x, w, y, sh, stream);
    return launch_direct_fallback(x, w, y, sh, stream);
}

}  // namespace conv2d_b200
