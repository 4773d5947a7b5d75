// General case on the fp32 CUDA cores (Section 4, Algorithm 2): dispatch to the tuned kernel's instances (the kernel
// and its design notes are in ffma_kernel.cuh; its instances are compiled per filter size in general_ffma_r*.cu), plus
// a shape-agnostic direct kernel for every other filter size.
#include "common.cuh"

namespace conv2d_b200 {

// The tuned instances, one translation unit per filter size (general_ffma_r*.cu).
conv2d_status_t launch_ffma_1x1(const float* x, const float* w, float* y, const Shape& sh, cudaStream_t stream);
conv2d_status_t launch_ffma_2x2(const float* x, const float* w, float* y, const Shape& sh, cudaStream_t stream);
conv2d_status_t launch_ffma_3x3(const float* x, const float* w, float* y, const Shape& sh, cudaStream_t stream);
conv2d_status_t launch_ffma_4x4(const float* x, const float* w, float* y, const Shape& sh, cudaStream_t stream);
conv2d_status_t launch_ffma_5x5(const float* x, const float* w, float* y, const Shape& sh, cudaStream_t stream);
conv2d_status_t launch_ffma_7x7(const float* x, const float* w, float* y, const Shape& sh, cudaStream_t stream);

namespace {

// One thread per output, loops over c, r, s in that order: correct for every shape, tuned for none.
__global__ void direct_kernel(const float* __restrict__ x, const float* __restrict__ w, float* __restrict__ y,
                              int C, int H, int W, int K, int R, int S, int P, int Q, long long total)
{
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long o = (long long)blockIdx.x * blockDim.x + threadIdx.x; o < total; o += stride) {
        const int q = (int)(o % Q);
        const int p = (int)((o / Q) % P);
        const int k = (int)((o / ((long long)Q * P)) % K);
        const int n = (int)(o / ((long long)Q * P * K));
        const float* xb = x + ((size_t)n * C * H + p) * W + q;
        const float* wb = w + (size_t)k * C * R * S;
        float acc = 0.f;
        for (int c = 0; c < C; ++c)
            for (int r = 0; r < R; ++r)
                for (int s = 0; s < S; ++s)
                    acc = fmaf(__ldg(xb + ((size_t)c * H + r) * W + s), __ldg(wb + ((size_t)c * R + r) * S + s), acc);
        y[o] = acc;
    }
}

}  // namespace

conv2d_status_t launch_direct_fallback(const float* x, const float* w, float* y, const Shape& sh, cudaStream_t stream)
{
    const long long total = (long long)sh.N * sh.K * sh.P * sh.Q;
    const int threads = 256;
    long long blocks = (total + threads - 1) / threads;
    if (blocks > (long long)sm_count() * 64) blocks = (long long)sm_count() * 64;
    direct_kernel<<<(unsigned)blocks, threads, 0, stream>>>(x, w, y, sh.C, sh.H, sh.W, sh.K, sh.R, sh.S, sh.P, sh.Q, total);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? CONV2D_OK : CONV2D_ERR_CUDA;
}

conv2d_status_t launch_general_ffma(const float* x, const float* w, float* y, const Shape& sh, cudaStream_t stream)
{
    constexpr int kFiltersPerBlock = 64;                     // (kTileK of the tuned kernel: grid.y counts blocks of 64 filters)
    if (sh.N > 65535 || (sh.K + kFiltersPerBlock - 1) / kFiltersPerBlock > 65535) return launch_direct_fallback(x, w, y, sh, stream);
    if (sh.R == 1 && sh.S == 1) return launch_ffma_1x1(x, w, y, sh, stream);
    if (sh.R == 2 && sh.S == 2) return launch_ffma_2x2(x, w, y, sh, stream);      // (stride-2 rewriting of 3 x 3)
    if (sh.R == 3 && sh.S == 3) return launch_ffma_3x3(x, w, y, sh, stream);
    if (sh.R == 4 && sh.S == 4) return launch_ffma_4x4(x, w, y, sh, stream);      // (stride-2 rewriting of 7 x 7)
    if (sh.R == 5 && sh.S == 5) return launch_ffma_5x5(x, w, y, sh, stream);
    if (sh.R == 7 && sh.S == 7) return launch_ffma_7x7(x, w, y, sh, stream);
    return launch_direct_fallback(x, w, y, sh, stream);
}

}  // namespace conv2d_b200
