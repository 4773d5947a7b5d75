// C-ABI boundary: argument validation, dispatch and the host-buffer convenience path.
#include <atomic>

#include "common.cuh"

namespace conv2d_b200 {

static std::atomic<unsigned long long> g_launches{0};
void count_launch(int launches) { g_launches.fetch_add((unsigned long long)launches, std::memory_order_relaxed); }

namespace {

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Validates extents and fills the derived output size.
conv2d_status_t make_shape(int N, int C, int H, int W, int K, int R, int S, Shape* sh)
{
    if (N <= 0 || C <= 0 || H <= 0 || W <= 0 || K <= 0 || R <= 0 || S <= 0) return CONV2D_ERR_SHAPE;
    if (R > H || S > W) return CONV2D_ERR_SHAPE;
    const long long P = H - R + 1, Q = W - S + 1;
    const long long lim = 0x7fffffffLL;   // kernels index single tensors with 32-bit element counts per image plane set
    if ((long long)N * C * H * W > 4 * lim || (long long)N * K * P * Q > 4 * lim) return CONV2D_ERR_SHAPE;
    if ((long long)C * H * W > lim || (long long)K * P * Q > lim || (long long)K * C * R * S > lim) return CONV2D_ERR_SHAPE;
    *sh = Shape{N, C, H, W, K, R, S, (int)P, (int)Q};
    return CONV2D_OK;
}

// Zero extension of every H x W plane by pad_h rows above and below and pad_w columns left and right.
// One block row (blockIdx.y) per plane, 32-bit arithmetic inside a plane.
__global__ void pad_planes_kernel(const float* __restrict__ x, float* __restrict__ xp, int H, int W, int pad_h, int pad_w,
                                  unsigned* status_to_clear)
{
    // (the fp32 path has no kernel that clears the status block in front of the workspace)
    if (status_to_clear && blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x < kStatusBytes / sizeof(unsigned))
        status_to_clear[threadIdx.x] = 0u;
    const int Hp = H + 2 * pad_h, Wp = W + 2 * pad_w;
    const float* src = x + (size_t)blockIdx.y * H * W;
    float* dst = xp + (size_t)blockIdx.y * Hp * Wp;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < Hp * Wp; i += gridDim.x * blockDim.x) {
        const int hp = i / Wp;
        const int h = hp - pad_h, wc = i - hp * Wp - pad_w;
        dst[i] = (h >= 0 && h < H && wc >= 0 && wc < W) ? __ldg(src + h * W + wc) : 0.f;
    }
}

size_t round_up_256(size_t v) { return (v + 255) / 256 * 256; }

// Strided convolution as a stride-1 convolution over stride*stride times as many channels ("space to depth"):
//   x2[n][(c*st + a)*st + b][h2][w2] = xz[n][c][st*h2 + a][st*w2 + b]      (xz = zero-padded x, 0 outside)
//   w2[k][(c*st + a)*st + b][r2][s2] = w[k][c][st*r2 + a][st*s2 + b]       (0 where st*r2 + a >= R or st*s2 + b >= S)
// so that sum_{c,r,s} xz[c][st*p + r][st*q + s] w[k][c][r][s] = sum over (c,a,b),(r2,s2) of x2[..][p + r2][q + s2] w2[..].
__global__ void space_to_depth_kernel(const float* __restrict__ x, float* __restrict__ x2, int H, int W,
                                      int pad_h, int pad_w, int st, int H2, int W2, unsigned* status_to_clear)
{
    if (status_to_clear && blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x < kStatusBytes / sizeof(unsigned))
        status_to_clear[threadIdx.x] = 0u;
    // blockIdx.y = source plane (n, c); it produces the st*st planes (a, b) of the rewritten image
    const float* src = x + (size_t)blockIdx.y * H * W;
    float* dst = x2 + (size_t)blockIdx.y * st * st * H2 * W2;
    const int per_plane = H2 * W2, total = st * st * per_plane;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x) {
        const int ab = i / per_plane, rem = i - ab * per_plane;
        const int a = ab / st, b = ab - a * st;
        const int h2 = rem / W2, w2 = rem - h2 * W2;
        const int h = st * h2 + a - pad_h, wc = st * w2 + b - pad_w;
        dst[i] = (h >= 0 && h < H && wc >= 0 && wc < W) ? __ldg(src + h * W + wc) : 0.f;
    }
}
__global__ void filters_to_depth_kernel(const float* __restrict__ w, float* __restrict__ w2, int K, int C, int R, int S,
                                        int st, int R2, int S2)
{
    const long long total = (long long)K * C * st * st * R2 * S2;
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
        long long r = i;
        const int s2 = (int)(r % S2); r /= S2;
        const int r2 = (int)(r % R2); r /= R2;
        const int b = (int)(r % st); r /= st;
        const int a = (int)(r % st); r /= st;
        const int c = (int)(r % C); r /= C;
        const int k = (int)r;
        const int rr = st * r2 + a, ss = st * s2 + b;
        w2[i] = (rr < R && ss < S) ? __ldg(w + (((size_t)k * C + c) * R + rr) * S + ss) : 0.f;
    }
}

// Derived sizes of the strided problem; returns false on a bad argument.
struct StridedGeom { int P, Q, C2, H2, W2, R2, S2; };
bool strided_geom(int C, int H, int W, int R, int S, int pad_h, int pad_w, int st, StridedGeom* g)
{
    if (st < 1 || st > 8 || pad_h < 0 || pad_w < 0 || pad_h > 4096 || pad_w > 4096) return false;
    if (C <= 0 || H <= 0 || W <= 0 || R <= 0 || S <= 0 || C > (1 << 20)) return false;
    const int Hz = H + 2 * pad_h, Wz = W + 2 * pad_w;
    if (R > Hz || S > Wz) return false;
    g->P = (Hz - R) / st + 1;
    g->Q = (Wz - S) / st + 1;
    g->R2 = (R + st - 1) / st;
    g->S2 = (S + st - 1) / st;
    g->C2 = C * st * st;
    g->H2 = g->P + g->R2 - 1;
    g->W2 = g->Q + g->S2 - 1;
    return true;
}

conv2d_status_t check_device()
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return CONV2D_ERR_CUDA;
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return CONV2D_ERR_CUDA;
    return major == 10 ? CONV2D_OK : CONV2D_ERR_ARCH;
}

}  // namespace
}  // namespace conv2d_b200

using namespace conv2d_b200;

extern "C" {

conv2d_status_t conv2d_fwd_workspace_size(int N, int C, int H, int W, int K, int R, int S,
                                          conv2d_algo_t algo, size_t* bytes)
{
    if (!bytes) return CONV2D_ERR_NULL;
    *bytes = 0;
    Shape sh;
    conv2d_status_t st = make_shape(N, C, H, W, K, R, S, &sh);
    if (st != CONV2D_OK) return st;
    switch (algo) {
        case CONV2D_ALGO_FFMA: return CONV2D_OK;
        case CONV2D_ALGO_TF32:
            if (!tf32_supported(sh)) return CONV2D_ERR_UNSUPPORTED;
            *bytes = tf32_workspace_bytes(sh);
            return CONV2D_OK;
        case CONV2D_ALGO_AUTO:
            if (tf32_supported(sh)) *bytes = tf32_workspace_bytes(sh);
            return CONV2D_OK;
        case CONV2D_ALGO_16BIT:
            if (!b16_supported(sh)) return CONV2D_ERR_UNSUPPORTED;
            *bytes = b16_workspace_bytes(sh);
            return CONV2D_OK;
        default: return CONV2D_ERR_UNSUPPORTED;
    }
}

conv2d_status_t conv2d_fwd_plan_describe(int N, int C, int H, int W, int K, int R, int S,
                                         conv2d_algo_t algo, char* text, size_t text_bytes)
{
    if (!text || text_bytes == 0) return CONV2D_ERR_NULL;
    text[0] = 0;
    Shape sh;
    conv2d_status_t st = make_shape(N, C, H, W, K, R, S, &sh);
    if (st != CONV2D_OK) return st;
    if (algo != CONV2D_ALGO_TF32 && algo != CONV2D_ALGO_AUTO && algo != CONV2D_ALGO_16BIT) return CONV2D_ERR_UNSUPPORTED;
    const int need = describe_tensor_core_plan(sh, algo == CONV2D_ALGO_16BIT, text, text_bytes);
    return (need < 0 || (size_t)need >= text_bytes) ? CONV2D_ERR_WORKSPACE : CONV2D_OK;
}

conv2d_status_t conv2d_fwd_single_channel(const float* x, const float* w, float* y,
                                          int N, int H, int W, int K, int R, int S,
                                          void* workspace, size_t workspace_bytes,
                                          unsigned flags, void* cuda_stream)
{
    (void)workspace; (void)workspace_bytes;
    if (!x || !w || !y) return CONV2D_ERR_NULL;
    Shape sh;
    conv2d_status_t st = make_shape(N, 1, H, W, K, R, S, &sh);
    if (st != CONV2D_OK) return st;
    if (!aligned16(x) || !aligned16(w) || !aligned16(y)) return CONV2D_ERR_ALIGN;
    if (flags != 0) return CONV2D_ERR_UNSUPPORTED;
    if (N > 65535) return CONV2D_ERR_UNSUPPORTED;
    st = check_device();
    if (st != CONV2D_OK) return st;
    return launch_single_channel(x, w, y, sh, static_cast<cudaStream_t>(cuda_stream));
}

// The general entry; *status_in_workspace (optional) is set when the tensor-core launcher ran, i.e. when the
// status block at the start of the workspace was cleared by this call and is the place to look for a time-out.
static conv2d_status_t general_dispatch(const float* x, const float* w, float* y,
                                        int N, int C, int H, int W, int K, int R, int S,
                                        conv2d_algo_t algo,
                                        void* workspace, size_t workspace_bytes,
                                        unsigned flags, void* cuda_stream, bool* status_in_workspace)
{
    if (status_in_workspace) *status_in_workspace = false;
    if (!x || !w || !y) return CONV2D_ERR_NULL;
    Shape sh;
    conv2d_status_t st = make_shape(N, C, H, W, K, R, S, &sh);
    if (st != CONV2D_OK) return st;
    if (!aligned16(x) || !aligned16(w) || !aligned16(y) || !aligned16(workspace)) return CONV2D_ERR_ALIGN;
    if (flags & ~(unsigned)CONV2D_FLAG_WEIGHTS_PACKED) return CONV2D_ERR_UNSUPPORTED;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);

    if (algo != CONV2D_ALGO_TF32 && algo != CONV2D_ALGO_AUTO && algo != CONV2D_ALGO_FFMA) return CONV2D_ERR_UNSUPPORTED;
    if (algo == CONV2D_ALGO_TF32 && !workspace) return tf32_supported(sh) ? CONV2D_ERR_NULL : CONV2D_ERR_UNSUPPORTED;
    st = check_device();
    if (st != CONV2D_OK) return st;
    if (algo != CONV2D_ALGO_FFMA && workspace) {
        // one planning pass: the launcher reports "no instance" or "workspace too small" itself
        st = launch_general_tf32(x, w, y, sh, workspace, workspace_bytes, (flags & CONV2D_FLAG_WEIGHTS_PACKED) != 0, stream);
        if (st == CONV2D_OK && status_in_workspace) *status_in_workspace = true;
        if (algo == CONV2D_ALGO_TF32 || (st != CONV2D_ERR_UNSUPPORTED && st != CONV2D_ERR_WORKSPACE)) return st;
    }
    return launch_general_ffma(x, w, y, sh, stream);
}

conv2d_status_t conv2d_fwd_general(const float* x, const float* w, float* y,
                                   int N, int C, int H, int W, int K, int R, int S,
                                   conv2d_algo_t algo,
                                   void* workspace, size_t workspace_bytes,
                                   unsigned flags, void* cuda_stream)
{
    return general_dispatch(x, w, y, N, C, H, W, K, R, S, algo, workspace, workspace_bytes, flags, cuda_stream, nullptr);
}

conv2d_status_t conv2d_fwd_general_16bit(const void* x16, const void* w16, float* y,
                                         int N, int C, int H, int W, int K, int R, int S,
                                         conv2d_operand_t operand, void* workspace, size_t workspace_bytes,
                                         unsigned flags, void* cuda_stream)
{
    if (!x16 || !w16 || !y || !workspace) return CONV2D_ERR_NULL;
    Shape sh;
    conv2d_status_t st = make_shape(N, C, H, W, K, R, S, &sh);
    if (st != CONV2D_OK) return st;
    if (!aligned16(x16) || !aligned16(w16) || !aligned16(y) || !aligned16(workspace)) return CONV2D_ERR_ALIGN;
    if (flags & ~(unsigned)CONV2D_FLAG_WEIGHTS_PACKED) return CONV2D_ERR_UNSUPPORTED;
    if (operand != CONV2D_OPERAND_BF16 && operand != CONV2D_OPERAND_FP16) return CONV2D_ERR_UNSUPPORTED;
    st = check_device();
    if (st != CONV2D_OK) return st;
    return launch_general_b16(x16, w16, y, sh, operand == CONV2D_OPERAND_FP16, workspace, workspace_bytes,
                              (flags & CONV2D_FLAG_WEIGHTS_PACKED) != 0, static_cast<cudaStream_t>(cuda_stream));
}

conv2d_status_t conv2d_fwd_padded_workspace_size(int N, int C, int H, int W, int K, int R, int S, int pad_h, int pad_w,
                                                 conv2d_algo_t algo, size_t* bytes)
{
    if (!bytes) return CONV2D_ERR_NULL;
    *bytes = 0;
    if (pad_h < 0 || pad_w < 0 || pad_h > 4096 || pad_w > 4096 || H <= 0 || W <= 0) return CONV2D_ERR_SHAPE;
    size_t inner = 0;
    const conv2d_status_t st = conv2d_fwd_workspace_size(N, C, H + 2 * pad_h, W + 2 * pad_w, K, R, S, algo, &inner);
    if (st != CONV2D_OK) return st;
    if (inner < kStatusBytes) inner = kStatusBytes;      // the status block is there for every algorithm
    *bytes = round_up_256(inner) + (size_t)N * C * (H + 2 * pad_h) * (W + 2 * pad_w) * sizeof(float);
    return CONV2D_OK;
}

conv2d_status_t conv2d_fwd_general_padded(const float* x, const float* w, float* y,
                                          int N, int C, int H, int W, int K, int R, int S, int pad_h, int pad_w,
                                          conv2d_algo_t algo, void* workspace, size_t workspace_bytes,
                                          unsigned flags, void* cuda_stream)
{
    if (!x || !w || !y || !workspace) return CONV2D_ERR_NULL;
    size_t need = 0, inner = 0;
    conv2d_status_t st = conv2d_fwd_padded_workspace_size(N, C, H, W, K, R, S, pad_h, pad_w, algo, &need);
    if (st != CONV2D_OK) return st;
    if (!aligned16(x) || !aligned16(w) || !aligned16(y) || !aligned16(workspace)) return CONV2D_ERR_ALIGN;
    if (flags & ~(unsigned)CONV2D_FLAG_WEIGHTS_PACKED) return CONV2D_ERR_UNSUPPORTED;
    if (algo != CONV2D_ALGO_TF32 && algo != CONV2D_ALGO_AUTO && algo != CONV2D_ALGO_FFMA) return CONV2D_ERR_UNSUPPORTED;
    if ((long long)N * C > 65535) return CONV2D_ERR_UNSUPPORTED;      // one block row of the extension kernel per plane
    if (workspace_bytes < need) return CONV2D_ERR_WORKSPACE;
    st = conv2d_fwd_workspace_size(N, C, H + 2 * pad_h, W + 2 * pad_w, K, R, S, algo, &inner);
    if (st != CONV2D_OK) return st;
    st = check_device();
    if (st != CONV2D_OK) return st;
    // The tensor-core kernel takes the padding itself where it has an instance with patch addressing (no extra
    // pass over x); its workspace is the front part of this call's workspace as usual.
    if (algo != CONV2D_ALGO_FFMA && (pad_h || pad_w)) {
        Shape shp;
        if (make_shape(N, C, H + 2 * pad_h, W + 2 * pad_w, K, R, S, &shp) == CONV2D_OK) {
            shp.H = H; shp.W = W; shp.pad_h = pad_h; shp.pad_w = pad_w;       // P, Q are those of the extended image
            const conv2d_status_t native = launch_general_tf32(x, w, y, shp, workspace, workspace_bytes,
                                                               (flags & CONV2D_FLAG_WEIGHTS_PACKED) != 0,
                                                               static_cast<cudaStream_t>(cuda_stream));
            if (native != CONV2D_ERR_UNSUPPORTED && native != CONV2D_ERR_WORKSPACE) return native;
        }
    }
    const bool own_status = inner < kStatusBytes;          // fp32 path: no workspace of its own
    float* xp = reinterpret_cast<float*>(static_cast<unsigned char*>(workspace) + round_up_256(own_status ? kStatusBytes : inner));
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const int plane_p = (H + 2 * pad_h) * (W + 2 * pad_w);
    const dim3 grid((unsigned)((plane_p + 1023) / 1024 > 64 ? 64 : (plane_p + 1023) / 1024), (unsigned)(N * C));
    pad_planes_kernel<<<grid, 256, 0, stream>>>(x, xp, H, W, pad_h, pad_w, own_status ? static_cast<unsigned*>(workspace) : nullptr);
    count_launch(1);
    if (cudaGetLastError() != cudaSuccess) return CONV2D_ERR_CUDA;
    return conv2d_fwd_general(xp, w, y, N, C, H + 2 * pad_h, W + 2 * pad_w, K, R, S, algo, workspace, inner, flags, cuda_stream);
}

conv2d_status_t conv2d_fwd_strided_workspace_size(int N, int C, int H, int W, int K, int R, int S, int pad_h, int pad_w,
                                                  int stride, conv2d_algo_t algo, size_t* bytes)
{
    if (!bytes) return CONV2D_ERR_NULL;
    *bytes = 0;
    StridedGeom g;
    if (N <= 0 || K <= 0 || !strided_geom(C, H, W, R, S, pad_h, pad_w, stride, &g)) return CONV2D_ERR_SHAPE;
    size_t inner = 0;
    const conv2d_status_t st = conv2d_fwd_workspace_size(N, g.C2, g.H2, g.W2, K, g.R2, g.S2, algo, &inner);
    if (st != CONV2D_OK) return st;
    if (inner < kStatusBytes) inner = kStatusBytes;
    *bytes = round_up_256(inner) + round_up_256((size_t)N * g.C2 * g.H2 * g.W2 * sizeof(float))
           + (size_t)K * g.C2 * g.R2 * g.S2 * sizeof(float);
    return CONV2D_OK;
}

conv2d_status_t conv2d_fwd_general_strided(const float* x, const float* w, float* y,
                                           int N, int C, int H, int W, int K, int R, int S, int pad_h, int pad_w, int stride,
                                           conv2d_algo_t algo, void* workspace, size_t workspace_bytes,
                                           unsigned flags, void* cuda_stream)
{
    if (!x || !w || !y || !workspace) return CONV2D_ERR_NULL;
    size_t need = 0, inner = 0;
    conv2d_status_t st = conv2d_fwd_strided_workspace_size(N, C, H, W, K, R, S, pad_h, pad_w, stride, algo, &need);
    if (st != CONV2D_OK) return st;
    if (!aligned16(x) || !aligned16(w) || !aligned16(y) || !aligned16(workspace)) return CONV2D_ERR_ALIGN;
    if (flags & ~(unsigned)CONV2D_FLAG_WEIGHTS_PACKED) return CONV2D_ERR_UNSUPPORTED;
    if (algo != CONV2D_ALGO_TF32 && algo != CONV2D_ALGO_AUTO && algo != CONV2D_ALGO_FFMA) return CONV2D_ERR_UNSUPPORTED;
    if ((long long)N * C > 65535) return CONV2D_ERR_UNSUPPORTED;      // one block row of the rewriting kernel per plane
    if (workspace_bytes < need) return CONV2D_ERR_WORKSPACE;
    if (stride == 1)            // nothing to rewrite: the padded entry (its workspace is a prefix of this one's)
        return conv2d_fwd_general_padded(x, w, y, N, C, H, W, K, R, S, pad_h, pad_w, algo, workspace, workspace_bytes, flags, cuda_stream);
    StridedGeom g;
    strided_geom(C, H, W, R, S, pad_h, pad_w, stride, &g);
    st = conv2d_fwd_workspace_size(N, g.C2, g.H2, g.W2, K, g.R2, g.S2, algo, &inner);
    if (st != CONV2D_OK) return st;
    st = check_device();
    if (st != CONV2D_OK) return st;
    const bool own_status = inner < kStatusBytes;
    unsigned char* base = static_cast<unsigned char*>(workspace);
    float* x2 = reinterpret_cast<float*>(base + round_up_256(own_status ? kStatusBytes : inner));
    float* w2 = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(x2) + round_up_256((size_t)N * g.C2 * g.H2 * g.W2 * sizeof(float)));
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    auto blocks_for = [](long long total) { long long b = (total + 255) / 256; return (unsigned)(b > sm_count() * 32LL ? sm_count() * 32LL : b); };
    {
        const int work = stride * stride * g.H2 * g.W2;
        const dim3 grid((unsigned)((work + 1023) / 1024 > 64 ? 64 : (work + 1023) / 1024), (unsigned)(N * C));
        space_to_depth_kernel<<<grid, 256, 0, stream>>>(x, x2, H, W, pad_h, pad_w, stride, g.H2, g.W2,
                                                        own_status ? static_cast<unsigned*>(workspace) : nullptr);
    }
    count_launch(1);
    if (!(flags & CONV2D_FLAG_WEIGHTS_PACKED)) {
        filters_to_depth_kernel<<<blocks_for((long long)K * g.C2 * g.R2 * g.S2), 256, 0, stream>>>(w, w2, K, C, R, S, stride, g.R2, g.S2);
        count_launch(1);
    }
    if (cudaGetLastError() != cudaSuccess) return CONV2D_ERR_CUDA;
    return conv2d_fwd_general(x2, w2, y, N, g.C2, g.H2, g.W2, K, g.R2, g.S2, algo, workspace, inner, flags, cuda_stream);
}

conv2d_status_t conv2d_fwd_general_noalloc(const float* x, const float* w, float* y,
                                           int N, int C, int H, int W, int K, int R, int S,
                                           int wait, void* cuda_stream)
{
    if (!x || !w || !y) return CONV2D_ERR_NULL;
    Shape sh;
    conv2d_status_t st = make_shape(N, C, H, W, K, R, S, &sh);
    if (st != CONV2D_OK) return st;
    if (!aligned16(x) || !aligned16(w) || !aligned16(y)) return CONV2D_ERR_ALIGN;
    st = check_device();
    if (st != CONV2D_OK) return st;
    return launch_general_tf32_noalloc(x, w, y, sh, wait != 0, static_cast<cudaStream_t>(cuda_stream));
}

conv2d_status_t conv2d_fwd_host(const float* x_host, const float* w_host, float* y_host,
                                float* x, float* w, float* y,
                                int N, int C, int H, int W, int K, int R, int S,
                                conv2d_algo_t algo,
                                void* workspace, size_t workspace_bytes, void* cuda_stream)
{
    if (!x_host || !w_host || !y_host || !x || !w || !y) return CONV2D_ERR_NULL;
    Shape sh;
    conv2d_status_t st = make_shape(N, C, H, W, K, R, S, &sh);
    if (st != CONV2D_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const size_t xb = (size_t)N * C * H * W * sizeof(float);
    const size_t wb = (size_t)K * C * R * S * sizeof(float);
    const size_t yb = (size_t)N * K * sh.P * sh.Q * sizeof(float);
    if (cudaMemcpyAsync(x, x_host, xb, cudaMemcpyHostToDevice, stream) != cudaSuccess) return CONV2D_ERR_CUDA;
    if (cudaMemcpyAsync(w, w_host, wb, cudaMemcpyHostToDevice, stream) != cudaSuccess) return CONV2D_ERR_CUDA;
    // Only the tensor-core launcher clears and uses the status block in the workspace; after any other kernel the
    // workspace (which may be NULL, of size 0, or never written) must not be read for a status.
    bool status_in_workspace = false;
    if (C == 1 && algo != CONV2D_ALGO_TF32)
        st = conv2d_fwd_single_channel(x, w, y, N, H, W, K, R, S, nullptr, 0, 0, cuda_stream);
    else
        st = general_dispatch(x, w, y, N, C, H, W, K, R, S, algo, workspace, workspace_bytes, 0, cuda_stream, &status_in_workspace);
    if (st != CONV2D_OK) return st;
    if (cudaMemcpyAsync(y_host, y, yb, cudaMemcpyDeviceToHost, stream) != cudaSuccess) return CONV2D_ERR_CUDA;
    return conv2d_get_status(status_in_workspace ? workspace : nullptr, cuda_stream);
}

conv2d_status_t conv2d_get_status(const void* workspace, void* cuda_stream)
{
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (cudaStreamSynchronize(stream) != cudaSuccess) return CONV2D_ERR_CUDA;
    bool raised = false;
    if (consume_device_timeout(&raised) != cudaSuccess) return CONV2D_ERR_CUDA;
    if (raised) return CONV2D_ERR_DEVICE_TIMEOUT;
    // the fixed array of conv2d_fwd_general_noalloc: its status word stays set until that entry's next call
    if (noalloc_device_timeout(&raised) != cudaSuccess) return CONV2D_ERR_CUDA;
    if (raised) return CONV2D_ERR_DEVICE_TIMEOUT;
    if (!workspace) return CONV2D_OK;
    unsigned word = 0;
    if (cudaMemcpy(&word, workspace, sizeof word, cudaMemcpyDeviceToHost) != cudaSuccess) return CONV2D_ERR_CUDA;
    return word == 0 ? CONV2D_OK : CONV2D_ERR_DEVICE_TIMEOUT;
}

const char* conv2d_status_string(conv2d_status_t status)
{
    switch (status) {
        case CONV2D_OK: return "ok";
        case CONV2D_ERR_NULL: return "a required pointer is NULL";
        case CONV2D_ERR_SHAPE: return "invalid shape (non-positive extent, filter larger than image, or too large)";
        case CONV2D_ERR_ALIGN: return "pointer not 16-byte aligned";
        case CONV2D_ERR_WORKSPACE: return "workspace too small";
        case CONV2D_ERR_UNSUPPORTED: return "no kernel instance for this algorithm/shape/flags";
        case CONV2D_ERR_ARCH: return "device is not compute capability 10.x (B200)";
        case CONV2D_ERR_CUDA: return "CUDA runtime error";
        case CONV2D_ERR_DEVICE_TIMEOUT: return "a bounded on-device wait expired";
        default: return "unknown status";
    }
}

unsigned long long conv2d_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

}  // extern "C"
