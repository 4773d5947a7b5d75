// Internal declarations shared by the translation units of libconv2d_b200.
#pragma once

#include <cstdlib>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "conv2d_b200.h"

namespace conv2d_b200 {

// Problem extents, library symbols (N images, C channels, H x W image, K filters, R x S taps).
struct Shape {
    int N, C, H, W, K, R, S, P, Q;
    int pad_h = 0, pad_w = 0;   // zero padding; only the tensor-core path with patch addressing takes it natively
};

// Capacity of the per-device constant-memory filter bank of the single-channel kernel, in floats.
constexpr int kConstFilterFloats = 16384;

// Bytes reserved at the start of the workspace for the device status word.
constexpr size_t kStatusBytes = 256;

// Reads and clears the device word that kernels without a workspace raise when a bounded wait expires.
// Returns cudaSuccess and sets *raised, or the CUDA error.  The stream must already be idle.
cudaError_t consume_device_timeout(bool* raised);

// Every kernel launch goes through this so that conv2d_launch_count() is exact.
void count_launch(int launches = 1);

// Raises a kernel's dynamic shared-memory limit to `bytes` unless this call site already did so on the
// current device (`done`: one static array per call site, i.e. per kernel instance).  The runtime call costs a
// few microseconds, which matters for kernels that run for ten.
inline cudaError_t raise_smem_limit(const void* kernel, size_t bytes, size_t (&done)[64])
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64 && done[dev] >= bytes) return cudaSuccess;
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (e == cudaSuccess && dev >= 0 && dev < 64) done[dev] = bytes;
    return e;
}

// Multiprocessors of the current device (looked up once per device; 148 on B200, which is also the answer when
// the query fails).  Planners size their grids and pick their tiles from it.
inline int sm_count()
{
    static int cached[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (cached[dev] == 0) {
        int n = 0;
        cached[dev] = (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0) ? n : 148;
    }
    return cached[dev];
}

// Tuning and test switches come from the environment, but only in a process that was started with
// CONV2D_B200_TUNING set (looked up once): production calls never scan the environment, and stray variables
// cannot change what the library does.
inline int env_int(const char* name, int dflt)
{
    static const bool tuning = getenv("CONV2D_B200_TUNING") != nullptr;
    if (!tuning) return dflt;
    const char* v = getenv(name);
    return (v && *v) ? atoi(v) : dflt;
}

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

// The same for a kernel whose blocks form clusters of `cluster_x` consecutive blocks.
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                               unsigned cluster_x, Args... args)
{
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = env_int("CONV2D_B200_TF32_PDL", 1) != 0 ? 1 : 0;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = cluster_x;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Launchers.  Each returns CONV2D_OK, CONV2D_ERR_UNSUPPORTED (no instance) or CONV2D_ERR_CUDA.
conv2d_status_t launch_single_channel(const float* x, const float* w, float* y, const Shape& sh, cudaStream_t stream);
conv2d_status_t launch_general_ffma(const float* x, const float* w, float* y, const Shape& sh, cudaStream_t stream);
conv2d_status_t launch_direct_fallback(const float* x, const float* w, float* y, const Shape& sh, cudaStream_t stream);

// Tensor-core path.
bool tf32_supported(const Shape& sh);
size_t tf32_workspace_bytes(const Shape& sh);   // includes the status block
// (returns CONV2D_ERR_UNSUPPORTED without an instance, CONV2D_ERR_WORKSPACE when workspace_bytes is too small)
conv2d_status_t launch_general_tf32(const float* x, const float* w, float* y, const Shape& sh,
                                    void* workspace, size_t workspace_bytes, bool weights_packed, cudaStream_t stream);

// 1 x 1 filters with every operand moved by tensor-map (TMA) copies; `workspace` holds the status block and, for fp32
// shapes with more channels than a resident filter bank takes, the filters rounded to TF32 (`weights_packed`: they
// are there already).
// CONV2D_ERR_UNSUPPORTED when the shape or its alignment has no such instance (the caller then takes the general kernel).
bool pointwise_tma_supported(const Shape& sh, bool b16);
conv2d_status_t launch_pointwise_tma(const void* x, const void* w, float* y, const Shape& sh, bool b16, bool fp16,
                                     void* workspace, size_t workspace_bytes, bool weights_packed, cudaStream_t stream);
size_t pointwise_tma_workspace_extra(const Shape& sh, bool b16);   // bytes after the status block, 0 if none
int describe_pointwise_tma_plan(const Shape& sh, bool b16, char* text, size_t text_bytes);   // -1: no such instance

// Text description of the tensor-core plan of a shape (snprintf semantics: returns the length it needs).
int describe_tensor_core_plan(const Shape& sh, bool b16, char* text, size_t text_bytes);

// Same kernel with 16-bit operands (x, w hold bf16 or fp16 elements in the same NCHW / KCRS order), fp32 output.
bool b16_supported(const Shape& sh);
size_t b16_workspace_bytes(const Shape& sh);
conv2d_status_t launch_general_b16(const void* x, const void* w, float* y, const Shape& sh, bool fp16,
                                   void* workspace, size_t workspace_bytes, bool weights_packed, cudaStream_t stream);

// Variant of the tensor-core path whose scratch is a fixed array inside the library image.
constexpr size_t kNoAllocScratchBytes = kStatusBytes + (size_t)8 * 1024 * 1024;
// Status word of that array on the current device (false when no such call has run there); stream idle.
cudaError_t noalloc_device_timeout(bool* raised);
conv2d_status_t launch_general_tf32_noalloc(const float* x, const float* w, float* y, const Shape& sh,
                                            bool wait, cudaStream_t stream);

}  // namespace conv2d_b200
