// fp32 general-case kernel: the instances for 1 x 1 filters (16 channels per staged block).
#include "ffma_kernel.cuh"

namespace conv2d_b200 {

conv2d_status_t launch_ffma_1x1(const float* x, const float* w, float* y, const Shape& sh, cudaStream_t stream)
{
    return launch_instance<1, 1, 16>(x, w, y, sh, stream);
}

}  // namespace conv2d_b200
