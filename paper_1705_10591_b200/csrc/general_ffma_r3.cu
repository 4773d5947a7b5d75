// fp32 general-case kernel: the instances for 3 x 3 filters (8 channels per staged block).
#include "ffma_kernel.cuh"

namespace conv2d_b200 {

conv2d_status_t launch_ffma_3x3(const float* x, const float* w, float* y, const Shape& sh, cudaStream_t stream)
{
    return launch_instance<3, 3, 8>(x, w, y, sh, stream);
}

}  // namespace conv2d_b200
