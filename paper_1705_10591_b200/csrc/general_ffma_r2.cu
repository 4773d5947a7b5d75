// fp32 general-case kernel: the instances for 2 x 2 filters (8 channels per staged block).
#include "ffma_kernel.cuh"

namespace conv2d_b200 {

conv2d_status_t launch_ffma_2x2(const float* x, const float* w, float* y, const Shape& sh, cudaStream_t stream)
{
    return launch_instance<2, 2, 8>(x, w, y, sh, stream);
}

}  // namespace conv2d_b200
