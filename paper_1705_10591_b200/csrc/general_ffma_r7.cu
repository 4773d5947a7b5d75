// fp32 general-case kernel: the instances for 7 x 7 filters (2 channels per staged block).
#include "ffma_kernel.cuh"

namespace conv2d_b200 {

conv2d_status_t launch_ffma_7x7(const float* x, const float* w, float* y, const Shape& sh, cudaStream_t stream)
{
    return launch_instance<7, 7, 2>(x, w, y, sh, stream);
}

}  // namespace conv2d_b200
