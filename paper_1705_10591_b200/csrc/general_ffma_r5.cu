// fp32 general-case kernel: the instances for 5 x 5 filters (4 channels per staged block).
#include "ffma_kernel.cuh"

namespace conv2d_b200 {

conv2d_status_t launch_ffma_5x5(const float* x, const float* w, float* y, const Shape& sh, cudaStream_t stream)
{
    return launch_instance<5, 5, 4>(x, w, y, sh, stream);
}

}  // namespace conv2d_b200
