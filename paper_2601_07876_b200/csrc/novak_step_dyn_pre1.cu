// Graph-capturable step kernel instantiations, gradient pre-processing mode PRE_SCALE.
#include "novak_step_dyn.cuh"

namespace novak {

void *step_dyn_kernel_pre1(int nesterov, int grad_dtype)
{
    return reinterpret_cast<void *>(pick_step_dyn_kernel<PRE_SCALE>(nesterov, grad_dtype));
}

}  // namespace novak
