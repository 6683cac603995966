// Graph-capturable step kernel instantiations, gradient pre-processing mode PRE_NONE.
#include "novak_step_dyn.cuh"

namespace novak {

void *step_dyn_kernel_pre0(int nesterov, int grad_dtype)
{
    return reinterpret_cast<void *>(pick_step_dyn_kernel<PRE_NONE>(nesterov, grad_dtype));
}

}  // namespace novak
