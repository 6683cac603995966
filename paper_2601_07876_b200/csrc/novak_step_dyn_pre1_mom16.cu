// Graph-capturable step kernel instantiations, gradient pre-processing mode PRE_SCALE, moments
// stored as bf16.
#include "novak_step_dyn.cuh"

namespace novak {

void *step_dyn_kernel_pre1_mom16(int nesterov, int grad_dtype)
{
    return reinterpret_cast<void *>(pick_step_dyn_kernel<PRE_SCALE | PRE_MOM16>(nesterov, grad_dtype));
}

}  // namespace novak
