// Graph-capturable step kernel instantiations, gradient pre-processing mode PRE_CENTER, moments
// stored as bf16.
#include "novak_step_dyn.cuh"

namespace novak {

void *step_dyn_kernel_pre2_mom16(int nesterov, int grad_dtype)
{
    return reinterpret_cast<void *>(pick_step_dyn_kernel<PRE_CENTER | PRE_MOM16>(nesterov, grad_dtype));
}

}  // namespace novak
