// Graph-capturable step kernel instantiations, gradient pre-processing mode PRE_NONE, moments
// stored as bf16, storing a bf16 copy of the updated parameters as well.
#include "novak_step_dyn.cuh"

namespace novak {

void *step_dyn_kernel_pre0_copy_mom16(int nesterov, int grad_dtype)
{
    return reinterpret_cast<void *>(pick_step_dyn_kernel<PRE_NONE | PRE_COPY16 | PRE_MOM16>(nesterov, grad_dtype));
}

}  // namespace novak
