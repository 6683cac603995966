// Step kernel instantiations for the gradient as given, with
// the moments stored as bf16.
#include "novak_step_kernel.cuh"

namespace novak {

void *step_kernel_pre0_mom16(int nesterov, int grad_dtype, int la)
{
    return reinterpret_cast<void *>(pick_step_kernel<PRE_NONE | PRE_MOM16>(nesterov, grad_dtype, la));
}

}  // namespace novak
