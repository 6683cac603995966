// Step kernel instantiations for centralized and scaled gradients.
#include "novak_step_kernel.cuh"

namespace novak {

void *step_kernel_pre2(int nesterov, int grad_dtype, int la)
{
    return reinterpret_cast<void *>(pick_step_kernel<PRE_CENTER>(nesterov, grad_dtype, la));
}

}  // namespace novak
