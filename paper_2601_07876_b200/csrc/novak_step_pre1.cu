// Step kernel instantiations for the gradient scaled by the clip factor.
#include "novak_step_kernel.cuh"

namespace novak {

void *step_kernel_pre1(int nesterov, int grad_dtype, int la)
{
    return reinterpret_cast<void *>(pick_step_kernel<PRE_SCALE>(nesterov, grad_dtype, la));
}

}  // namespace novak
