// Step kernel instantiations for the gradient as given (the default path).
#include "novak_step_kernel.cuh"

namespace novak {

void *step_kernel_pre0(int nesterov, int grad_dtype, int la)
{
    return reinterpret_cast<void *>(pick_step_kernel<PRE_NONE>(nesterov, grad_dtype, la));
}

}  // namespace novak
