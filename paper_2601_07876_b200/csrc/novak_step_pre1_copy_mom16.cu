// Step kernel instantiations for the gradient scaled by the clip factor, with
// the moments stored as bf16, storing a bf16 copy of the
// updated parameters beside the fp32 ones.
#include "novak_step_kernel.cuh"

namespace novak {

void *step_kernel_pre1_copy_mom16(int nesterov, int grad_dtype, int la)
{
    return reinterpret_cast<void *>(pick_step_kernel<PRE_SCALE | PRE_COPY16 | PRE_MOM16>(nesterov, grad_dtype, la));
}

}  // namespace novak
