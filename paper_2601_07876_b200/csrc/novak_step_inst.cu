// Every instantiation of the step kernel for ONE gradient pre-processing mode.
// The build compiles this file once per mode, in parallel:
//   -DNOVAK_PRE_MODE=<PRE_NONE|PRE_SCALE|PRE_CENTER, optionally | PRE_COPY16 | PRE_MOM16,
//                     as a number>
//   -DNOVAK_INST_DYN   for the graph-capturable kernel (scalars and lookahead
//                      action read from device memory) instead of the plain one.
//   -DNOVAK_INST_ADAPT for the kernel that runs layer adaptation and the update
//                      in one launch (every mode but the row-owning ones).
// Each object exports one selector: step_kernel_mode<N>, step_dyn_kernel_mode<N>
// or step_adapt_kernel_mode<N>.
#ifndef NOVAK_PRE_MODE
#error "compile with -DNOVAK_PRE_MODE=<mode bits>"
#endif

// The row-owning kernel (PRE_CENTER_ROWS modes) runs in CTAs of 128 threads, eight
// resident per SM (six where lookahead arrays are read): see kOwnBlockThreads.
#if ((NOVAK_PRE_MODE) & 3) == 3 && !defined(NOVAK_INST_DYN) && !defined(NOVAK_INST_ADAPT)
#define NOVAK_BLOCK 128
#define NOVAK_MIN_CTAS 8
#define NOVAK_MIN_CTAS_WIDE 6
#endif

#define NOVAK_PASTE2(a, b) a##b
#define NOVAK_PASTE(a, b) NOVAK_PASTE2(a, b)

#ifdef NOVAK_INST_DYN
#include "novak_step_dyn.cuh"

namespace novak {

void *NOVAK_PASTE(step_dyn_kernel_mode, NOVAK_PRE_MODE)(int nesterov, int grad_dtype)
{
    return reinterpret_cast<void *>(pick_step_dyn_kernel<NOVAK_PRE_MODE>(nesterov, grad_dtype));
}

}  // namespace novak
#elif defined(NOVAK_INST_ADAPT)
#include "novak_step_adapt.cuh"

namespace novak {

void *NOVAK_PASTE(step_adapt_kernel_mode, NOVAK_PRE_MODE)(int nesterov, int grad_dtype, int la)
{
    return pick_step_adapt_kernel<NOVAK_PRE_MODE>(nesterov, grad_dtype, la);
}

#if (NOVAK_PRE_MODE) == 0
// The wait of the kernel's update part on its own (once in the library: this object).
cudaError_t launch_adapt_wait_probe(const unsigned long long *word, unsigned epoch,
                                    const unsigned *error, unsigned long long *out, cudaStream_t stream)
{
    novak_adapt_wait_probe_kernel<<<1, 32, 0, stream>>>(word, epoch, error, out);
    return cudaGetLastError();
}
#endif

}  // namespace novak
#else
#include "novak_step_kernel.cuh"

namespace novak {

void *NOVAK_PASTE(step_kernel_mode, NOVAK_PRE_MODE)(int nesterov, int grad_dtype, int la)
{
    return pick_step_kernel<NOVAK_PRE_MODE>(nesterov, grad_dtype, la);
}

}  // namespace novak
#endif
