// Launch side of the kernel that runs layer adaptation and the update in one
// launch (novak_step_adapt.cuh): picks the instantiation and launches it.
#include "novak_internal.h"

#include "novak.h"

#ifndef NOVAK_BLOCK
#define NOVAK_BLOCK 256
#endif

namespace novak {

// novak_step_inst.cu, compiled with -DNOVAK_INST_ADAPT once per mode but the row-owning
// ones (PRE_NONE, PRE_SCALE, PRE_CENTER, each with or without the bf16 copy and bf16
// moments), exports step_adapt_kernel_mode<N>.
#define NOVAK_FOR_EACH_ADAPT_MODE(X) \
    X(0) X(1) X(2) X(4) X(5) X(6) X(8) X(9) X(10) X(12) X(13) X(14)
#define NOVAK_DECLARE(N) void *step_adapt_kernel_mode##N(int nesterov, int grad_dtype, int la);
NOVAK_FOR_EACH_ADAPT_MODE(NOVAK_DECLARE)
#undef NOVAK_DECLARE

namespace {
constexpr int kBlock = NOVAK_BLOCK;
}  // namespace

cudaError_t launch_step_adapt(const int *item_first, const Chunk *item_chunk, int n_items, int lag,
                              const TensorRec *d_recs, const PrepOut *prep, const int *tensor_first,
                              double *chunk_u2, double *chunk_p2, float *trust, AdaptCtl *ctl,
                              unsigned *arrived, unsigned long long *ready, unsigned *host_error,
                              float *direction, int slot_elems,
                              const StepScalars &s, unsigned epoch, int nesterov, int grad_dtype,
                              int la, const LaunchCfg &cfg, cudaStream_t stream)
{
    using Fn = void (*)(const int *, const Chunk *, int, int, const TensorRec *, const PrepOut *,
                        const int *, double *,
                        double *, float *, AdaptCtl *, unsigned *, unsigned long long *, unsigned *,
                        float *, int, StepScalars, unsigned);
    void *raw = nullptr;
    switch (cfg.pre) {
#define NOVAK_CASE(N) case N: raw = step_adapt_kernel_mode##N(nesterov, grad_dtype, la); break;
        NOVAK_FOR_EACH_ADAPT_MODE(NOVAK_CASE)
#undef NOVAK_CASE
    default: break;
    }
    Fn fn = reinterpret_cast<Fn>(raw);
    if (!fn || !item_first || !item_chunk || n_items <= 0 || lag < 0 || epoch == 0u || !ctl || !arrived || !ready ||
        !host_error || !tensor_first || ((cfg.pre & PRE_MASK) != PRE_NONE && !prep) || !chunk_u2 || !chunk_p2 || !trust || !direction ||
        slot_elems <= 0 || (slot_elems & 3) != 0)
        return cudaErrorInvalidValue;
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(static_cast<unsigned>(n_items) + static_cast<unsigned>(lag));
    lc.blockDim = dim3(kBlock);
    lc.dynamicSmemBytes = 0;
    lc.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = (cfg.pdl & 1) ? 1 : 0;
    return cudaLaunchKernelEx(&lc, fn, item_first, item_chunk, n_items, lag, d_recs, prep, tensor_first,
                              chunk_u2, chunk_p2, trust, ctl, arrived, ready, host_error, direction,
                              slot_elems, s, epoch);
}

}  // namespace novak
