// Launch side of the graph-capturable step: the one-thread kernel that advances
// the device-resident step counter and scalar plan, and the selection of the
// step kernel that reads them.
#include "novak_plan.h"

#include "novak_internal.h"

#ifndef NOVAK_BLOCK
#define NOVAK_BLOCK 256
#endif

namespace novak {

void *step_dyn_kernel_pre0(int nesterov, int grad_dtype);
void *step_dyn_kernel_pre1(int nesterov, int grad_dtype);
void *step_dyn_kernel_pre2(int nesterov, int grad_dtype);

namespace {

// t <- t + 1 and everything the host planner would compute for that step, from
// the hyperparameters given by value and the learning rate and weight decay
// kept in device memory.
__global__ void novak_plan_kernel(DevPlan *__restrict__ dp, novak_host::Hyper h)
{
    asm volatile("griddepcontrol.launch_dependents;");
    asm volatile("griddepcontrol.wait;" ::: "memory");    // the previous step reads *dp
    if (blockIdx.x != 0 || threadIdx.x != 0) return;
    const long long t = dp->t + 1;
    h.lr = dp->lr;
    h.wd = dp->weight_decay;
    const novak_host::Plan p = novak_host::make_plan(h, t);
    dp->t = t;
    dp->s = novak_host::make_scalars(h, p);
    dp->la = novak_host::lookahead_action(h, t);
    dp->nesterov = p.nesterov;
    dp->rect_branch = p.rect_branch;
    dp->is_sync = p.is_sync;
    if (p.is_sync) {
        dp->n_syncs += 1;
        dp->last_sync = t;
    }
    dp->bc1 = p.bc1; dp->bc2 = p.bc2;
    dp->rho_inf = p.rho_inf; dp->rho_t = p.rho_t;
    dp->r_t = p.r_t; dp->step_size = p.step_size; dp->decay = p.decay;
    dp->beta1_t = p.beta1_t; dp->beta2_t = p.beta2_t;
}

using StepDynFn = void (*)(const Chunk *, int, const TensorRec *, const PrepOut *, const DevPlan *,
                           int);

}  // namespace

cudaError_t launch_plan(DevPlan *d_plan, const void *hyper, size_t hyper_bytes, int pdl,
                        cudaStream_t stream)
{
    if (!d_plan || !hyper || hyper_bytes != sizeof(novak_host::Hyper)) return cudaErrorInvalidValue;
    novak_host::Hyper h = *static_cast<const novak_host::Hyper *>(hyper);
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(1);
    lc.blockDim = dim3(32);
    lc.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = (pdl & 1) ? 1 : 0;
    return cudaLaunchKernelEx(&lc, novak_plan_kernel, d_plan, h);
}

cudaError_t launch_step_dyn(const Chunk *d_chunks, int n_chunks, const TensorRec *d_recs,
                            const PrepOut *prep, const DevPlan *d_plan, int nesterov,
                            int grad_dtype, const LaunchCfg &cfg, cudaStream_t stream)
{
    void *raw = nullptr;
    switch (cfg.pre) {
    case PRE_NONE: raw = step_dyn_kernel_pre0(nesterov, grad_dtype); break;
    case PRE_SCALE: raw = step_dyn_kernel_pre1(nesterov, grad_dtype); break;
    case PRE_CENTER: raw = step_dyn_kernel_pre2(nesterov, grad_dtype); break;
    default: break;
    }
    StepDynFn fn = reinterpret_cast<StepDynFn>(raw);
    if (!fn || !d_plan || n_chunks <= 0 || cfg.grid <= 0) return cudaErrorInvalidValue;
    if (cfg.pre != PRE_NONE && prep == nullptr) return cudaErrorInvalidValue;
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(static_cast<unsigned>(cfg.grid));
    lc.blockDim = dim3(NOVAK_BLOCK);
    lc.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = (cfg.pdl & 1) ? 1 : 0;
    return cudaLaunchKernelEx(&lc, fn, d_chunks, n_chunks, d_recs, prep, d_plan, cfg.reverse);
}

}  // namespace novak
