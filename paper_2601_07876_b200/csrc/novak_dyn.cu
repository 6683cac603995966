// Launch side of the graph-capturable step: the one-thread kernels that keep the
// device-resident step counter and scalar plan, and the selection of the step
// kernel that reads them.
#include "novak_plan.h"

#include "novak_internal.h"

#ifndef NOVAK_BLOCK
#define NOVAK_BLOCK 256
#endif

namespace novak {

// novak_step_inst.cu, compiled once per gradient pre-processing mode with
// -DNOVAK_INST_DYN, holds the kernels; mode N exports step_dyn_kernel_mode<N>.
#define NOVAK_FOR_EACH_PRE_MODE(X) X(0) X(1) X(2) X(4) X(5) X(6) X(8) X(9) X(10) X(12) X(13) X(14)
#define NOVAK_DECLARE(N) void *step_dyn_kernel_mode##N(int nesterov, int grad_dtype);
NOVAK_FOR_EACH_PRE_MODE(NOVAK_DECLARE)
#undef NOVAK_DECLARE

namespace {

// Everything the host planner would compute for step t, from the
// hyperparameters given by value.
__device__ void fill_slot(PlanSlot *out, const novak_host::Hyper &h, long long t)
{
    const novak_host::Plan p = novak_host::make_plan(h, t);
    out->s = novak_host::make_scalars(h, p);
    out->la = novak_host::lookahead_action(h, t);
    out->nesterov = p.nesterov;
    out->rect_branch = p.rect_branch;
    out->is_sync = p.is_sync;
    out->bc1 = p.bc1; out->bc2 = p.bc2;
    out->rho_inf = p.rho_inf; out->rho_t = p.rho_t;
    out->r_t = p.r_t; out->step_size = p.step_size; out->decay = p.decay;
    out->beta1_t = p.beta1_t; out->beta2_t = p.beta2_t;
}

// After the host has uploaded counters or rates: the plan of the next step.
__global__ void novak_plan_arm_kernel(DevPlan *__restrict__ dp, novak_host::Hyper h)
{
    if (blockIdx.x != 0 || threadIdx.x != 0) return;
    h.lr = dp->lr;
    h.wd = dp->weight_decay;
    fill_slot(&dp->slot[dp->t & 1], h, dp->t);
}

// Launched behind the step kernel of step t.  That kernel releases its
// dependents only after its own wait, so the plan kernel in front of it has
// completed and dp->t is stable: the plan of step t + 1 is computed while step
// t runs and published, together with step t's synchronisation counters, once
// step t has completed.
__global__ void novak_plan_next_kernel(DevPlan *__restrict__ dp, novak_host::Hyper h)
{
    asm volatile("griddepcontrol.launch_dependents;");
    if (blockIdx.x != 0 || threadIdx.x != 0) return;
    const long long t = dp->t;
    h.lr = dp->lr;
    h.wd = dp->weight_decay;
    PlanSlot next;
    fill_slot(&next, h, t + 1);
    asm volatile("griddepcontrol.wait;" ::: "memory");     // step t has read slot[t & 1]
    dp->slot[(t + 1) & 1] = next;
    if (dp->slot[t & 1].is_sync) {
        dp->n_syncs += 1;
        dp->last_sync = t;
    }
    dp->t = t + 1;
}

using StepDynFn = void (*)(const Chunk *, int, const TensorRec *, const PrepOut *, const float *,
                           const DevPlan *, int);

}  // namespace

cudaError_t launch_plan_arm(DevPlan *d_plan, const void *hyper, size_t hyper_bytes,
                            cudaStream_t stream)
{
    if (!d_plan || !hyper || hyper_bytes != sizeof(novak_host::Hyper)) return cudaErrorInvalidValue;
    const novak_host::Hyper h = *static_cast<const novak_host::Hyper *>(hyper);
    novak_plan_arm_kernel<<<1, 32, 0, stream>>>(d_plan, h);
    return cudaGetLastError();
}

cudaError_t launch_plan_next(DevPlan *d_plan, const void *hyper, size_t hyper_bytes, int pdl,
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
    return cudaLaunchKernelEx(&lc, novak_plan_next_kernel, d_plan, h);
}

cudaError_t launch_step_dyn(const Chunk *d_chunks, int n_chunks, const TensorRec *d_recs,
                            const PrepOut *prep, const float *trust, const DevPlan *d_plan,
                            int nesterov, int grad_dtype, const LaunchCfg &cfg,
                            cudaStream_t stream)
{
    void *raw = nullptr;
    switch (cfg.pre) {
#define NOVAK_CASE(N) case N: raw = step_dyn_kernel_mode##N(nesterov, grad_dtype); break;
        NOVAK_FOR_EACH_PRE_MODE(NOVAK_CASE)
#undef NOVAK_CASE
    default: break;
    }
    StepDynFn fn = reinterpret_cast<StepDynFn>(raw);
    if (!fn || !d_plan || n_chunks <= 0 || cfg.grid <= 0) return cudaErrorInvalidValue;
    if ((cfg.pre & PRE_MASK) != PRE_NONE && prep == nullptr) return cudaErrorInvalidValue;
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(static_cast<unsigned>(cfg.grid));
    lc.blockDim = dim3(NOVAK_BLOCK);
    lc.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = (cfg.pdl & 1) ? 1 : 0;
    return cudaLaunchKernelEx(&lc, fn, d_chunks, n_chunks, d_recs, prep, trust, d_plan, cfg.reverse);
}

}  // namespace novak
