// Graph-capturable form of the step kernel (template; instantiated by
// novak_step_dyn_pre*.cu).  Same arithmetic, same access pattern and the same
// building blocks as novak_step_kernel, but the per-step scalars and the
// lookahead action are read from device memory (the armed slot of DevPlan),
// so that a captured launch replays as the NEXT step rather than as the
// captured one.  The kernel only reads the plan; novak_plan_next_kernel,
// launched behind it, advances it.  The lookahead action, a
// template parameter of the plain kernel, is a uniform run-time switch here.
#pragma once

#include "novak_step_kernel.cuh"

#ifndef NOVAK_DYN_MIN_CTAS
#define NOVAK_DYN_MIN_CTAS 4
#endif

namespace novak {
namespace {

// The plain kernel's loop over chunk-table entries for one lookahead action.
template <int NEST, int GT, int LA, int PRE>
__device__ __forceinline__ void dyn_entries(const Chunk *__restrict__ chunks, int n_chunks,
                                            const TensorRec *__restrict__ recs, const PreArgs &pre0,
                                            const float *trust,
                                            const StepScalars &s, int reverse, int c, Chunk ch,
                                            TensorRec r)
{
    PreArgs pre = pre0;
#pragma unroll 1
    for (;;) {
        // Eq. 24a: the tensor's trust ratio stretches the step (layer adaptation)
        pre.step = trust != nullptr ? pre0.step * trust[ch.tensor] : pre0.step;
        pre.mean = ((PRE & PRE_MASK) == PRE_CENTER) ? r.mean : nullptr;
        pre.row_len = r.row_len;
        pre.elem0 = static_cast<uint32_t>(ch.offset);
        pre.copy = ((PRE & PRE_COPY16) != 0) ? r.p16 + ch.offset : nullptr;
        run_entry<NEST, GT, LA, PRE>(ch, r, s, pre);
        c += gridDim.x;
        if (c >= n_chunks) break;
        ch = chunks[reverse ? n_chunks - 1 - c : c];
        r = recs[ch.tensor];
    }
}

// PRE: PRE_NONE, PRE_SCALE or PRE_CENTER, with or without PRE_COPY16 and PRE_MOM16.  The
// kernel holds every lookahead action's code; at four resident CTAs per SM (64
// registers) it spills a little on the heavier actions, which costs less than
// the lost CTA of the 80-register build when the gradient is pre-processed.
template <int NEST, int GT, int PRE>
__global__ void __launch_bounds__(NOVAK_BLOCK, NOVAK_DYN_MIN_CTAS)
novak_step_dyn_kernel(const Chunk *__restrict__ chunks, int n_chunks,
                      const TensorRec *__restrict__ recs, const PrepOut *prep,
                      const float *trust, const DevPlan *plan, int reverse)
{
    const int c = blockIdx.x;
    if (c >= n_chunks) return;
    const Chunk ch = chunks[reverse ? n_chunks - 1 - c : c];
    const TensorRec r = recs[ch.tensor];
    grid_dependency_wait();              // the previous plan kernel's (and the statistics pass's) output
    // Only now may the plan kernel behind this one start: it reads the step
    // counter, which the plan kernel in front has just finished writing.
    grid_dependency_release();

    const PlanSlot *slot = &plan->slot[plan->t & 1];
    const StepScalars s = slot->s;
    const int la = slot->la;
    PreArgs pre;
    pre.copy = nullptr;
    pre.factor = 1.0f;
    pre.step = s.step;
    if constexpr ((PRE & PRE_MASK) != PRE_NONE) {
        pre.factor = prep->factor;
        pre.step *= prep->auto_scale;
    }
    switch (la) {
#define NOVAK_DYN_CASE(X) \
    case (X): dyn_entries<NEST, GT, (X), PRE>(chunks, n_chunks, recs, pre, trust, s, reverse, c, ch, r); break;
        NOVAK_DYN_CASE(LA_NONE)
        NOVAK_DYN_CASE(LA_S_INIT | LA_S_WRITE)
        NOVAK_DYN_CASE(LA_S_INIT | LA_S_WRITE | LA_SYNC)
        NOVAK_DYN_CASE(LA_S_READ | LA_S_WRITE | LA_SYNC)
        NOVAK_DYN_CASE(LA_A_WRITE)
        NOVAK_DYN_CASE(LA_A_WRITE | LA_S_INIT | LA_S_WRITE)
        NOVAK_DYN_CASE(LA_A_READ | LA_A_WRITE)
        NOVAK_DYN_CASE(LA_A_READ | LA_S_READ | LA_S_WRITE | LA_SYNC | LA_TRAJ)
#undef NOVAK_DYN_CASE
    default: break;                      // not a lookahead action: leave everything untouched
    }
}

using StepDynFn = void (*)(const Chunk *, int, const TensorRec *, const PrepOut *, const float *,
                           const DevPlan *, int);

template <int PRE>
StepDynFn pick_step_dyn_kernel(int nesterov, int grad_dtype)
{
    const bool bf = grad_dtype == NOVAK_GRAD_BF16;
    if (grad_dtype != NOVAK_GRAD_F32 && !bf) return nullptr;
    switch (nesterov) {
    case NOVAK_NESTEROV_NONE:
        return bf ? novak_step_dyn_kernel<NOVAK_NESTEROV_NONE, NOVAK_GRAD_BF16, PRE>
                  : novak_step_dyn_kernel<NOVAK_NESTEROV_NONE, NOVAK_GRAD_F32, PRE>;
    case NOVAK_NESTEROV_APPROX:
        return bf ? novak_step_dyn_kernel<NOVAK_NESTEROV_APPROX, NOVAK_GRAD_BF16, PRE>
                  : novak_step_dyn_kernel<NOVAK_NESTEROV_APPROX, NOVAK_GRAD_F32, PRE>;
    case NOVAK_NESTEROV_CLASSICAL:
        return bf ? novak_step_dyn_kernel<NOVAK_NESTEROV_CLASSICAL, NOVAK_GRAD_BF16, PRE>
                  : novak_step_dyn_kernel<NOVAK_NESTEROV_CLASSICAL, NOVAK_GRAD_F32, PRE>;
    default: return nullptr;
    }
}

}  // namespace
}  // namespace novak
