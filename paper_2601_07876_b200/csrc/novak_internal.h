// Internal types shared by the host planner (novak_host.cpp) and the device
// code (novak_kernels.cu) of the NOVAK step library.  Not part of the C ABI.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace novak {

// Per-tensor record in device memory: where the tensor's streams start.
struct TensorRec {
    float *p;        // parameters theta, fp32, updated in place
    const void *g;   // gradient, fp32 or bf16, read only
    float *m;        // first moment   (Eq. 1)
    float *v;        // second moment  (Eq. 2)
    float *slow;     // slow weights   (Eq. 28), NULL when lookahead is off
    float *acc;      // running sum of the window's fast iterates (TRAJ_MEAN)
};

// One unit of work: `len` consecutive elements of one tensor.
struct __align__(16) Chunk {
    int32_t tensor;
    int32_t len;
    int64_t offset;
};

// Per-step scalars, computed in double on the host and rounded once
// (Section 8.1: computed once per step and broadcast to every thread).
struct StepScalars {
    float beta1, omb1;     // beta1, 1-beta1
    float beta2, omb2;     // beta2, 1-beta2
    float beta_n;          // Eq. 13
    float inv_bc1, inv_bc2;// 1/(1-beta1^t), 1/(1-beta2^t)   (Eq. 5)
    float eps;
    float decay;           // 1 - alpha lambda              (Eq. 18)
    float step;            // alpha r_t                     (Eq. 8-9, 24a)
    float la_alpha;        // alpha_LA                      (Eq. 30)
    float k;               // lookahead period as a float (divisor of the running sum)
};

// What the lookahead phase does on this step (bit mask; template parameter).
enum : int {
    LA_NONE = 0,
    LA_S_INIT = 1,   // slow_in := theta_in (first step, Eq. 28); slow is not read
    LA_S_READ = 2,
    LA_S_WRITE = 4,
    LA_A_READ = 8,   // running sum = acc + theta_fast (else = theta_fast)
    LA_A_WRITE = 16,
    LA_SYNC = 32,    // theta_out = slow_in + alpha_LA (target - slow_in)
    LA_TRAJ = 64     // target = running sum / k (else theta_fast)
};

struct LaunchCfg {
    int grid;
    int reverse;     // walk the chunk table from the end
    int pdl;         // launch with programmatic stream serialization
};

// Threads per CTA of the step kernel (fixed at compile time).
int step_block_threads();

// Resident CTAs per SM of the step kernel instantiation for these modes.
cudaError_t step_occupancy(int nesterov, int grad_dtype, int la, int *ctas_per_sm);

// Launches the fused step kernel.  Returns cudaErrorInvalidValue for a mode
// combination that has no instantiation.
cudaError_t launch_step(const Chunk *d_chunks, int n_chunks, const TensorRec *d_recs,
                        const StepScalars &s, int nesterov, int grad_dtype, int la,
                        const LaunchCfg &cfg, cudaStream_t stream);

// ---- work table for callers that cannot allocate device memory --------------
// Capacity of the statically allocated table behind novak_step_noalloc.
constexpr int kNoAllocMaxTensors = 4096;
constexpr int kNoAllocMaxChunks = 131072;

// Device addresses of the static table on the CURRENT device (resolved once per
// device with cudaGetSymbolAddress).  No allocation.
cudaError_t noalloc_table(TensorRec **d_recs, Chunk **d_chunks);

}  // namespace novak
