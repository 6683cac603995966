// What the fused step kernel reads: the work table's records, the per-step
// scalars and the mode constants of its template parameters.  Shared with the
// host planner; not part of the C ABI.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace novak {

// Per-tensor record in device memory: where the tensor's streams start.
struct __align__(16) TensorRec {
    float *p;          // parameters theta, fp32: where theta_t is written
    const void *g;     // gradient, fp32 or bf16, read only
    void *m;           // first moment   (Eq. 1), fp32, or bf16 under PRE_MOM16
    void *v;           // second moment  (Eq. 2), same type as m
    float *slow;       // slow weights   (Eq. 28), NULL when lookahead is off
    float *acc;        // running sum of the window's fast iterates (TRAJ_MEAN)
    float2 *mean;      // row means of the raw gradient (Eq. 26) as hi + lo, NULL: not centralized
    __nv_bfloat16 *p16; // bf16 copy of theta written by the step, NULL: none
    const float *p_in; // where theta_{t-1} is read: p itself, or the tensor's slice of the
                       // save buffer on the step behind a true-Nesterov look-ahead (the
                       // parameter tensor then still holds Eq. 10's extrapolated point)
    uint32_t row_len;  // elements per row (product of dimensions 1..d), 0: not centralized
    uint32_t reserved;
};
static_assert(sizeof(TensorRec) == 80, "TensorRec is 80 bytes");

// One unit of work: `len` consecutive elements of one tensor.
struct __align__(16) Chunk {
    int32_t tensor;
    int32_t len;
    int64_t offset;
};

// Per-step scalars, computed in double on the host and rounded once
// (Section 8.1: computed once per step and broadcast to every thread).
struct StepScalars {
    float beta1, omb1;     // coefficient of Eq. 1 at this step (Eq. 3 when warmed up), 1 - it
    float beta2, omb2;     // coefficient of Eq. 2 at this step (Eq. 4 when warmed up), 1 - it
    float blend_b1, blend_omb1;  // base beta1, 1-beta1 of the classical blend (Eq. 16)
    float beta_n;          // Eq. 13
    float inv_bc1, inv_bc2;// 1/(1-beta1^t), 1/(1-beta2^t)   (Eq. 5)
    float eps;
    float decay;           // 1 - alpha lambda              (Eq. 18)
    float step;            // alpha r_t                     (Eq. 8-9, 24a)
    float la_alpha;        // alpha_LA                      (Eq. 30)
    float k;               // lookahead period as a float (divisor of the running sum)
    float sparse_tau;      // Eq. 27: directions with |u| <= tau are dropped; -1 when off
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

// Gradient processing before the Nesterov approximation (phase 2; template
// parameter of the step kernel).
enum : int {
    PRE_NONE = 0,    // g as given
    PRE_SCALE = 1,   // g <- factor g, the clip factor read from device memory
    PRE_CENTER = 2,  // g <- factor (g - row mean) for tensors that have rows (Eq. 26)
    PRE_CENTER_ROWS = 3,  // Eq. 26 without a pass of its own: the step kernel's CTAs own whole
                          // rows and form the means themselves (no clipping, no factor)
    PRE_MASK = 3,
    // OR-ed onto the above: the step also stores a bf16 copy of the new parameters
    PRE_COPY16 = 4,
    // OR-ed onto the above: m and v are stored as bf16 (read back as stored, advanced
    // in fp32, the step uses the unrounded values, stored rounded to nearest even)
    PRE_MOM16 = 8
};

// Result of the gradient statistics pass, in device memory; the step kernel
// reads `factor` from here, so the host never waits for it.
struct __align__(16) PrepOut {
    double norm;       // global L2 norm of the raw gradient
    float factor;      // clip factor: c_clip/norm when norm > c_clip, else 1
    unsigned ticket;   // CTAs of the statistics kernel that have finished
    // automatic learning-rate scaling (Eq. 20-22); the two averages persist from step to step
    double pnorm;      // global L2 norm of the parameters before the step
    double g_bar;      // Eq. 20
    double theta_bar;  // Eq. 21
    float auto_scale;  // Eq. 22, 1 when the scaling is off
    float reserved;
    // sums of squares of this process's gradients and parameters; a group sharded over
    // several processes all-reduces the two before norm and factors are formed
    double local_sums[2];
};

}  // namespace novak
