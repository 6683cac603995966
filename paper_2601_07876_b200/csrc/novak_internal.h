// Internal types shared by the host planner (novak_host.cpp) and the device
// code (novak_*.cu) of the NOVAK step library.  Not part of the C ABI.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace novak {

// Per-tensor record in device memory: where the tensor's streams start.
struct __align__(16) TensorRec {
    float *p;          // parameters theta, fp32, updated in place
    const void *g;     // gradient, fp32 or bf16, read only
    float *m;          // first moment   (Eq. 1)
    float *v;          // second moment  (Eq. 2)
    float *slow;       // slow weights   (Eq. 28), NULL when lookahead is off
    float *acc;        // running sum of the window's fast iterates (TRAJ_MEAN)
    float2 *mean;      // row means of the raw gradient (Eq. 26) as hi + lo, NULL: not centralized
    __nv_bfloat16 *p16; // bf16 copy of theta written by the step, NULL: none
    uint32_t row_len;  // elements per row (product of dimensions 1..d), 0: not centralized
    uint32_t reserved;
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
    PRE_MASK = 3,
    // OR-ed onto the above: the step also stores a bf16 copy of the new parameters
    PRE_COPY16 = 4
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
};

struct LaunchCfg {
    int grid;
    int reverse;     // walk the chunk table from the end
    int pdl;         // launch with programmatic stream serialization (bit 0)
    int pre;         // PRE_* (with PRE_COPY16 where a bf16 copy is written)
};

// Threads per CTA of the step kernel (fixed at compile time).
int step_block_threads();

// Resident CTAs per SM of the step kernel instantiation for these modes.
cudaError_t step_occupancy(int nesterov, int grad_dtype, int la, int pre, int *ctas_per_sm);

// Launches the fused step kernel.  Returns cudaErrorInvalidValue for a mode
// combination that has no instantiation.  `prep` may be NULL when cfg.pre is
// PRE_NONE; `trust` (one factor per tensor, Eq. 25) is NULL without layer
// adaptation.  The chunk entries' tensor indices address recs and trust, so
// d_chunks may point into the middle of the table.
cudaError_t launch_step(const Chunk *d_chunks, int n_chunks, const TensorRec *d_recs,
                        const PrepOut *prep, const float *trust, const StepScalars &s, int nesterov,
                        int grad_dtype, int la, const LaunchCfg &cfg, cudaStream_t stream);

// Layer-wise adaptation (Eq. 19 / 25), two kernels over the whole chunk table:
// per entry the sums of squares of theta_t and of this step's base direction
// u_t (moments advanced in registers, nothing stored) into chunk_p2 / chunk_u2
// (n_chunks doubles each), then one CTA per tensor adds its entries
// [tensor_first[i], tensor_first[i+1]) in order and writes
// trust[i] = clip(||theta|| / ||u||, 0.1, 10), 1 where ||u|| = 0.
cudaError_t launch_trust_stats(const Chunk *d_chunks, int n_chunks, const TensorRec *d_recs,
                               int n_tensors, const int *tensor_first, const PrepOut *prep,
                               const StepScalars &s, int nesterov, int grad_dtype, int pre,
                               double *chunk_u2, double *chunk_p2, float *trust, int pdl,
                               cudaStream_t stream);

// One unit of work of the statistics pass for a tensor with rows (Eq. 26).
// Rows of up to kRowWarpMax elements: n_rows (a multiple of 8 but for a tensor's
// last unit) whole rows starting at row0
// (part_len = 0), a warp (or, below 128 elements, a thread) per row.  Longer
// rows: one slice [part_off, part_off + part_len) of row row0 for the whole
// CTA; the row is cut into n_parts slices of at most kRowUnitElems elements, of
// which this is number part_idx (units of one row are consecutive in the table).
struct __align__(16) RowUnit {
    int32_t tensor;
    uint32_t row0;
    uint32_t n_rows;
    uint32_t part_off;
    uint32_t part_len;
    uint32_t n_parts;
    uint32_t part_idx;
    uint32_t reserved;
};

// Elements a row unit aims at, and rows per unit where a thread takes a row.
constexpr uint32_t kRowUnitElems = 8192;
constexpr uint32_t kRowUnitThreads = 256;
constexpr uint32_t kRowWarpMax = 2048;     // longest row a single warp streams

// What the statistics pass works on, all in device memory.
struct StatsPlan {
    const Chunk *plain;      // chunk-table entries of the tensors without rows
    int n_plain;
    const RowUnit *units;    // row units of the tensors with rows
    int n_units;
    const TensorRec *recs;
    const Chunk *chunks;     // the whole chunk table (parameter norm of Eq. 21)
    int n_chunks;
    double *part_sq;         // grad_stats_work(n_plain, n_units, fp32) doubles (bf16 needs fewer)
    double *part_sum;        // n_units doubles
    double *chunk_psq;       // n_chunks doubles, NULL without Eq. 20-22
    double *cta_sq;          // 2 x grad_stats_ctas(...) doubles
    PrepOut *prep;
};

// CTAs of the first kernel (= sums of squares it leaves), CTAs of the second.
int grad_stats_work(int n_plain, int n_units, int grad_dtype);
int grad_stats_ctas(int n_work, int n_chunks);

// Launches the gradient statistics pass (two kernels; three with auto_gamma >
// 0, which adds the sum of squares of the parameters): the global norm of the
// raw gradient and the clip factor into *prep, the row means of Eq. 26 into
// the tensor records' mean arrays, and Eq. 20-22's averages and factor into
// *prep (the factor is written as 1 when auto_gamma = 0).
cudaError_t launch_grad_stats(const StatsPlan &plan, int grad_dtype, double c_clip,
                              double auto_gamma, int pdl, cudaStream_t stream);

// ---- work table for callers that cannot allocate device memory --------------
// Capacity of the statically allocated table behind novak_step_noalloc.
constexpr int kNoAllocMaxTensors = 4096;
constexpr int kNoAllocMaxChunks = 131072;

// Device addresses of the static table on the CURRENT device (resolved once per
// device with cudaGetSymbolAddress).  No allocation.
cudaError_t noalloc_table(TensorRec **d_recs, Chunk **d_chunks);

}  // namespace novak
