// Internal types shared by the host side (novak_host*.cpp) and the device
// code (novak_*.cu) of the NOVAK step library.  Not part of the C ABI.
#pragma once

#include "novak_step_types.h"

namespace novak {

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

struct DevPlan;

// Layer-wise adaptation (Eq. 19 / 25), two kernels over the whole chunk table:
// per entry the sums of squares of theta_t and of this step's base direction
// u_t (moments advanced in registers, nothing stored) into chunk_p2 / chunk_u2
// (n_chunks doubles each), then one CTA per tensor adds its entries
// [tensor_first[i], tensor_first[i+1]) in order and writes
// trust[i] = clip(||theta|| / ||u||, 0.1, 10), 1 where ||u|| = 0.  With d_plan
// (graph-capturable step) the scalars come from its armed slot instead of s.
cudaError_t launch_trust_stats(const Chunk *d_chunks, int n_chunks, const TensorRec *d_recs,
                               int n_tensors, const int *tensor_first, const PrepOut *prep,
                               const StepScalars &s, const DevPlan *d_plan, int nesterov,
                               int grad_dtype, int pre, double *chunk_u2, double *chunk_p2,
                               float *trust, int pdl, cudaStream_t stream);

// ---- layer adaptation and step in one launch (novak_step_adapt.cuh) ---------
// State of the kernel in device memory, zero before the first launch.
constexpr int kAdaptGroupMax = 8;      // chunk-table entries per item at most
struct __align__(16) AdaptCtl {
    unsigned error;       // a bounded wait gave up (sticky)
    unsigned reserved[3];
};

// An item is up to kAdaptGroupMax consecutive chunk-table entries of one tensor,
// all but the last slot_elems long.  item_first: the n_items items' first chunk-
// table indices, tensors in order, every entry in one item; item_chunk: the
// item's entries as one span (tensor, offset of the first, total length).  CTA b
// takes the statistics of item b and the update of item b - lag; lag is at least
// the longest tensor's number of items minus one.  arrived: one counter per
// tensor; ready: one 64-bit word per tensor (launch number in the high half, the
// ratio's bits in the low half); both zero before the first launch.  epoch: a
// launch number no earlier launch on these buffers used (never 0).  host_error:
// device address of a host-mapped word, set to 1 if a wait gives up.  direction:
// scratch of slot_elems floats per chunk-table entry (entry c at c * slot_elems;
// slot_elems a multiple of 4 and at least the longest entry, the array 16-byte
// aligned), written and read within the launch.  prep: the statistics pass's
// output (clip factor, Eq. 22), needed unless cfg.pre is a PRE_NONE mode.  cfg.pre:
// any mode but the row-owning ones.  The grid is n_items + lag CTAs.
cudaError_t launch_step_adapt(const int *item_first, const Chunk *item_chunk, int n_items, int lag,
                              const TensorRec *d_recs, const PrepOut *prep, const int *tensor_first,
                              double *chunk_u2, double *chunk_p2, float *trust, AdaptCtl *ctl,
                              unsigned *arrived, unsigned long long *ready, unsigned *host_error,
                              float *direction, int slot_elems,
                              const StepScalars &s, unsigned epoch, int nesterov, int grad_dtype,
                              int la, const LaunchCfg &cfg, cudaStream_t stream);

// Runs that kernel's bounded wait on a word that nothing publishes (all zero, epoch
// non-zero): out[0] receives what the wait returned (0: it gave up), out[1] the
// nanoseconds it took.  error: a zero word in device memory.
cudaError_t launch_adapt_wait_probe(const unsigned long long *word, unsigned epoch,
                                    const unsigned *error, unsigned long long *out, cudaStream_t stream);

// One unit of work of the statistics pass for a tensor with rows (Eq. 26).
// Rows of up to kRowWarpMax elements: n_rows (a multiple of 8 but for a tensor's
// last unit) whole rows starting at row0
// (part_len = 0), a warp per row (half a warp up to kRowHalfWarpMax elements,
// eight lanes below 128, a thread below 32).  Longer
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

// Step kernel that centralizes by itself (PRE_CENTER_ROWS): rows of up to
// kOwnRowMax elements are owned by one CTA, in units of whole rows: as many as
// fit in kOwnUnitElems elements (at most kOwnUnitRows), or one longer row;
// rows beyond kOwnRowMax keep the statistics pass.
constexpr uint32_t kOwnRowMax = 32768;
constexpr uint32_t kOwnUnitElems = 4096;
constexpr uint32_t kOwnUnitRows = 256;
// Units of up to this many elements pass their gradient through shared memory.
constexpr uint32_t kOwnStageElems = 4096;
// Threads per CTA of that kernel.  Its CTAs meet at barriers between loading a
// unit's gradient and using the row sums, so a CTA moves at the pace of its
// slowest load; CTAs of 4 warps (8 resident per SM) lose less to that than CTAs
// of 8 (measured on the ResNet-50-shaped set: 0.129 against 0.138 ms per step;
// CTAs of 2 warps: 0.135).
constexpr int kOwnBlockThreads = 128;

// Launches it: CTAs [0, n_rest) take one chunk-table entry each of `rest` (the
// tensors without rows, and those with longer rows, whose means the statistics
// pass has left in their records); the next n_units CTAs one unit of whole rows
// each (RowUnit with part_len = 0).  cfg.pre: PRE_CENTER_ROWS with or without
// PRE_COPY16 and PRE_MOM16; cfg.grid and cfg.reverse are ignored.
cudaError_t launch_step_rows(const Chunk *d_rest, int n_rest, const RowUnit *d_units, int n_units,
                             const TensorRec *d_recs, const StepScalars &s, int nesterov,
                             int grad_dtype, int la, const LaunchCfg &cfg, cudaStream_t stream);

// Elements a row unit aims at, and rows per unit where a thread takes a row.
constexpr uint32_t kRowUnitElems = 16384;
constexpr uint32_t kRowUnitThreads = 256;
constexpr uint32_t kRowWarpMax = 8192;     // longest row a single warp streams
constexpr uint32_t kRowHalfWarpMax = 1024; // longest row that gets half a warp (two rows per warp)

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
// With finalize = false the pass stops at prep->local_sums (this process's sums
// of squares of gradients and parameters) and launch_grad_norm_scalars, given
// the all-reduced sums of the whole group, forms norm and factors.
cudaError_t launch_grad_stats(const StatsPlan &plan, int grad_dtype, double c_clip,
                              double auto_gamma, bool finalize, int pdl, cudaStream_t stream);
cudaError_t launch_grad_norm_scalars(PrepOut *prep, const double *d_totals, double c_clip,
                                     double auto_gamma, int pdl, cudaStream_t stream);

// ---- true Nesterov: the look-ahead of Eq. 10 and its undoing ----------------
// Per-tensor record of the two helper kernels: the parameters, and where the
// tensor sits inside a state region (first moment and save buffer share it).
struct __align__(16) LookRec {
    float *p;
    int64_t state_off;   // elements from the start of a region
};

// save <- theta, theta <- theta + beta_N m (Eq. 10) over the chunk table; the
// first-moment region holds fp32, or bf16 when moments_bf16 is set.
cudaError_t launch_extrapolate(const Chunk *d_chunks, int n_chunks, const LookRec *d_recs,
                               const void *m_region, int moments_bf16, float *save_region,
                               float beta_n, int grid, int pdl, cudaStream_t stream);
// theta <- save (Section 5.8: restore the parameters after the closure).
cudaError_t launch_restore(const Chunk *d_chunks, int n_chunks, const LookRec *d_recs,
                           const float *save_region, int grid, int pdl, cudaStream_t stream);

// ---- graph-capturable step: the step counter and the scalar plan in device memory
// One step's plan as the kernels and novak_get_info need it.
struct __align__(16) PlanSlot {
    StepScalars s;
    int la;                  // LA_* bits
    int nesterov;            // variant
    int rect_branch, is_sync;
    double bc1, bc2, rho_inf, rho_t, r_t, step_size, decay, beta1_t, beta2_t;
};

// t is the index of the step that runs NEXT; its plan is armed in slot[t & 1]
// and the plan of the step that ran last is still in slot[(t - 1) & 1].  The
// step kernel only reads; novak_plan_next_kernel, launched behind it, computes
// the plan of step t + 1 while the step runs and publishes it (and t + 1, and
// the synchronisation counters of step t) once the step has completed.  lr and
// weight_decay are what the next plan uses (uploaded by the host when an
// option changes them, followed by novak_plan_arm_kernel).
struct __align__(16) DevPlan {
    long long t, n_syncs, last_sync;
    double lr, weight_decay;
    PlanSlot slot[2];
};

// (Re)computes the armed plan slot[t & 1] from dp->t and the rates in *dp (after
// the host has uploaded counters or rates).  `hyper` is a novak_host::Hyper
// passed by value (opaque here).  Plain launch.
cudaError_t launch_plan_arm(DevPlan *d_plan, const void *hyper, size_t hyper_bytes,
                            cudaStream_t stream);
// Behind the step kernel: the plan of step t + 1, published when the step is done.
cudaError_t launch_plan_next(DevPlan *d_plan, const void *hyper, size_t hyper_bytes, int pdl,
                             cudaStream_t stream);
// The step kernel that takes its scalars and lookahead action from the armed slot.
// cfg.pre: PRE_NONE, PRE_SCALE or PRE_CENTER, with or without PRE_COPY16 and
// PRE_MOM16; cudaErrorInvalidValue otherwise.
cudaError_t launch_step_dyn(const Chunk *d_chunks, int n_chunks, const TensorRec *d_recs,
                            const PrepOut *prep, const float *trust, const DevPlan *d_plan,
                            int nesterov, int grad_dtype, const LaunchCfg &cfg,
                            cudaStream_t stream);

// ---- work table for callers that cannot allocate device memory --------------
// Capacity of the statically allocated table behind novak_step_noalloc.
constexpr int kNoAllocMaxTensors = 4096;
constexpr int kNoAllocMaxChunks = 131072;

// Device addresses of the static table on the CURRENT device (resolved once per
// device with cudaGetSymbolAddress).  No allocation.
cudaError_t noalloc_table(TensorRec **d_recs, Chunk **d_chunks);

}  // namespace novak
