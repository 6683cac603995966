// Layer-wise adaptation (Eq. 19 / 25) for sm_100a: the trust ratio
// ||theta_t||_2 / ||u_t||_2 of every tensor, clipped to [0.1, 10], left in
// device memory for the step kernel that follows on the stream.
//
// u_t is the direction THIS step produces, so the first kernel advances the
// moments exactly as the step kernel will (same device functions, same fp32
// operations) but keeps them in registers: it reads theta, g, m, v once
// (16 B per element) and writes two doubles per chunk-table entry.  The second
// kernel, one CTA per tensor, adds a tensor's entries in table order.  All
// sums are in double in a fixed order: bit-identical from run to run, no
// atomics, nothing spins.
#include "novak_trust.cuh"

namespace novak {
namespace {

template <int NEST, int GT, int PRE>
__global__ void __launch_bounds__(NOVAK_BLOCK)
novak_trust_stats_kernel(const Chunk *__restrict__ chunks, int n_chunks,
                         const TensorRec *__restrict__ recs, const PrepOut *prep,
                         const StepScalars s_host, const DevPlan *plan,
                         double *__restrict__ chunk_u2, double *__restrict__ chunk_p2)
{
    __shared__ double sh[kTrustWarps];

    grid_dependency_release();
    const int c = blockIdx.x;            // the grid has exactly n_chunks CTAs
    if (c >= n_chunks) return;
    const Chunk ch = chunks[c];
    const TensorRec r = recs[ch.tensor];
    grid_dependency_wait();              // parameters, moments, clip factor, row means
    // the graph-capturable step keeps this step's scalars in device memory
    const StepScalars s = plan != nullptr ? plan->slot[plan->t & 1].s : s_host;

    PreArgs pre;
    pre.copy = nullptr;
    pre.step = 0.0f;
    pre.factor = 1.0f;
    if constexpr ((PRE & PRE_MASK) != PRE_NONE) pre.factor = prep->factor;
    pre.mean = ((PRE & PRE_MASK) == PRE_CENTER) ? r.mean : nullptr;
    pre.row_len = r.row_len;
    pre.elem0 = static_cast<uint32_t>(ch.offset);

    double tp, tu;
    entry_trust_sums<NEST, GT, PRE>(ch, r, s, pre, sh, tp, tu);
    if (threadIdx.x == 0) {
        chunk_p2[c] = tp;
        chunk_u2[c] = tu;
    }
}

// One CTA per tensor: its entries' sums in table order, then Eq. 19's ratio.
__global__ void __launch_bounds__(NOVAK_BLOCK)
novak_trust_finish_kernel(const int *__restrict__ tensor_first,
                          const double *chunk_u2,
                          const double *chunk_p2, float *__restrict__ trust)
{
    __shared__ double sh[kTrustWarps];
    grid_dependency_release();
    const int t = blockIdx.x;
    const int c0 = tensor_first[t], c1 = tensor_first[t + 1];
    grid_dependency_wait();              // the first kernel's sums
    const float eta = tensor_trust_ratio(chunk_p2, chunk_u2, c0, c1, sh);
    if (threadIdx.x == 0) trust[t] = eta;
}

using TrustFn = void (*)(const Chunk *, int, const TensorRec *, const PrepOut *, StepScalars,
                         const DevPlan *, double *, double *);

template <int NEST, int GT>
TrustFn pick_pre(int pre)
{
    switch (pre) {
    case PRE_NONE: return novak_trust_stats_kernel<NEST, GT, PRE_NONE>;
    case PRE_SCALE: return novak_trust_stats_kernel<NEST, GT, PRE_SCALE>;
    case PRE_CENTER: return novak_trust_stats_kernel<NEST, GT, PRE_CENTER>;
    case PRE_NONE | PRE_MOM16: return novak_trust_stats_kernel<NEST, GT, PRE_NONE | PRE_MOM16>;
    case PRE_SCALE | PRE_MOM16: return novak_trust_stats_kernel<NEST, GT, PRE_SCALE | PRE_MOM16>;
    case PRE_CENTER | PRE_MOM16: return novak_trust_stats_kernel<NEST, GT, PRE_CENTER | PRE_MOM16>;
    default: return nullptr;
    }
}

template <int NEST>
TrustFn pick_dtype(int grad_dtype, int pre)
{
    switch (grad_dtype) {
    case NOVAK_GRAD_F32: return pick_pre<NEST, NOVAK_GRAD_F32>(pre);
    case NOVAK_GRAD_BF16: return pick_pre<NEST, NOVAK_GRAD_BF16>(pre);
    default: return nullptr;
    }
}

TrustFn pick_trust(int nesterov, int grad_dtype, int pre)
{
    switch (nesterov) {
    // the classical blend (Eq. 16) comes after the base direction: same kernel as "none"
    case NOVAK_NESTEROV_NONE:
    case NOVAK_NESTEROV_CLASSICAL: return pick_dtype<NOVAK_NESTEROV_NONE>(grad_dtype, pre);
    case NOVAK_NESTEROV_APPROX: return pick_dtype<NOVAK_NESTEROV_APPROX>(grad_dtype, pre);
    default: return nullptr;
    }
}

void fill_config(cudaLaunchConfig_t *lc, cudaLaunchAttribute *attr, unsigned grid, bool pdl,
                 cudaStream_t stream)
{
    *lc = cudaLaunchConfig_t{};
    lc->gridDim = dim3(grid);
    lc->blockDim = dim3(kTrustBlock);
    lc->dynamicSmemBytes = 0;
    lc->stream = stream;
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc->attrs = attr;
    lc->numAttrs = pdl ? 1 : 0;
}

}  // namespace

cudaError_t launch_trust_stats(const Chunk *d_chunks, int n_chunks, const TensorRec *d_recs,
                               int n_tensors, const int *tensor_first, const PrepOut *prep,
                               const StepScalars &s, const DevPlan *d_plan, int nesterov,
                               int grad_dtype, int pre, double *chunk_u2, double *chunk_p2,
                               float *trust, int pdl, cudaStream_t stream)
{
    TrustFn fn = pick_trust(nesterov, grad_dtype, pre);
    if (!fn || n_chunks <= 0 || n_tensors <= 0 || !tensor_first || !chunk_u2 || !chunk_p2 || !trust)
        return cudaErrorInvalidValue;
    if ((pre & PRE_MASK) != PRE_NONE && prep == nullptr) return cudaErrorInvalidValue;
    cudaLaunchConfig_t lc;
    cudaLaunchAttribute attr[1];
    fill_config(&lc, attr, static_cast<unsigned>(n_chunks), (pdl & 2) != 0, stream);
    cudaError_t e = cudaLaunchKernelEx(&lc, fn, d_chunks, n_chunks, d_recs, prep, s, d_plan, chunk_u2, chunk_p2);
    if (e != cudaSuccess) return e;
    fill_config(&lc, attr, static_cast<unsigned>(n_tensors), (pdl & 4) != 0, stream);
    const double *u2 = chunk_u2, *p2 = chunk_p2;
    return cudaLaunchKernelEx(&lc, novak_trust_finish_kernel, tensor_first, u2, p2, trust);
}

}  // namespace novak
