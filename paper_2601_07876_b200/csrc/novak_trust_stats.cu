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
#include "novak_step_kernel.cuh"

namespace novak {
namespace {

constexpr int kTrustBlock = NOVAK_BLOCK;
constexpr int kTrustWarps = kTrustBlock / 32;

__device__ __forceinline__ double trust_warp_sum(double x)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_down_sync(0xffffffffu, x, o);
    return x;
}

// Sum over the CTA, warps in index order; thread 0 holds the total.
__device__ __forceinline__ double trust_block_sum(double x, double *sh)
{
    x = trust_warp_sum(x);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    __syncthreads();
    if (lane == 0) sh[warp] = x;
    __syncthreads();
    double t = 0.0;
    if (threadIdx.x == 0) {
#pragma unroll
        for (int w = 0; w < kTrustWarps; ++w) t += sh[w];
    }
    return t;
}

// Squares of N parameters and of the N base directions their gradients give.
// Each group of N squares is added in fp32, groups in double.
template <int N, int NEST, int GT, int PRE>
__device__ __forceinline__ void accumulate(const float *p, const void *g, const void *m,
                                           const void *v, int idx, const StepScalars &s,
                                           const PreArgs &pre, double &sum_p, double &sum_u)
{
    const Vec<N> P = load_f32<N>(p, idx);
    Vec<N> G = load_grad<N, GT>(g, idx);
    const Vec<N> M = load_moment<N, (PRE & PRE_MOM16) != 0>(m, idx);
    const Vec<N> V = load_moment<N, (PRE & PRE_MOM16) != 0>(v, idx);
    preprocess<N, PRE>(G, row_position<PRE>(pre.elem0 + static_cast<uint32_t>(idx) * N, pre), pre);
    float sp = 0.0f, su = 0.0f;
#pragma unroll
    for (int e = 0; e < N; ++e) {
        float mm = M.a[e], vv = V.a[e], m_hat;
        const float u = base_direction<NEST>(G.a[e], mm, vv, m_hat, s);
        sp = fmaf(P.a[e], P.a[e], sp);
        su = fmaf(u, u, su);
    }
    sum_p += double(sp);
    sum_u += double(su);
}

template <int NEST, int GT, int PRE>
__global__ void __launch_bounds__(NOVAK_BLOCK)
novak_trust_stats_kernel(const Chunk *__restrict__ chunks, int n_chunks,
                         const TensorRec *__restrict__ recs, const PrepOut *prep,
                         const StepScalars s_host, const DevPlan *plan,
                         double *__restrict__ chunk_u2, double *__restrict__ chunk_p2)
{
    __shared__ double sh[kTrustWarps];
    constexpr int kGradBytes = (GT == NOVAK_GRAD_BF16) ? 2 : 4;
    constexpr int kMomBytes = (PRE & PRE_MOM16) ? 2 : 4;

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

    const float *p = r.p + ch.offset;
    const void *m = static_cast<const char *>(r.m) + ch.offset * kMomBytes;
    const void *v = static_cast<const char *>(r.v) + ch.offset * kMomBytes;
    const void *g = static_cast<const char *>(r.g) + ch.offset * kGradBytes;
    const uintptr_t bits = reinterpret_cast<uintptr_t>(p) |
                           ((reinterpret_cast<uintptr_t>(m) | reinterpret_cast<uintptr_t>(v))
                            << (kMomBytes == 2 ? 1 : 0));
    const bool aligned = (bits & 15u) == 0 &&
                         (reinterpret_cast<uintptr_t>(g) & (4u * kGradBytes - 1u)) == 0;
    double sum_p = 0.0, sum_u = 0.0;
    if (aligned) {
        const int nvec = ch.len >> 2;
#pragma unroll 2
        for (int i = threadIdx.x; i < nvec; i += kTrustBlock)
            accumulate<4, NEST, GT, PRE>(p, g, m, v, i, s, pre, sum_p, sum_u);
        const int idx = (nvec << 2) + threadIdx.x;          // ragged tail: < 4 elements
        if (idx < ch.len) accumulate<1, NEST, GT, PRE>(p, g, m, v, idx, s, pre, sum_p, sum_u);
    } else {
#pragma unroll 4
        for (int i = threadIdx.x; i < ch.len; i += kTrustBlock)
            accumulate<1, NEST, GT, PRE>(p, g, m, v, i, s, pre, sum_p, sum_u);
    }
    const double tp = trust_block_sum(sum_p, sh);
    const double tu = trust_block_sum(sum_u, sh);
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
    double sp = 0.0, su = 0.0;
    for (int c = c0 + threadIdx.x; c < c1; c += kTrustBlock) {
        sp += chunk_p2[c];
        su += chunk_u2[c];
    }
    const double tp = trust_block_sum(sp, sh);
    const double tu = trust_block_sum(su, sh);
    if (threadIdx.x == 0) {
        double eta = 1.0;                // ||u|| = 0: the ratio is undefined, the update zero
        if (tu > 0.0) {
            eta = sqrt(tp) / sqrt(tu);
            eta = eta < 0.1 ? 0.1 : (eta > 10.0 ? 10.0 : eta);
        }
        trust[t] = static_cast<float>(eta);
    }
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
