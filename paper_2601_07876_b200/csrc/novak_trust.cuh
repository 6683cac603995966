// Layer-wise adaptation (Eq. 19 / 25), device side shared by the two-kernel
// pass (novak_trust_stats.cu: the sums of squares of theta_t and of this step's
// base direction u_t over one chunk-table entry) and by the kernel that adapts
// and steps in one launch (novak_step_adapt.cuh: the same block and warp sums,
// the ratio of a tensor).
//
// u_t is the direction THIS step produces, so the moments are advanced exactly
// as the step kernel will advance them (same device functions, same fp32
// operations) but stay in registers.  All sums are carried in double and
// combined in a fixed order: bit-identical from run to run.
#pragma once

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

// The two sums over one chunk-table entry; thread 0 returns them in tp, tu.
template <int NEST, int GT, int PRE>
__device__ __forceinline__ void entry_trust_sums(const Chunk &ch, const TensorRec &r,
                                                 const StepScalars &s, const PreArgs &pre,
                                                 double *sh, double &tp, double &tu)
{
    constexpr int kGradBytes = (GT == NOVAK_GRAD_BF16) ? 2 : 4;
    constexpr int kMomBytes = (PRE & PRE_MOM16) ? 2 : 4;
    const float *p = r.p_in + ch.offset;     // theta_{t-1}
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
    tp = trust_block_sum(sum_p, sh);
    tu = trust_block_sum(sum_u, sh);
}

// Eq. 19 / 25 for one tensor from its entries' sums [c0, c1), added in table
// order by the whole CTA; thread 0 returns clip(||theta|| / ||u||, 0.1, 10), 1
// where ||u|| = 0 (the ratio is undefined there, the update zero).  The sums
// may have been written by other CTAs of the same grid: L2 loads.
__device__ __forceinline__ float tensor_trust_ratio(const double *chunk_p2, const double *chunk_u2,
                                                    int c0, int c1, double *sh)
{
    double sp = 0.0, su = 0.0;
    for (int c = c0 + threadIdx.x; c < c1; c += kTrustBlock) {
        sp += __ldcg(chunk_p2 + c);
        su += __ldcg(chunk_u2 + c);
    }
    const double tp = trust_block_sum(sp, sh);
    const double tu = trust_block_sum(su, sh);
    double eta = 1.0;
    if (threadIdx.x == 0 && tu > 0.0) {
        eta = sqrt(tp) / sqrt(tu);
        eta = eta < 0.1 ? 0.1 : (eta > 10.0 ? 10.0 : eta);
    }
    return static_cast<float>(eta);
}

}  // namespace
}  // namespace novak
