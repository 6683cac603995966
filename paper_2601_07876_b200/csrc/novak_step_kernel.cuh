// Fused multi-tensor NOVAK step kernel for sm_100a (template; instantiated by
// novak_step_pre*.cu, one translation unit per gradient pre-processing mode).
//
// One launch covers every tensor of a parameter group.  A CTA takes entries of
// the chunk table; for each it reads theta, g, m, v (and the lookahead arrays
// on the steps that need them) exactly once with 128-bit coalesced accesses,
// does the paper's phases 2 and 4-10 in registers (fp32, IEEE sqrt and
// division, no fast-math) and writes theta, m, v (and the lookahead arrays)
// exactly once.  There is no shared memory, no atomic, no barrier and no spin
// of any kind, so a launch does a bounded amount of work per CTA and cannot
// hang.
//
// The step is HBM bound: 28 B per element against ~45 fp32 instructions, so
// the design goal is bytes in flight per SM, not arithmetic: each thread
// issues NOVAK_UNROLL independent 16-byte loads per stream before the first
// use.
#pragma once

#include "novak_internal.h"

#include "novak.h"

#include <cuda_bf16.h>

#ifndef NOVAK_BLOCK
#define NOVAK_BLOCK 256
#endif
#ifndef NOVAK_UNROLL
#define NOVAK_UNROLL 2
#endif
#ifndef NOVAK_MIN_CTAS
#define NOVAK_MIN_CTAS 4
#endif

namespace novak {
namespace {

constexpr int kBlock = NOVAK_BLOCK;
constexpr int kUnroll = NOVAK_UNROLL;

template <int N>
struct Vec {
    float a[N];
};

// ---- global memory access: streaming hints, each address touched once per step
template <int N>
__device__ __forceinline__ Vec<N> load_f32(const float *base, int idx);

template <>
__device__ __forceinline__ Vec<4> load_f32<4>(const float *base, int idx)
{
    const float4 t = __ldcs(reinterpret_cast<const float4 *>(base) + idx);
    Vec<4> r;
    r.a[0] = t.x; r.a[1] = t.y; r.a[2] = t.z; r.a[3] = t.w;
    return r;
}

template <>
__device__ __forceinline__ Vec<1> load_f32<1>(const float *base, int idx)
{
    Vec<1> r;
    r.a[0] = __ldcs(base + idx);
    return r;
}

template <int N>
__device__ __forceinline__ void store_f32(float *base, int idx, const Vec<N> &x);

template <>
__device__ __forceinline__ void store_f32<4>(float *base, int idx, const Vec<4> &x)
{
    __stcs(reinterpret_cast<float4 *>(base) + idx,
           make_float4(x.a[0], x.a[1], x.a[2], x.a[3]));
}

template <>
__device__ __forceinline__ void store_f32<1>(float *base, int idx, const Vec<1> &x)
{
    __stcs(base + idx, x.a[0]);
}

// fp32 -> bf16, round to nearest even: the model copy of the updated parameters.
template <int N>
__device__ __forceinline__ void store_bf16(__nv_bfloat16 *base, int idx, const Vec<N> &x)
{
    if constexpr (N == 4) {
        const __nv_bfloat162 lo = __floats2bfloat162_rn(x.a[0], x.a[1]);
        const __nv_bfloat162 hi = __floats2bfloat162_rn(x.a[2], x.a[3]);
        uint2 t;
        t.x = *reinterpret_cast<const unsigned *>(&lo);
        t.y = *reinterpret_cast<const unsigned *>(&hi);
        __stcs(reinterpret_cast<uint2 *>(base) + idx, t);
    } else {
        base[idx] = __float2bfloat16_rn(x.a[0]);
    }
}

// bf16 -> fp32 is exact: the 16 bits are the upper half of the fp32 pattern.
template <int N, int GT>
__device__ __forceinline__ Vec<N> load_grad(const void *base, int idx)
{
    if constexpr (GT == NOVAK_GRAD_F32) {
        return load_f32<N>(static_cast<const float *>(base), idx);
    } else if constexpr (N == 4) {
        const uint2 t = __ldcs(static_cast<const uint2 *>(base) + idx);
        Vec<4> r;
        r.a[0] = __uint_as_float(t.x << 16);
        r.a[1] = __uint_as_float(t.x & 0xffff0000u);
        r.a[2] = __uint_as_float(t.y << 16);
        r.a[3] = __uint_as_float(t.y & 0xffff0000u);
        return r;
    } else {
        const unsigned short t = __ldcs(static_cast<const unsigned short *>(base) + idx);
        Vec<1> r;
        r.a[0] = __uint_as_float(static_cast<unsigned>(t) << 16);
        return r;
    }
}

// Moments as stored: fp32, or bf16 (M16) widened exactly on load and rounded to
// nearest even on store.
template <int N, bool M16>
__device__ __forceinline__ Vec<N> load_moment(const void *base, int idx)
{
    if constexpr (M16) return load_grad<N, NOVAK_GRAD_BF16>(base, idx);
    else return load_f32<N>(static_cast<const float *>(base), idx);
}

template <int N, bool M16>
__device__ __forceinline__ void store_moment(void *base, int idx, const Vec<N> &x)
{
    if constexpr (M16) store_bf16<N>(static_cast<__nv_bfloat16 *>(base), idx, x);
    else store_f32<N>(static_cast<float *>(base), idx, x);
}

// ---- phase 2 before the Nesterov approximation: clip factor and centralization
struct PreArgs {
    __nv_bfloat16 *copy; // bf16 copy of the chunk's parameters (PRE_COPY16), else unused
    float step;          // alpha r_t, times the tensor's trust ratio under layer adaptation
    float factor;        // clip factor (1 when clipping is off or inactive)
    const float2 *mean;  // row means of the raw gradient (hi + lo), NULL: tensor not centralized
    uint32_t row_len;
    uint32_t elem0;      // index within the tensor of the span's first element
};

// g <- factor (g - mean of its row), Eq. 26 with the clip factor applied after
// the (linear) centring.  `e` is the tensor index of G's first element.  A
// vector usually lies inside one row; the row mean is re-read only where it
// crosses into the next one.  The mean comes as hi + lo: where g and the mean
// nearly cancel, g - hi is exact and lo supplies the mean's remaining bits, so
// the centred gradient carries a relative rounding error only.
// Where a vector starts inside its tensor's rows, with that row's mean.
struct RowPos {
    uint32_t row, rem;
    float2 mu;
};

template <int PRE>
__device__ __forceinline__ RowPos row_position(uint32_t e, const PreArgs &a)
{
    RowPos r;
    r.row = 0u; r.rem = 0u; r.mu = make_float2(0.0f, 0.0f);
    if constexpr ((PRE & PRE_MASK) == PRE_CENTER) {
        if (a.mean != nullptr) {
            r.row = e / a.row_len;
            r.rem = e - r.row * a.row_len;
            r.mu = a.mean[r.row];
        }
    }
    return r;
}

template <int N, int PRE>
__device__ __forceinline__ void preprocess(Vec<N> &G, const RowPos &pos, const PreArgs &a)
{
    if constexpr ((PRE & PRE_MASK) == PRE_CENTER) {
        if (a.mean != nullptr) {
            uint32_t row = pos.row;
            uint32_t rem = pos.rem;
            float2 mu = pos.mu;
#pragma unroll
            for (int j = 0; j < N; ++j) {
                if (rem == a.row_len) {     // stepped over the end of the row
                    rem = 0;
                    ++row;
                    mu = a.mean[row];
                }
                G.a[j] = (G.a[j] - mu.x) - mu.y;
                ++rem;
            }
        }
    }
    if constexpr ((PRE & PRE_MASK) != PRE_NONE) {
#pragma unroll
        for (int j = 0; j < N; ++j) G.a[j] *= a.factor;
    }
}

// ---- phases 2 (Nesterov approximation), 4, 5 and 8 up to the base direction:
// advances m and v with the processed gradient g and returns u of Eq. 17.
template <int NEST>
__device__ __forceinline__ float base_direction(float g, float &m, float &v, float &m_hat,
                                                const StepScalars &s)
{
    // Phase 2, Eq. 13: g~ = g + beta_N (g - m_{t-1})
    if constexpr (NEST == NOVAK_NESTEROV_APPROX)
        g = fmaf(s.beta_n, g - m, g);
    // Phase 4, Eq. 1-2
    m = fmaf(s.beta1, m, s.omb1 * g);
    v = fmaf(s.beta2, v, s.omb2 * (g * g));
    // Phase 5, Eq. 5
    m_hat = m * s.inv_bc1;
    const float v_hat = v * s.inv_bc2;
    // Phase 8, Eq. 17 (IEEE sqrt and division)
#ifdef NOVAK_APPROX_MATH
    float rt, u;
    asm("sqrt.approx.f32 %0, %1;" : "=f"(rt) : "f"(v_hat));
    asm("div.full.f32 %0, %1, %2;" : "=f"(u) : "f"(m_hat), "f"(rt + s.eps));
    return u;
#else
    return m_hat / (sqrtf(v_hat) + s.eps);
#endif
}

// ---- the per-element update, phases 2 and 4-10 (Section 5.1)
template <int NEST, int LA>
__device__ __forceinline__ void update_element(float &p, float g, float &m, float &v,
                                               float &slow, float &acc,
                                               const StepScalars &s, float step)
{
    float m_hat;
    float u = base_direction<NEST>(g, m, v, m_hat, s);
    // Eq. 27: u 1{|u| > tau}.  With the mask off tau is -1 and nothing, NaN
    // included, compares below it.
    u = (fabsf(u) <= s.sparse_tau) ? 0.0f : u;
    // Eq. 16 for the classical blend
    if constexpr (NEST == NOVAK_NESTEROV_CLASSICAL)
        u = fmaf(s.blend_b1, m_hat, s.blend_omb1 * u);
    // Phase 9, Eq. 18 + 24: decay with the base rate, step with alpha r_t
    const float theta_in = p;
    const float theta_fast = fmaf(theta_in, s.decay, -(step * u));
    // Phase 10, Eq. 28-31
    float out = theta_fast;
    float sum = theta_fast;
    if constexpr ((LA & LA_A_READ) != 0)
        sum = acc + theta_fast;
    if constexpr ((LA & LA_A_WRITE) != 0)
        acc = sum;
    if constexpr ((LA & LA_SYNC) != 0) {
        const float slow_in = (LA & LA_S_INIT) ? theta_in : slow;
        const float target = (LA & LA_TRAJ) ? __fdiv_rn(sum, s.k) : theta_fast;
        out = fmaf(s.la_alpha, target - slow_in, slow_in);
        slow = out;
    } else if constexpr ((LA & LA_S_INIT) != 0) {
        slow = theta_in;
    }
    p = out;
}

// One full tile: U vectors per thread and per stream, every load issued
// before the first use so that U x (4..6) 16-byte requests are in flight.
template <int N, int U, int NEST, int GT, int LA, int PRE>
__device__ __forceinline__ void run_tile(float *p, const void *g, void *m, void *v,
                                         float *slow, float *acc, int first,
                                         const StepScalars &s, const PreArgs &pre)
{
    constexpr bool kMom16 = (PRE & PRE_MOM16) != 0;
    constexpr bool kReadS = (LA & LA_S_READ) != 0;
    constexpr bool kWriteS = (LA & LA_S_WRITE) != 0;
    constexpr bool kReadA = (LA & LA_A_READ) != 0;
    constexpr bool kWriteA = (LA & LA_A_WRITE) != 0;
    // On steps without a synchronisation (fewer live registers) the row means
    // are fetched together with the streams, so that their latency overlaps.
    constexpr bool kEarlyMean = (LA & LA_SYNC) == 0 && (PRE & PRE_MASK) == PRE_CENTER;
    Vec<N> P[U], G[U], M[U], V[U], S[U], A[U];
    RowPos R[U];
#pragma unroll
    for (int j = 0; j < U; ++j) {
        const int idx = first + j * kBlock;
        if constexpr (kEarlyMean)
            R[j] = row_position<PRE>(pre.elem0 + static_cast<uint32_t>(idx) * N, pre);
        P[j] = load_f32<N>(p, idx);
        G[j] = load_grad<N, GT>(g, idx);
        M[j] = load_moment<N, kMom16>(m, idx);
        V[j] = load_moment<N, kMom16>(v, idx);
        if constexpr (kReadS) S[j] = load_f32<N>(slow, idx);
        if constexpr (kReadA) A[j] = load_f32<N>(acc, idx);
    }
#pragma unroll
    for (int j = 0; j < U; ++j) {
        const int idx = first + j * kBlock;
        if constexpr (!kEarlyMean)
            R[j] = row_position<PRE>(pre.elem0 + static_cast<uint32_t>(idx) * N, pre);
        preprocess<N, PRE>(G[j], R[j], pre);
#pragma unroll
        for (int e = 0; e < N; ++e)
            update_element<NEST, LA>(P[j].a[e], G[j].a[e], M[j].a[e], V[j].a[e],
                                     S[j].a[e], A[j].a[e], s, pre.step);
        store_f32<N>(p, idx, P[j]);
        if constexpr ((PRE & PRE_COPY16) != 0) store_bf16<N>(pre.copy, idx, P[j]);
        store_moment<N, kMom16>(m, idx, M[j]);
        store_moment<N, kMom16>(v, idx, V[j]);
        if constexpr (kWriteS) store_f32<N>(slow, idx, S[j]);
        if constexpr (kWriteA) store_f32<N>(acc, idx, A[j]);
    }
}

// nvec vectors of N elements: full tiles of U vectors per thread, then the
// remainder one vector per thread at a time.
template <int N, int U, int NEST, int GT, int LA, int PRE>
__device__ __forceinline__ void run_span(float *p, const void *g, void *m, void *v,
                                         float *slow, float *acc, int nvec,
                                         const StepScalars &s, const PreArgs &pre)
{
    constexpr int kTile = kBlock * U;
    int base = 0;
#pragma unroll 1
    for (; base + kTile <= nvec; base += kTile)
        run_tile<N, U, NEST, GT, LA, PRE>(p, g, m, v, slow, acc, base + threadIdx.x, s, pre);
#pragma unroll 1
    for (int idx = base + threadIdx.x; idx < nvec; idx += kBlock)
        run_tile<N, 1, NEST, GT, LA, PRE>(p, g, m, v, slow, acc, idx, s, pre);
}

// Programmatic dependent launch (PTX griddepcontrol).  launch_dependents lets
// the next kernel on the stream become resident once every CTA of this grid
// has started; wait blocks until the previous grid on the stream has completed
// and its writes are visible.  Both are no-ops in a plain launch.
__device__ __forceinline__ void grid_dependency_release()
{
    asm volatile("griddepcontrol.launch_dependents;");
}
__device__ __forceinline__ void grid_dependency_wait()
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

template <int NEST, int GT, int LA, int PRE>
__global__ void __launch_bounds__(NOVAK_BLOCK, NOVAK_MIN_CTAS)
novak_step_kernel(const Chunk *__restrict__ chunks, int n_chunks,
                  const TensorRec *__restrict__ recs, const PrepOut *prep,
                  const float *trust, const StepScalars s, int reverse)
{
    constexpr int kGradBytes = (GT == NOVAK_GRAD_BF16) ? 2 : 4;
    constexpr int kMomBytes = (PRE & PRE_MOM16) ? 2 : 4;
    constexpr bool kUseS = (LA & (LA_S_READ | LA_S_WRITE)) != 0;
    constexpr bool kUseA = (LA & (LA_A_READ | LA_A_WRITE)) != 0;

    grid_dependency_release();
    int c = blockIdx.x;
    if (c >= n_chunks) return;
    // The work table is written by copies only, never by a kernel, so it may be
    // read before the previous kernel on the stream has finished.  prep, trust
    // and the row means ARE the previous kernels' output and this grid may be
    // resident while they are written: they are not declared read-only
    // (no __restrict__, no non-coherent loads) and are read after the wait.
    Chunk ch = chunks[reverse ? n_chunks - 1 - c : c];
    TensorRec r = recs[ch.tensor];
    grid_dependency_wait();

    // The clip factor is the statistics kernel's output: read it only now.
    PreArgs pre;
    pre.factor = 1.0f;
    float step = s.step;
    if constexpr ((PRE & PRE_MASK) != PRE_NONE) {
        pre.factor = prep->factor;
        step *= prep->auto_scale;        // Eq. 22 (1 when the scaling is off), Eq. 24a
    }

#pragma unroll 1
    for (;;) {
        // Eq. 24a: the tensor's trust ratio stretches the step (layer adaptation)
        pre.step = trust != nullptr ? step * trust[ch.tensor] : step;
        pre.mean = ((PRE & PRE_MASK) == PRE_CENTER) ? r.mean : nullptr;
        pre.row_len = r.row_len;
        pre.elem0 = static_cast<uint32_t>(ch.offset);
        pre.copy = ((PRE & PRE_COPY16) != 0) ? r.p16 + ch.offset : nullptr;
        float *p = r.p + ch.offset;
        void *m = static_cast<char *>(r.m) + ch.offset * kMomBytes;
        void *v = static_cast<char *>(r.v) + ch.offset * kMomBytes;
        float *slow = kUseS ? r.slow + ch.offset : nullptr;
        float *acc = kUseA ? r.acc + ch.offset : nullptr;
        const void *g = static_cast<const char *>(r.g) + ch.offset * kGradBytes;

        // four bf16 moments are one 64-bit access: half the parameters' alignment
        uintptr_t bits = reinterpret_cast<uintptr_t>(p) |
                         ((reinterpret_cast<uintptr_t>(m) | reinterpret_cast<uintptr_t>(v))
                          << (kMomBytes == 2 ? 1 : 0));
        if (kUseS) bits |= reinterpret_cast<uintptr_t>(slow);
        if (kUseA) bits |= reinterpret_cast<uintptr_t>(acc);
        // the 64-bit stores of the bf16 copy need half the parameters' alignment
        if ((PRE & PRE_COPY16) != 0) bits |= reinterpret_cast<uintptr_t>(pre.copy) << 1;
        const bool aligned = (bits & 15u) == 0 &&
                             (reinterpret_cast<uintptr_t>(g) & (4u * kGradBytes - 1u)) == 0;
        if (aligned) {
            const int nvec = ch.len >> 2;
            run_span<4, kUnroll, NEST, GT, LA, PRE>(p, g, m, v, slow, acc, nvec, s, pre);
            // ragged tail of a tensor: at most 3 elements
            const int idx = (nvec << 2) + threadIdx.x;
            if (idx < ch.len)
                run_tile<1, 1, NEST, GT, LA, PRE>(p, g, m, v, slow, acc, idx, s, pre);
        } else {
            // parameter, gradient and state do not share 16-byte alignment
            run_span<1, 4, NEST, GT, LA, PRE>(p, g, m, v, slow, acc, ch.len, s, pre);
        }
        c += gridDim.x;
        if (c >= n_chunks) break;
        ch = chunks[reverse ? n_chunks - 1 - c : c];
        r = recs[ch.tensor];
    }
}

using StepKernelFn = void (*)(const Chunk *, int, const TensorRec *, const PrepOut *,
                              const float *, StepScalars, int);

template <int NEST, int GT, int PRE>
StepKernelFn pick_la(int la)
{
    switch (la) {
#define NOVAK_LA_CASE(X) case (X): return novak_step_kernel<NEST, GT, (X), PRE>;
        NOVAK_LA_CASE(LA_NONE)
        NOVAK_LA_CASE(LA_S_INIT | LA_S_WRITE)
        NOVAK_LA_CASE(LA_S_INIT | LA_S_WRITE | LA_SYNC)
        NOVAK_LA_CASE(LA_S_READ | LA_S_WRITE | LA_SYNC)
        NOVAK_LA_CASE(LA_A_WRITE)
        NOVAK_LA_CASE(LA_A_WRITE | LA_S_INIT | LA_S_WRITE)
        NOVAK_LA_CASE(LA_A_READ | LA_A_WRITE)
        NOVAK_LA_CASE(LA_A_READ | LA_S_READ | LA_S_WRITE | LA_SYNC | LA_TRAJ)
#undef NOVAK_LA_CASE
    default: return nullptr;
    }
}

template <int NEST, int PRE>
StepKernelFn pick_gt(int grad_dtype, int la)
{
    switch (grad_dtype) {
    case NOVAK_GRAD_F32: return pick_la<NEST, NOVAK_GRAD_F32, PRE>(la);
    case NOVAK_GRAD_BF16: return pick_la<NEST, NOVAK_GRAD_BF16, PRE>(la);
    default: return nullptr;
    }
}

// Every instantiation for one pre-processing mode (3 variants x 2 gradient
// types x 8 lookahead actions).
template <int PRE>
StepKernelFn pick_step_kernel(int nesterov, int grad_dtype, int la)
{
    switch (nesterov) {
    case NOVAK_NESTEROV_NONE: return pick_gt<NOVAK_NESTEROV_NONE, PRE>(grad_dtype, la);
    case NOVAK_NESTEROV_APPROX: return pick_gt<NOVAK_NESTEROV_APPROX, PRE>(grad_dtype, la);
    case NOVAK_NESTEROV_CLASSICAL: return pick_gt<NOVAK_NESTEROV_CLASSICAL, PRE>(grad_dtype, la);
    default: return nullptr;
    }
}

}  // namespace
}  // namespace novak
