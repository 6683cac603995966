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
// Resident CTAs per SM of the instantiations that read a lookahead array or set
// one up at t = 1 (up to six input and five output streams): one fewer, i.e. up
// to 85 registers instead of 64, so that two vectors per stream stay in
// registers without spilling.
#ifndef NOVAK_MIN_CTAS_WIDE
#define NOVAK_MIN_CTAS_WIDE 3
#endif

namespace novak {
namespace {

constexpr int kBlock = NOVAK_BLOCK;
constexpr int kUnroll = NOVAK_UNROLL;

template <int N>
struct Vec {
    float a[N];
};

// ---- global memory access.  LD_STREAM (the step's own accesses): streaming
// hints, each address is touched once per step.  LD_KEEP: cached in L2 only,
// normal eviction priority, for a pass whose bytes another pass reads again soon.
enum : int { LD_STREAM = 0, LD_KEEP = 1 };

template <int POL, typename T>
__device__ __forceinline__ T ld_global(const T *p)
{
    if constexpr (POL == LD_KEEP) return __ldcg(p);
    else return __ldcs(p);
}

template <int N, int POL = LD_STREAM>
__device__ __forceinline__ Vec<N> load_f32(const float *base, int idx)
{
    Vec<N> r;
    if constexpr (N == 4) {
        const float4 t = ld_global<POL>(reinterpret_cast<const float4 *>(base) + idx);
        r.a[0] = t.x; r.a[1] = t.y; r.a[2] = t.z; r.a[3] = t.w;
    } else {
        r.a[0] = ld_global<POL>(base + idx);
    }
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
template <int N, int GT, int POL = LD_STREAM>
__device__ __forceinline__ Vec<N> load_grad(const void *base, int idx)
{
    if constexpr (GT == NOVAK_GRAD_F32) {
        return load_f32<N, POL>(static_cast<const float *>(base), idx);
    } else if constexpr (N == 4) {
        const uint2 t = ld_global<POL>(static_cast<const uint2 *>(base) + idx);
        Vec<4> r;
        r.a[0] = __uint_as_float(t.x << 16);
        r.a[1] = __uint_as_float(t.x & 0xffff0000u);
        r.a[2] = __uint_as_float(t.y << 16);
        r.a[3] = __uint_as_float(t.y & 0xffff0000u);
        return r;
    } else {
        const unsigned short t = ld_global<POL>(static_cast<const unsigned short *>(base) + idx);
        Vec<1> r;
        r.a[0] = __uint_as_float(static_cast<unsigned>(t) << 16);
        return r;
    }
}

// Four consecutive gradient elements starting at element 4 idx, fetched one by
// one: for a gradient whose offset from a 16-byte boundary differs from the
// parameters', while every other stream keeps its 128-bit accesses.
template <int GT>
__device__ __forceinline__ Vec<4> load_grad_split(const void *base, int idx)
{
    Vec<4> r;
#pragma unroll
    for (int e = 0; e < 4; ++e) r.a[e] = load_grad<1, GT>(base, 4 * idx + e).a[0];
    return r;
}

// Moments as stored: fp32, or bf16 (M16) widened exactly on load and rounded to
// nearest even on store.
template <int N, bool M16, int POL = LD_STREAM>
__device__ __forceinline__ Vec<N> load_moment(const void *base, int idx)
{
    if constexpr (M16) return load_grad<N, NOVAK_GRAD_BF16, POL>(base, idx);
    else return load_f32<N, POL>(static_cast<const float *>(base), idx);
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
    if constexpr ((PRE & PRE_MASK) == PRE_CENTER || (PRE & PRE_MASK) == PRE_CENTER_ROWS) {
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
    if constexpr ((PRE & PRE_MASK) == PRE_CENTER || (PRE & PRE_MASK) == PRE_CENTER_ROWS) {
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
    if constexpr ((PRE & PRE_MASK) == PRE_SCALE || (PRE & PRE_MASK) == PRE_CENTER) {
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
// GSPLIT (N = 4 only): the gradient is fetched element by element.
template <int N, int U, int NEST, int GT, int LA, int PRE, bool GSPLIT = false>
__device__ __forceinline__ void run_tile(float *p, const float *pin, const void *g, void *m, void *v,
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
        P[j] = load_f32<N>(pin, idx);
        if constexpr (GSPLIT) G[j] = load_grad_split<GT>(g, idx);
        else G[j] = load_grad<N, GT>(g, idx);
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
template <int N, int U, int NEST, int GT, int LA, int PRE, bool GSPLIT = false>
__device__ __forceinline__ void run_span(float *p, const float *pin, const void *g, void *m, void *v,
                                         float *slow, float *acc, int nvec,
                                         const StepScalars &s, const PreArgs &pre)
{
    constexpr int kTile = kBlock * U;
    int base = 0;
#pragma unroll 1
    for (; base + kTile <= nvec; base += kTile)
        run_tile<N, U, NEST, GT, LA, PRE, GSPLIT>(p, pin, g, m, v, slow, acc, base + threadIdx.x, s, pre);
#pragma unroll 1
    for (int idx = base + threadIdx.x; idx < nvec; idx += kBlock)
        run_tile<N, 1, NEST, GT, LA, PRE, GSPLIT>(p, pin, g, m, v, slow, acc, idx, s, pre);
}

// One chunk-table entry: 128-bit accesses where every stream shares 16-byte
// alignment; the same with the gradient alone fetched element by element where
// only the gradient is off; 4-byte accesses for everything otherwise.
template <int NEST, int GT, int LA, int PRE>
__device__ __forceinline__ void run_entry(const Chunk &ch, const TensorRec &r, const StepScalars &s,
                                          const PreArgs &pre)
{
    constexpr int kGradBytes = (GT == NOVAK_GRAD_BF16) ? 2 : 4;
    constexpr int kMomBytes = (PRE & PRE_MOM16) ? 2 : 4;
    constexpr bool kUseS = (LA & (LA_S_READ | LA_S_WRITE)) != 0;
    constexpr bool kUseA = (LA & (LA_A_READ | LA_A_WRITE)) != 0;
    float *p = r.p + ch.offset;
    const float *pin = r.p_in + ch.offset;
    void *m = static_cast<char *>(r.m) + ch.offset * kMomBytes;
    void *v = static_cast<char *>(r.v) + ch.offset * kMomBytes;
    float *slow = kUseS ? r.slow + ch.offset : nullptr;
    float *acc = kUseA ? r.acc + ch.offset : nullptr;
    const void *g = static_cast<const char *>(r.g) + ch.offset * kGradBytes;

    // four bf16 moments are one 64-bit access: half the parameters' alignment
    uintptr_t bits = reinterpret_cast<uintptr_t>(p) | reinterpret_cast<uintptr_t>(pin) |
                     ((reinterpret_cast<uintptr_t>(m) | reinterpret_cast<uintptr_t>(v))
                      << (kMomBytes == 2 ? 1 : 0));
    if (kUseS) bits |= reinterpret_cast<uintptr_t>(slow);
    if (kUseA) bits |= reinterpret_cast<uintptr_t>(acc);
    // the 64-bit stores of the bf16 copy need half the parameters' alignment
    if ((PRE & PRE_COPY16) != 0) bits |= reinterpret_cast<uintptr_t>(pre.copy) << 1;
    const bool state_aligned = (bits & 15u) == 0;
    const bool grad_aligned = (reinterpret_cast<uintptr_t>(g) & (4u * kGradBytes - 1u)) == 0;
    if (state_aligned) {
        const int nvec = ch.len >> 2;
        if (grad_aligned)
            run_span<4, kUnroll, NEST, GT, LA, PRE>(p, pin, g, m, v, slow, acc, nvec, s, pre);
        else
            run_span<4, kUnroll, NEST, GT, LA, PRE, true>(p, pin, g, m, v, slow, acc, nvec, s, pre);
        // ragged tail of a tensor: at most 3 elements
        const int idx = (nvec << 2) + threadIdx.x;
        if (idx < ch.len)
            run_tile<1, 1, NEST, GT, LA, PRE>(p, pin, g, m, v, slow, acc, idx, s, pre);
    } else {
        // parameter and state do not share 16-byte alignment
        run_span<1, 4, NEST, GT, LA, PRE>(p, pin, g, m, v, slow, acc, ch.len, s, pre);
    }
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

// Resident CTAs per SM an instantiation is compiled for.
constexpr int step_min_ctas(int la)
{
    // (the first step of a TRAJ_MEAN window only adds an output stream and measured
    // 3-6 % faster at four CTAs)
    return (la & (LA_S_READ | LA_A_READ | LA_S_INIT)) != 0 ? NOVAK_MIN_CTAS_WIDE : NOVAK_MIN_CTAS;
}

template <int NEST, int GT, int LA, int PRE>
__global__ void __launch_bounds__(NOVAK_BLOCK, step_min_ctas(LA))
novak_step_kernel(const Chunk *__restrict__ chunks, int n_chunks,
                  const TensorRec *__restrict__ recs, const PrepOut *prep,
                  const float *trust, const StepScalars s, int reverse)
{
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
    if constexpr ((PRE & PRE_MASK) == PRE_SCALE || (PRE & PRE_MASK) == PRE_CENTER) {
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
        run_entry<NEST, GT, LA, PRE>(ch, r, s, pre);
        c += gridDim.x;
        if (c >= n_chunks) break;
        ch = chunks[reverse ? n_chunks - 1 - c : c];
        r = recs[ch.tensor];
    }
}

// ---- PRE_CENTER_ROWS: Eq. 26 inside the step kernel ------------------------
// The row mean is a statistic of ONE row, so a CTA that owns whole rows can
// form it from the gradient it is about to consume.  Units of up to
// kOwnStageElems elements: the CTA loads its rows' gradient once, all loads in
// flight together, into shared memory (as fp32), adds the rows up from there
// and then takes the gradient of the ordinary update from shared memory
// instead of global memory.  A single longer row: added up from global memory
// by the whole CTA (default caching), then read again by the update, which
// finds it in L1 / L2.  Either way DRAM sees every byte once (28 B per
// element) and the step is one launch; the first tile's parameters and state
// are already on their way while the rows are added up.

// Gradient elements [e0, e0 + L) of a tensor, added up in double by `nthreads`
// threads of which this is number t: 4-element vectors where the row allows it
// (after up to three leading elements), single elements at both ends.
template <int GT>
__device__ __forceinline__ double row_partial_sum(const void *g_tensor, int64_t e0, uint32_t L,
                                                  uint32_t t, uint32_t nthreads)
{
    constexpr uint32_t kB = (GT == NOVAK_GRAD_BF16) ? 2u : 4u;
    const char *row = static_cast<const char *>(g_tensor) + static_cast<size_t>(e0) * kB;
    auto elem = [&](uint32_t i) -> float {
        if constexpr (GT == NOVAK_GRAD_F32) return reinterpret_cast<const float *>(row)[i];
        else return __uint_as_float(static_cast<unsigned>(
            reinterpret_cast<const unsigned short *>(row)[i]) << 16);
    };
    const uint32_t mis = static_cast<uint32_t>((reinterpret_cast<uintptr_t>(row) / kB) & 3u);
    const uint32_t head = min(L, (4u - mis) & 3u);
    const uint32_t nvec = (L - head) >> 2;
    const uint32_t tail0 = head + (nvec << 2);
    double sum = 0.0;
    if (t < head) sum += double(elem(t));
    const char *body = row + static_cast<size_t>(head) * kB;
#pragma unroll 8
    for (uint32_t v = t; v < nvec; v += nthreads) {
        float x0, x1, x2, x3;
        if constexpr (GT == NOVAK_GRAD_F32) {
            const float4 q = reinterpret_cast<const float4 *>(body)[v];
            x0 = q.x; x1 = q.y; x2 = q.z; x3 = q.w;
        } else {
            const uint2 q = reinterpret_cast<const uint2 *>(body)[v];
            x0 = __uint_as_float(q.x << 16); x1 = __uint_as_float(q.x & 0xffff0000u);
            x2 = __uint_as_float(q.y << 16); x3 = __uint_as_float(q.y & 0xffff0000u);
        }
        sum += (double(x0) + double(x1)) + (double(x2) + double(x3));
    }
    if (t < L - tail0) sum += double(elem(tail0 + t));
    return sum;
}

// A mean as hi + lo floats (see preprocess()).
__device__ __forceinline__ float2 split_mean(double sum, uint32_t L)
{
    const double mu = sum / double(L);
    const float hi = static_cast<float>(mu);
    return make_float2(hi, static_cast<float>(mu - double(hi)));
}

// Means of the unit's n_rows rows of L elements (the first starting at element
// e0 of the tensor) into sh_mean[0 .. n_rows).  A warp per row where the unit
// has a row for every warp, the whole CTA row after row otherwise.  Fixed
// summation order: bit-identical from run to run.
template <int GT>
__device__ __forceinline__ void unit_row_means(const void *g_tensor, int64_t e0, uint32_t n_rows,
                                               uint32_t L, float2 *sh_mean, double *sh_red)
{
    constexpr uint32_t kWarps = kBlock / 32;
    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31u;
    if (n_rows >= kWarps) {
        for (uint32_t r = warp; r < n_rows; r += kWarps) {
            double sum = row_partial_sum<GT>(g_tensor, e0 + r * L, L, lane, 32u);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
            if (lane == 0u) sh_mean[r] = split_mean(sum, L);
        }
    } else {
        for (uint32_t r = 0; r < n_rows; ++r) {
            double sum = row_partial_sum<GT>(g_tensor, e0 + r * L, L, threadIdx.x, kBlock);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
            __syncthreads();             // sh_red may still be read for the previous row
            if (lane == 0u) sh_red[warp] = sum;
            __syncthreads();
            if (threadIdx.x == 0) {
                double total = 0.0;
#pragma unroll
                for (uint32_t w = 0; w < kWarps; ++w) total += sh_red[w];
                sh_mean[r] = split_mean(total, L);
            }
        }
    }
    __syncthreads();
}

// The unit's n gradient elements as fp32 into shared memory, sh_g[mis + i] =
// g[i]: `mis` is the parameters' offset (in elements) from a 16-byte boundary,
// so that the update's aligned 4-element vectors are aligned in shared memory
// too.  128-bit (64-bit for bf16) global loads, four per thread in flight, where
// the gradient shares that phase; element by element otherwise.
template <int GT>
__device__ __forceinline__ void stage_gradient(const void *g_unit, uint32_t n, uint32_t mis, float *sh_g)
{
    constexpr uint32_t kB = (GT == NOVAK_GRAD_BF16) ? 2u : 4u;
    const char *src = static_cast<const char *>(g_unit);
    const uint32_t t = threadIdx.x;
    const uint32_t gmis = static_cast<uint32_t>((reinterpret_cast<uintptr_t>(src) / kB) & 3u);
    if (gmis == mis) {
        const uint32_t head = min(n, (4u - mis) & 3u);
        const uint32_t nvec = (n - head) >> 2;
        const uint32_t tail0 = head + (nvec << 2);
        if (t < head) sh_g[mis + t] = load_grad<1, GT>(src, static_cast<int>(t)).a[0];
        if (t < n - tail0) sh_g[mis + tail0 + t] = load_grad<1, GT>(src, static_cast<int>(tail0 + t)).a[0];
        const char *body = src + static_cast<size_t>(head) * kB;
        float4 *dst = reinterpret_cast<float4 *>(sh_g + mis + head);
#pragma unroll 1
        for (uint32_t v0 = 0; v0 < nvec; v0 += 4u * kBlock) {
            Vec<4> x[4];
#pragma unroll
            for (uint32_t k = 0; k < 4u; ++k) {
                const uint32_t v = v0 + k * kBlock + t;
                if (v < nvec) x[k] = load_grad<4, GT>(body, static_cast<int>(v));
            }
#pragma unroll
            for (uint32_t k = 0; k < 4u; ++k) {
                const uint32_t v = v0 + k * kBlock + t;
                if (v < nvec) dst[v] = make_float4(x[k].a[0], x[k].a[1], x[k].a[2], x[k].a[3]);
            }
        }
    } else {
#pragma unroll 1
        for (uint32_t i0 = 0; i0 < n; i0 += 8u * kBlock) {
            float x[8];
#pragma unroll
            for (uint32_t k = 0; k < 8u; ++k) {
                const uint32_t i = i0 + k * kBlock + t;
                if (i < n) x[k] = load_grad<1, GT>(src, static_cast<int>(i)).a[0];
            }
#pragma unroll
            for (uint32_t k = 0; k < 8u; ++k) {
                const uint32_t i = i0 + k * kBlock + t;
                if (i < n) sh_g[mis + i] = x[k];
            }
        }
    }
}

// Means of n_rows rows of L staged elements (rows[r * L + i]) into sh_mean:
// a warp per row where the unit has a row for every warp, the whole CTA row
// after row otherwise.  Fixed order.
__device__ __forceinline__ void staged_row_means(const float *rows, uint32_t n_rows, uint32_t L,
                                                 float2 *sh_mean, double *sh_red)
{
    constexpr uint32_t kWarps = kBlock / 32;
    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31u;
    // rows of whole, aligned 4-element vectors: one 128-bit read per four elements
    const bool quads = (L & 3u) == 0u && (reinterpret_cast<uintptr_t>(rows) & 15u) == 0;
    auto strided_sum = [&](const float *row, uint32_t t, uint32_t nthreads) -> double {
        double sum = 0.0;
        if (quads) {
            const float4 *q = reinterpret_cast<const float4 *>(row);
            for (uint32_t i = t; i < (L >> 2); i += nthreads) {
                const float4 x = q[i];
                sum += (double(x.x) + double(x.y)) + (double(x.z) + double(x.w));
            }
        } else {
            for (uint32_t i = t; i < L; i += nthreads) sum += double(row[i]);
        }
        return sum;
    };
    if (n_rows >= kWarps) {
        for (uint32_t r = warp; r < n_rows; r += kWarps) {
            double sum = strided_sum(rows + r * L, lane, 32u);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
            if (lane == 0u) sh_mean[r] = split_mean(sum, L);
        }
    } else {
        for (uint32_t r = 0; r < n_rows; ++r) {
            double sum = strided_sum(rows + r * L, threadIdx.x, kBlock);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
            __syncthreads();             // sh_red may still be read for the previous row
            if (lane == 0u) sh_red[warp] = sum;
            __syncthreads();
            if (threadIdx.x == 0) {
                double total = 0.0;
#pragma unroll
                for (uint32_t w = 0; w < kWarps; ++w) total += sh_red[w];
                sh_mean[r] = split_mean(total, L);
            }
        }
    }
    __syncthreads();
}

// The streams of one unit's vector body: nvec aligned 4-element vectors.
struct UnitBody {
    float *p;
    const float *pin;
    const void *g;
    void *m, *v;
    float *slow, *acc;
    __nv_bfloat16 *copy;
    int nvec;
    bool g_vector;      // the gradient shares the streams' 16-byte phase
    const float4 *staged;   // the body's gradient in shared memory, NULL: take it from g
};

// One tile of a unit's body in three steps, so that a tile's parameter and
// state loads can be in flight while the CTA is still adding up its rows:
// everything but the gradient, then the gradient, then the update and the
// stores.  Vectors beyond nvec are skipped (a unit rarely fills its last tile).
template <int U>
struct TileRegs {
    Vec<4> P[U], G[U], M[U], V[U], S[U], A[U];
};

template <int U, int LA, int PRE>
__device__ __forceinline__ void unit_tile_prefetch(TileRegs<U> &t, const UnitBody &b, int first)
{
    constexpr bool kMom16 = (PRE & PRE_MOM16) != 0;
#pragma unroll
    for (int j = 0; j < U; ++j) {
        const int idx = first + j * kBlock;
        if (idx < b.nvec) {
            t.P[j] = load_f32<4>(b.pin, idx);
            t.M[j] = load_moment<4, kMom16>(b.m, idx);
            t.V[j] = load_moment<4, kMom16>(b.v, idx);
            if constexpr ((LA & LA_S_READ) != 0) t.S[j] = load_f32<4>(b.slow, idx);
            if constexpr ((LA & LA_A_READ) != 0) t.A[j] = load_f32<4>(b.acc, idx);
        }
    }
}

template <int U, int GT>
__device__ __forceinline__ void unit_tile_grad(TileRegs<U> &t, const UnitBody &b, int first)
{
#pragma unroll
    for (int j = 0; j < U; ++j) {
        const int idx = first + j * kBlock;
        if (idx < b.nvec && b.staged == nullptr)     // (a staged gradient is taken at the update)
            t.G[j] = b.g_vector ? load_grad<4, GT>(b.g, idx) : load_grad_split<GT>(b.g, idx);
    }
}

template <int U, int NEST, int LA, int PRE>
__device__ __forceinline__ void unit_tile_finish(TileRegs<U> &t, const UnitBody &b, int first,
                                                 const StepScalars &s, const PreArgs &pre)
{
    constexpr bool kMom16 = (PRE & PRE_MOM16) != 0;
#pragma unroll
    for (int j = 0; j < U; ++j) {
        const int idx = first + j * kBlock;
        if (idx < b.nvec) {
            if (b.staged != nullptr) {           // the gradient waits in shared memory
                const float4 q = b.staged[idx];
                t.G[j].a[0] = q.x; t.G[j].a[1] = q.y; t.G[j].a[2] = q.z; t.G[j].a[3] = q.w;
            }
            preprocess<4, PRE>(t.G[j], row_position<PRE>(pre.elem0 + static_cast<uint32_t>(idx) * 4u, pre), pre);
#pragma unroll
            for (int e = 0; e < 4; ++e)
                update_element<NEST, LA>(t.P[j].a[e], t.G[j].a[e], t.M[j].a[e], t.V[j].a[e],
                                         t.S[j].a[e], t.A[j].a[e], s, pre.step);
            store_f32<4>(b.p, idx, t.P[j]);
            if constexpr ((PRE & PRE_COPY16) != 0) store_bf16<4>(b.copy, idx, t.P[j]);
            store_moment<4, kMom16>(b.m, idx, t.M[j]);
            store_moment<4, kMom16>(b.v, idx, t.V[j]);
            if constexpr ((LA & LA_S_WRITE) != 0) store_f32<4>(b.slow, idx, t.S[j]);
            if constexpr ((LA & LA_A_WRITE) != 0) store_f32<4>(b.acc, idx, t.A[j]);
        }
    }
}

// Vectors per thread and stream of the row-owning kernel's tiles, and its
// registers per thread: as the plain kernel's.  (Measured on the ResNet-50-
// shaped set with CTAs of 256 threads, ms per step: two vectors at four CTAs
// 0.138; four vectors at three CTAs, a whole unit in flight at once, 0.158; one
// vector at six CTAs 0.182.)
#ifndef NOVAK_ROWS_U
#define NOVAK_ROWS_U 2
#endif
template <int LA>
constexpr int kRowsUnroll = (LA & (LA_S_READ | LA_A_READ)) != 0 ? 2 : NOVAK_ROWS_U;
#ifndef NOVAK_ROWS_MIN_CTAS
#define NOVAK_ROWS_MIN_CTAS step_min_ctas(LA)
#endif

template <int NEST, int GT, int LA, int PRE>
__global__ void __launch_bounds__(NOVAK_BLOCK, NOVAK_ROWS_MIN_CTAS)
novak_step_rows_kernel(const Chunk *__restrict__ rest, int n_rest,
                       const RowUnit *__restrict__ units, int n_units,
                       const TensorRec *__restrict__ recs, const StepScalars s)
{
    static_assert((PRE & PRE_MASK) == PRE_CENTER_ROWS, "the row-owning kernel is its own mode");
    static_assert((PRE & PRE_MASK) != PRE_CENTER_ROWS || kBlock == kOwnBlockThreads,
                  "compiled for the block size it is launched with");
    constexpr int kGradBytes = (GT == NOVAK_GRAD_BF16) ? 2 : 4;
    constexpr int kMomBytes = (PRE & PRE_MOM16) ? 2 : 4;
    constexpr bool kUseS = (LA & (LA_S_READ | LA_S_WRITE)) != 0;
    constexpr bool kUseA = (LA & (LA_A_READ | LA_A_WRITE)) != 0;
    constexpr int kU = kRowsUnroll<LA>;
    constexpr int kTile = kBlock * kU;
    __shared__ __align__(16) float sh_g[kOwnStageElems + 4];
    __shared__ float2 sh_mean[kOwnUnitRows];
    __shared__ double sh_red[kBlock / 32];

    grid_dependency_release();
    const int blk = blockIdx.x;
    PreArgs pre;
    pre.factor = 1.0f;
    pre.step = s.step;
    if (blk < n_rest) {
        // a tensor without rows (mean is NULL), or with rows too long to own: their
        // means are in the record, written by the statistics pass before this launch
        const Chunk ch = rest[blk];
        const TensorRec r = recs[ch.tensor];
        grid_dependency_wait();
        pre.mean = r.mean;
        pre.row_len = r.row_len;
        pre.elem0 = static_cast<uint32_t>(ch.offset);
        pre.copy = ((PRE & PRE_COPY16) != 0) ? r.p16 + ch.offset : nullptr;
        run_entry<NEST, GT, LA, PRE>(ch, r, s, pre);
        return;
    }
    if (blk - n_rest >= n_units) return;
    const RowUnit u = units[blk - n_rest];
    const TensorRec r = recs[u.tensor];
    grid_dependency_wait();

    const uint32_t L = r.row_len;
    const int64_t e0 = static_cast<int64_t>(u.row0) * L;   // the unit's first element in its tensor
    const uint32_t n = u.n_rows * L;

    // The unit starts wherever its first row starts: up to three single elements
    // bring every stream to a 16-byte boundary together (parameters and state
    // share their tensor's phase), then vectors, then up to three at the end.
    const uint32_t mis = static_cast<uint32_t>((reinterpret_cast<uintptr_t>(r.p + e0) >> 2) & 3u);
    const uint32_t head = min(n, (4u - mis) & 3u);
    const int64_t b0 = e0 + head;
    UnitBody b;
    b.p = r.p + b0;
    b.pin = r.p_in + b0;
    b.g = static_cast<const char *>(r.g) + b0 * kGradBytes;
    b.m = static_cast<char *>(r.m) + b0 * kMomBytes;
    b.v = static_cast<char *>(r.v) + b0 * kMomBytes;
    b.slow = kUseS ? r.slow + b0 : nullptr;
    b.acc = kUseA ? r.acc + b0 : nullptr;
    b.copy = ((PRE & PRE_COPY16) != 0) ? r.p16 + b0 : nullptr;
    b.nvec = static_cast<int>((n - head) >> 2);
    b.g_vector = (reinterpret_cast<uintptr_t>(b.g) & (4u * kGradBytes - 1u)) == 0;
    // vectors need every stream on its boundary; streams that disagree (state attached
    // for other parameter addresses, a bf16 copy at another phase): single elements
    uintptr_t bits = reinterpret_cast<uintptr_t>(b.p) | reinterpret_cast<uintptr_t>(b.pin) |
                     ((reinterpret_cast<uintptr_t>(b.m) | reinterpret_cast<uintptr_t>(b.v))
                      << (kMomBytes == 2 ? 1 : 0));
    if (kUseS) bits |= reinterpret_cast<uintptr_t>(b.slow);
    if (kUseA) bits |= reinterpret_cast<uintptr_t>(b.acc);
    if ((PRE & PRE_COPY16) != 0) bits |= reinterpret_cast<uintptr_t>(b.copy) << 1;
    const bool vectors = (bits & 15u) == 0;
    if (!vectors) b.nvec = 0;

    // first tile: parameters and state on their way while the rows are added up
    TileRegs<kU> t;
    unit_tile_prefetch<kU, LA, PRE>(t, b, threadIdx.x);
    b.staged = nullptr;
    if (n <= kOwnStageElems) {
        stage_gradient<GT>(static_cast<const char *>(r.g) + e0 * kGradBytes, n, mis, sh_g);
        __syncthreads();
        staged_row_means(sh_g + mis, u.n_rows, L, sh_mean, sh_red);
        if (vectors) b.staged = reinterpret_cast<const float4 *>(sh_g + mis + head);
    } else {
        unit_row_means<GT>(r.g, e0, u.n_rows, L, sh_mean, sh_red);
    }
    pre.mean = sh_mean;                              // indexed by the row within the unit
    pre.row_len = L;
    pre.elem0 = head;                                // position within the unit
    pre.copy = b.copy;
    unit_tile_grad<kU, GT>(t, b, threadIdx.x);  // from shared memory, or cache hits
    unit_tile_finish<kU, NEST, LA, PRE>(t, b, threadIdx.x, s, pre);
#pragma unroll 1
    for (int base = kTile; base < b.nvec; base += kTile) {
        unit_tile_prefetch<kU, LA, PRE>(t, b, base + threadIdx.x);
        unit_tile_grad<kU, GT>(t, b, base + threadIdx.x);
        unit_tile_finish<kU, NEST, LA, PRE>(t, b, base + threadIdx.x, s, pre);
    }

    // the single elements at both ends (all of the unit where vectors are not possible)
    Chunk ch;
    ch.tensor = u.tensor;
    if (head != 0u) {
        ch.len = static_cast<int32_t>(head);
        ch.offset = e0;
        pre.elem0 = 0u;
        pre.copy = ((PRE & PRE_COPY16) != 0) ? r.p16 + ch.offset : nullptr;
        run_entry<NEST, GT, LA, PRE>(ch, r, s, pre);
    }
    const uint32_t done = head + (static_cast<uint32_t>(b.nvec) << 2);
    if (done < n) {
        ch.len = static_cast<int32_t>(n - done);
        ch.offset = e0 + done;
        pre.elem0 = done;
        pre.copy = ((PRE & PRE_COPY16) != 0) ? r.p16 + ch.offset : nullptr;
        run_entry<NEST, GT, LA, PRE>(ch, r, s, pre);
    }
}

using StepKernelFn = void (*)(const Chunk *, int, const TensorRec *, const PrepOut *,
                              const float *, StepScalars, int);
using StepRowsKernelFn = void (*)(const Chunk *, int, const RowUnit *, int, const TensorRec *,
                                  StepScalars);

// The instantiation for a step's modes, as an untyped pointer: a StepKernelFn,
// or a StepRowsKernelFn when PRE is a PRE_CENTER_ROWS mode.
template <int NEST, int GT, int PRE>
void *pick_la(int la)
{
    switch (la) {
#define NOVAK_LA_CASE(X) case (X): \
        if constexpr ((PRE & PRE_MASK) == PRE_CENTER_ROWS) \
            return reinterpret_cast<void *>(novak_step_rows_kernel<NEST, GT, (X), PRE>); \
        else \
            return reinterpret_cast<void *>(novak_step_kernel<NEST, GT, (X), PRE>);
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
void *pick_gt(int grad_dtype, int la)
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
void *pick_step_kernel(int nesterov, int grad_dtype, int la)
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
