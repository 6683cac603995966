// Layer-wise adaptation (Eq. 19 / 25) and the step in ONE launch for sm_100a.
//
// The trust ratio of a tensor needs ||u_t|| over the whole tensor before any of
// its elements moves.  Run as two passes over the whole group
// (novak_trust_stats.cu, then the step kernel) theta, g, m, v are read twice,
// and the second pass finds nothing of the first in L2: 16 + 28 B per element
// from DRAM.  Here the work is cut differently.  The group is a list of ITEMS (a
// few consecutive chunk-table entries of one tensor each), and CTA number b does
// two things:
//
//   S part, item b: the whole of phases 2-8 for the item's elements - moments
//       advanced and stored for good, the direction the update will multiply by
//       the step (Eq. 17 after Eq. 27 and Eq. 16) left in a scratch array, the
//       squares of theta and of the base direction added up.  The CTA that
//       completes a tensor's last S part adds the tensor's sums in table order
//       (fixed order: bit-identical from run to run) and publishes the ratio as
//       one 64-bit word (launch number, ratio).
//   U part, item b - lag: phases 9-10 from theta and the stored direction, both
//       of which the S part of that item touched a few tens of MB of traffic
//       ago and which are still in the 126 MB L2.
//
// DRAM sees theta, g, m, v once and m, v, theta written once: about 30 B per
// element instead of 44.  The operations and their order are those of
// update_element(), cut in two after the direction: results are bit-identical
// to the two-pass route.
//
// The wait and forward progress: the U part waits for its tensor's word.  lag
// is at least the number of items of the longest tensor minus one, so the S
// parts it waits for belong to CTAs with a lower block index (or to this CTA,
// which has finished its own S part by then), and an S part never waits.  The
// hardware hands out the CTAs of a grid in increasing block index as slots
// become free (the behaviour single-pass scans with look-back rely on as well),
// so those CTAs are running or have finished, and the word is there when it is
// asked for or shortly after (a longer lag makes the wait rarer but lets theta
// and the direction leave L2 before the U part comes for them; measured, the
// shortest lag is the fastest).  With gradient pre-processing on, the clip
// factor, the row means and Eq. 22 come from the statistics pass in front of
// this launch and the S part applies them to g first.
// Nothing in the programming model promises that order, so the wait is
// bounded: after about two seconds (at once, when another CTA has already given
// up) a warp gives up, raises an error flag in host-mapped memory, leaves its
// share of the item's parameters untouched (the moments HAVE advanced) and
// returns; the next call on the handle reports it, and
// NOVAK_OPT_LAYER_ADAPTATION_IN_STEP = 0 selects the three-launch form.
#pragma once

#include "novak_trust.cuh"

namespace novak {
namespace {

constexpr unsigned long long kAdaptWaitLimitNs = 2000000000ull;
constexpr unsigned kAdaptWaitLimitSpins = 1u << 25;

__device__ __forceinline__ unsigned long long global_timer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ unsigned long long load_acquire(const unsigned long long *p)
{
    unsigned long long v;
    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ void store_release(unsigned long long *p, unsigned long long v)
{
    asm volatile("st.release.gpu.global.u64 [%0], %1;" :: "l"(p), "l"(v) : "memory");
}

// A tensor's published word: the launch it belongs to (high half) and the ratio.
__device__ __forceinline__ unsigned long long pack_ratio(unsigned epoch, float ratio)
{
    return (static_cast<unsigned long long>(epoch) << 32) | __float_as_uint(ratio);
}

// Waits until the word's launch number is `epoch`; returns the word, or 0 when
// it gave up (time or iteration limit, or another CTA has given up already).
__device__ __forceinline__ unsigned long long wait_for_ratio(const unsigned long long *word,
                                                             unsigned epoch, const unsigned *error)
{
    unsigned long long w = load_acquire(word);
    if (static_cast<unsigned>(w >> 32) == epoch) return w;
    const unsigned long long t0 = global_timer_ns();
    for (unsigned spins = 0; spins < kAdaptWaitLimitSpins; ++spins) {
        __nanosleep(100);
        w = load_acquire(word);
        if (static_cast<unsigned>(w >> 32) == epoch) return w;
        if ((spins & 255u) == 255u &&
            (*reinterpret_cast<const volatile unsigned *>(error) != 0u ||
             global_timer_ns() - t0 > kAdaptWaitLimitNs))
            return 0ull;
    }
    return 0ull;
}

// The bound of that wait, on its own: one thread waits for a word that nothing
// publishes and reports what it got (0: gave up) and how long it waited.
__global__ void novak_adapt_wait_probe_kernel(const unsigned long long *word, unsigned epoch,
                                              const unsigned *error, unsigned long long *out)
{
    if (blockIdx.x != 0 || threadIdx.x != 0) return;
    const unsigned long long t0 = global_timer_ns();
    out[0] = wait_for_ratio(word, epoch, error);
    out[1] = global_timer_ns() - t0;
}

// ---- the direction a step applies, formed once -------------------------------
// An S item advances the moments for good and leaves, element by element, the
// direction the update multiplies by the step (Eq. 17 after the mask of Eq. 27
// and the blend of Eq. 16) in a scratch array; the U item reads it back from L2.
// The operations and their order are those of update_element(), cut in two
// after the direction: results are bit-identical to the two-pass route.

// Phases 2, 4, 5, 8 for U vectors of N elements per thread (vectors beyond nvec
// are skipped): every load issued before the first use; moments advanced and
// stored, direction stored, the squares of theta and of the base direction
// added up vector by vector in index order.
template <int N, int U, int NEST, int GT, int PRE>
__device__ __forceinline__ void direction_tile(const float *p, const void *g, void *m, void *v,
                                               float *d, int first, int nvec, const StepScalars &s,
                                               const PreArgs &pre, double &sum_p, double &sum_u)
{
    constexpr bool kMom16 = (PRE & PRE_MOM16) != 0;
    Vec<N> P[U], G[U], M[U], V[U];
#pragma unroll
    for (int j = 0; j < U; ++j) {
        const int idx = first + j * kBlock;
        if (idx < nvec) {
            P[j] = load_f32<N, LD_KEEP>(p, idx);        // the U item reads theta again
            G[j] = load_grad<N, GT>(g, idx);
            M[j] = load_moment<N, kMom16>(m, idx);
            V[j] = load_moment<N, kMom16>(v, idx);
        }
    }
#pragma unroll
    for (int j = 0; j < U; ++j) {
        const int idx = first + j * kBlock;
        if (idx < nvec) {
            Vec<N> D;
            // phase 2 on the gradient first: clip factor and row means, the statistics pass's output
            preprocess<N, PRE>(G[j], row_position<PRE>(pre.elem0 + static_cast<uint32_t>(idx) * N, pre), pre);
            float sp = 0.0f, su = 0.0f;
#pragma unroll
            for (int e = 0; e < N; ++e) {
                float m_hat;
                float u = base_direction<NEST>(G[j].a[e], M[j].a[e], V[j].a[e], m_hat, s);
                sp = fmaf(P[j].a[e], P[j].a[e], sp);
                su = fmaf(u, u, su);                            // Eq. 19: the unmasked base direction
                u = (fabsf(u) <= s.sparse_tau) ? 0.0f : u;      // Eq. 27
                if constexpr (NEST == NOVAK_NESTEROV_CLASSICAL)
                    u = fmaf(s.blend_b1, m_hat, s.blend_omb1 * u);      // Eq. 16
                D.a[e] = u;
            }
            sum_p += double(sp);
            sum_u += double(su);
            store_moment<N, kMom16>(m, idx, M[j]);
            store_moment<N, kMom16>(v, idx, V[j]);
            // default policy: the line stays in L2 for the U item
            if constexpr (N == 4)
                reinterpret_cast<float4 *>(d)[idx] = make_float4(D.a[0], D.a[1], D.a[2], D.a[3]);
            else
                d[idx] = D.a[0];
        }
    }
}

// One chunk-table entry of an S item; every thread returns its share of the
// two sums (the vectors it took, in index order).
template <int NEST, int GT, int PRE>
__device__ __forceinline__ void entry_direction(const Chunk &ch, const TensorRec &r, float *d,
                                                const StepScalars &s, const PreArgs &pre,
                                                double &sum_p, double &sum_u)
{
    constexpr int kGradBytes = (GT == NOVAK_GRAD_BF16) ? 2 : 4;
    constexpr int kMomBytes = (PRE & PRE_MOM16) ? 2 : 4;
    const float *p = r.p_in + ch.offset;     // theta_{t-1}
    void *m = static_cast<char *>(r.m) + ch.offset * kMomBytes;
    void *v = static_cast<char *>(r.v) + ch.offset * kMomBytes;
    const void *g = static_cast<const char *>(r.g) + ch.offset * kGradBytes;
    const uintptr_t bits = reinterpret_cast<uintptr_t>(p) |
                           ((reinterpret_cast<uintptr_t>(m) | reinterpret_cast<uintptr_t>(v))
                            << (kMomBytes == 2 ? 1 : 0));
    const bool aligned = (bits & 15u) == 0 &&
                         (reinterpret_cast<uintptr_t>(g) & (4u * kGradBytes - 1u)) == 0;
    sum_p = 0.0;
    sum_u = 0.0;
    if (aligned) {
        const int nvec = ch.len >> 2;
#pragma unroll 1
        for (int base = 0; base < nvec; base += kBlock * 2)
            direction_tile<4, 2, NEST, GT, PRE>(p, g, m, v, d, base + threadIdx.x, nvec, s, pre, sum_p, sum_u);
        // ragged tail: < 4 elements
        direction_tile<1, 1, NEST, GT, PRE>(p, g, m, v, d, (nvec << 2) + threadIdx.x, ch.len, s,
                                            pre, sum_p, sum_u);
    } else {
#pragma unroll 1
        for (int base = 0; base < ch.len; base += kBlock * 4)
            direction_tile<1, 4, NEST, GT, PRE>(p, g, m, v, d, base + threadIdx.x, ch.len, s,
                                                pre, sum_p, sum_u);
    }
}

// Phases 9 and 10 (Eq. 18, 24, 28-31) for one element from its stored direction.
template <int LA>
__device__ __forceinline__ void apply_direction(float &p, float u, float &slow, float &acc,
                                                const StepScalars &s, float step)
{
    const float theta_in = p;
    const float theta_fast = fmaf(theta_in, s.decay, -(step * u));
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

// U vectors of N elements per thread, every load issued before the first use.
// The direction was written by another CTA of this grid: L2 loads.
template <int N, int U, int LA, int PRE>
__device__ __forceinline__ void apply_tile(float *p, const float *pin, const float *d, float *slow,
                                           float *acc, __nv_bfloat16 *copy, int first, int nvec,
                                           const StepScalars &s, float step)
{
    constexpr bool kReadS = (LA & LA_S_READ) != 0;
    constexpr bool kWriteS = (LA & LA_S_WRITE) != 0;
    constexpr bool kReadA = (LA & LA_A_READ) != 0;
    constexpr bool kWriteA = (LA & LA_A_WRITE) != 0;
    Vec<N> P[U], D[U], S[U], A[U];
#pragma unroll
    for (int j = 0; j < U; ++j) {
        const int idx = first + j * kBlock;
        if (idx < nvec) {
            P[j] = load_f32<N>(pin, idx);
            D[j] = load_f32<N, LD_KEEP>(d, idx);
            if constexpr (kReadS) S[j] = load_f32<N>(slow, idx);
            if constexpr (kReadA) A[j] = load_f32<N>(acc, idx);
        }
    }
#pragma unroll
    for (int j = 0; j < U; ++j) {
        const int idx = first + j * kBlock;
        if (idx < nvec) {
#pragma unroll
            for (int e = 0; e < N; ++e)
                apply_direction<LA>(P[j].a[e], D[j].a[e], S[j].a[e], A[j].a[e], s, step);
            store_f32<N>(p, idx, P[j]);
            if constexpr ((PRE & PRE_COPY16) != 0) store_bf16<N>(copy, idx, P[j]);
            if constexpr (kWriteS) store_f32<N>(slow, idx, S[j]);
            if constexpr (kWriteA) store_f32<N>(acc, idx, A[j]);
        }
    }
}

// A U item: its entries are consecutive in their tensor and in the direction
// scratch (every entry but a tensor's first and last is slot_elems long), one span.
template <int LA, int PRE>
__device__ __forceinline__ void entry_apply(const Chunk &ch, const TensorRec &r, const float *d,
                                            const StepScalars &s, float step)
{
    constexpr bool kUseS = (LA & (LA_S_READ | LA_S_WRITE)) != 0;
    constexpr bool kUseA = (LA & (LA_A_READ | LA_A_WRITE)) != 0;
    // an item is a few entries long: four vectors per thread where the registers allow
    constexpr int kU = (LA & (LA_S_READ | LA_A_READ)) != 0 ? 2 : 4;
    float *p = r.p + ch.offset;
    const float *pin = r.p_in + ch.offset;
    float *slow = kUseS ? r.slow + ch.offset : nullptr;
    float *acc = kUseA ? r.acc + ch.offset : nullptr;
    __nv_bfloat16 *copy = ((PRE & PRE_COPY16) != 0) ? r.p16 + ch.offset : nullptr;
    uintptr_t bits = reinterpret_cast<uintptr_t>(p) | reinterpret_cast<uintptr_t>(pin);
    if (kUseS) bits |= reinterpret_cast<uintptr_t>(slow);
    if (kUseA) bits |= reinterpret_cast<uintptr_t>(acc);
    if ((PRE & PRE_COPY16) != 0) bits |= reinterpret_cast<uintptr_t>(copy) << 1;
    if ((bits & 15u) == 0) {
        const int nvec = ch.len >> 2;
#pragma unroll 1
        for (int base = 0; base < nvec; base += kBlock * kU)
            apply_tile<4, kU, LA, PRE>(p, pin, d, slow, acc, copy, base + threadIdx.x, nvec, s, step);
        // ragged tail of a tensor: at most 3 elements
        apply_tile<1, 1, LA, PRE>(p, pin, d, slow, acc, copy, (nvec << 2) + threadIdx.x, ch.len, s, step);
    } else {
#pragma unroll 1
        for (int base = 0; base < ch.len; base += kBlock * 4)
            apply_tile<1, 4, LA, PRE>(p, pin, d, slow, acc, copy, base + threadIdx.x, ch.len, s, step);
    }
}

// Resident CTAs per SM as for the plain step kernel's instantiation of the same
// lookahead action (three for every action measured 0.233 against 0.220 ms per
// step on the ResNet-50-shaped set).
#ifndef NOVAK_ADAPT_MIN_CTAS
#define NOVAK_ADAPT_MIN_CTAS step_min_ctas(LA)
#endif
template <int NEST, int GT, int LA, int PRE>
__global__ void __launch_bounds__(NOVAK_BLOCK, NOVAK_ADAPT_MIN_CTAS)
novak_step_adapt_kernel(const int *__restrict__ item_first, const Chunk *__restrict__ item_chunk,
                        int n_items, int lag, const TensorRec *__restrict__ recs, const PrepOut *prep,
                        const int *__restrict__ tensor_first, double *chunk_u2, double *chunk_p2,
                        float *trust, AdaptCtl *ctl, unsigned *arrived, unsigned long long *ready,
                        unsigned *host_error, float *direction, int slot_elems,
                        const StepScalars s, unsigned epoch)
{
    static_assert((PRE & PRE_MASK) != PRE_CENTER_ROWS, "the row-owning kernel is a form of its own");
    __shared__ double sh[kTrustWarps];
    __shared__ double sh_part[kAdaptGroupMax][2][kTrustWarps];
    __shared__ int sh_flag;

    grid_dependency_release();
    const int bs = blockIdx.x;               // item of the S part
    const int bu = bs - lag;                 // item of the U part
    const bool has_s = bs < n_items;
    const bool has_u = bu >= 0 && bu < n_items;
    // The item table and the records are written by copies only, never by a
    // kernel: read before the previous kernel on the stream has finished.
    int c_s = 0, c_u = 0;
    Chunk ch_s = {}, ch_u = {};
    if (has_s) { c_s = item_first[bs]; ch_s = item_chunk[bs]; }
    if (has_u) { c_u = item_first[bu]; ch_u = item_chunk[bu]; }
    grid_dependency_wait();

    // The clip factor and Eq. 22 are the statistics pass's output (it may still have been
    // running while this grid became resident): plain loads, only now.
    float factor = 1.0f, step_all = s.step;
    if constexpr ((PRE & PRE_MASK) == PRE_SCALE || (PRE & PRE_MASK) == PRE_CENTER) {
        factor = prep->factor;
        step_all *= prep->auto_scale;        // 1 when the scaling is off; Eq. 24a
    }

    TensorRec r_u = {};
    unsigned long long word = 0ull;          // lane 0: the U part's tensor's word, once it is this launch's
    if (has_s) {
        // ---- S part: moments, direction and the two sums of squares of each entry;
        // entry c_s + j keeps element e at d[j * slot_elems + e]
        const TensorRec r = recs[ch_s.tensor];
        float *d = direction + static_cast<size_t>(c_s) * static_cast<size_t>(slot_elems);
        const int c0 = tensor_first[ch_s.tensor], c1 = tensor_first[ch_s.tensor + 1];
        const int cnt = (ch_s.len + slot_elems - 1) / slot_elems;      // <= kAdaptGroupMax
        const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
#pragma unroll 1
        for (int j = 0; j < cnt; ++j) {
            Chunk sub;
            sub.tensor = ch_s.tensor;
            sub.offset = ch_s.offset + static_cast<int64_t>(j) * slot_elems;
            sub.len = min(slot_elems, ch_s.len - j * slot_elems);
            PreArgs pre;
            pre.copy = nullptr;
            pre.step = 0.0f;
            pre.factor = factor;
            pre.mean = ((PRE & PRE_MASK) == PRE_CENTER) ? r.mean : nullptr;
            pre.row_len = r.row_len;
            pre.elem0 = static_cast<uint32_t>(sub.offset);
            double sp, su;
            entry_direction<NEST, GT, PRE>(sub, r, d + static_cast<size_t>(j) * slot_elems, s, pre, sp, su);
            sp = trust_warp_sum(sp);
            su = trust_warp_sum(su);
            if (lane == 0) {
                sh_part[j][0][warp] = sp;
                sh_part[j][1][warp] = su;
            }
        }
        // the U part's record and its tensor's word: on their way during the reduction below
        if (has_u) {
            r_u = recs[ch_u.tensor];
            if (lane == 0) word = load_acquire(&ready[ch_u.tensor]);
        }
        __syncthreads();
        if (static_cast<int>(threadIdx.x) < cnt) {
            // warps in index order, as the two-pass route adds them
            double tp = 0.0, tu = 0.0;
#pragma unroll
            for (int w = 0; w < kTrustWarps; ++w) {
                tp += sh_part[threadIdx.x][0][w];
                tu += sh_part[threadIdx.x][1][w];
            }
            chunk_p2[c_s + threadIdx.x] = tp;
            chunk_u2[c_s + threadIdx.x] = tu;
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            __threadfence();                 // the CTA's sums and directions before the arrival
            const unsigned total = static_cast<unsigned>(c1 - c0);
            const unsigned before = atomicAdd(&arrived[ch_s.tensor], static_cast<unsigned>(cnt));
            sh_flag = (before + static_cast<unsigned>(cnt) == total) ? 1 : 0;
            // the tensor's last item leaves the counter at 0 for the next launch
            if (sh_flag) atomicExch(&arrived[ch_s.tensor], 0u);
        }
        __syncthreads();
        if (sh_flag != 0) {                  // (uniform over the CTA)
            // the tensor's last item: every sum is there
            __threadfence();
            const float eta = tensor_trust_ratio(chunk_p2, chunk_u2, c0, c1, sh);
            if (threadIdx.x == 0) {
                trust[ch_s.tensor] = eta;    // for novak_get_trust_ratios
                store_release(&ready[ch_s.tensor], pack_ratio(epoch, eta));
            }
        }
    }
    if (!has_u) return;

    // ---- U part: phases 9-10 over an earlier item, stretched by its tensor's ratio.
    // Lane 0 of every warp polls; the warp goes on as soon as it has the ratio.
    if (!has_s) r_u = recs[ch_u.tensor];
    if ((threadIdx.x & 31u) == 0u) {
        if (static_cast<unsigned>(word >> 32) != epoch)
            word = wait_for_ratio(&ready[ch_u.tensor], epoch, &ctl->error);
        if (word == 0ull) {
            atomicExch(&ctl->error, 1u);
            *reinterpret_cast<volatile unsigned *>(host_error) = 1u;
        }
    }
    __syncwarp();                        // lane 0's acquire orders the whole warp's loads below
    word = __shfl_sync(0xffffffffu, word, 0);
    if (word == 0ull) return;            // (the update below has no CTA-wide barrier)
    const float step = step_all * __uint_as_float(static_cast<unsigned>(word));    // Eq. 24a
    entry_apply<LA, PRE>(ch_u, r_u, direction + static_cast<size_t>(c_u) * static_cast<size_t>(slot_elems),
                         s, step);
}

template <int NEST, int GT, int PRE>
void *pick_adapt_la(int la)
{
    switch (la) {
#define NOVAK_LA_CASE(X) case (X): return reinterpret_cast<void *>(novak_step_adapt_kernel<NEST, GT, (X), PRE>);
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
void *pick_adapt_gt(int grad_dtype, int la)
{
    switch (grad_dtype) {
    case NOVAK_GRAD_F32: return pick_adapt_la<NEST, NOVAK_GRAD_F32, PRE>(la);
    case NOVAK_GRAD_BF16: return pick_adapt_la<NEST, NOVAK_GRAD_BF16, PRE>(la);
    default: return nullptr;
    }
}

// Every instantiation for one mode (PRE_NONE, PRE_SCALE or PRE_CENTER, with or without
// PRE_COPY16 and PRE_MOM16).
template <int PRE>
void *pick_step_adapt_kernel(int nesterov, int grad_dtype, int la)
{
    switch (nesterov) {
    case NOVAK_NESTEROV_NONE: return pick_adapt_gt<NOVAK_NESTEROV_NONE, PRE>(grad_dtype, la);
    case NOVAK_NESTEROV_APPROX: return pick_adapt_gt<NOVAK_NESTEROV_APPROX, PRE>(grad_dtype, la);
    case NOVAK_NESTEROV_CLASSICAL: return pick_adapt_gt<NOVAK_NESTEROV_CLASSICAL, PRE>(grad_dtype, la);
    default: return nullptr;
    }
}

}  // namespace
}  // namespace novak
