// Layer-wise adaptation (Eq. 19 / 25) and the step in ONE launch for sm_100a.
//
// The trust ratio of a tensor needs ||u_t|| over the whole tensor before any of
// its elements moves, so theta, g, m, v of a tensor are needed twice.  Run as
// two passes over the whole group (novak_trust_stats.cu, then the step kernel)
// the second pass finds nothing of the first in L2: 16 + 28 B per element from
// DRAM.  Here both passes are ITEMS of one grid, one item per CTA: S items (the
// two sums of squares of one chunk-table entry, loads that stay in L2) and U
// items (the ordinary step over one entry, streaming loads), in an order in
// which the statistics run a fixed number of items ahead of the updates:
//
//     S(T0) S(T1) ... | U(T0) S(Tk) U(T1) S(Tk+1) ...        (whole tensors)
//
// so that a tensor's update follows its statistics by a few tens of MB of
// traffic, while its 16 B per element are still in the 126 MB L2.  CTA number b
// takes item number b.  The CTA that completes a tensor's last S item adds the
// tensor's sums in table order (fixed order: bit-identical from run to run) and
// publishes the ratio as one 64-bit word (launch number, ratio); a U item waits
// for its tensor's word, every warp polling for itself (no CTA-wide barrier on
// the way to the first load).
//
// The wait and forward progress: a U item waits only for S items that stand
// earlier in the order.  The hardware hands out the CTAs of a grid in
// increasing block index as slots become free (the behaviour single-pass scans
// with look-back rely on as well), so those S items belong to CTAs that are
// running or have finished, and S items never wait; with the lead between S
// and U the ratio is normally there long before it is asked for.  Nothing in
// the programming model promises that order, so the wait is bounded: after
// about two seconds (at once, when another CTA has already given up) a warp
// gives up, raises an error flag in host-mapped memory, leaves its part of the
// entry untouched and returns; the next call on the handle reports it, and
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

// Resident CTAs per SM as for the plain step kernel's instantiation of the same
// lookahead action (three for every action measured 0.233 against 0.220 ms per
// step on the ResNet-50-shaped set).
#ifndef NOVAK_ADAPT_MIN_CTAS
#define NOVAK_ADAPT_MIN_CTAS step_min_ctas(LA)
#endif
template <int NEST, int GT, int LA, int PRE>
__global__ void __launch_bounds__(NOVAK_BLOCK, NOVAK_ADAPT_MIN_CTAS)
novak_step_adapt_kernel(const int *__restrict__ item_code, const Chunk *__restrict__ item_chunk,
                        int n_items, const TensorRec *__restrict__ recs,
                        const int *__restrict__ tensor_first, double *chunk_u2, double *chunk_p2,
                        float *trust, AdaptCtl *ctl, unsigned *arrived, unsigned long long *ready,
                        unsigned *host_error, const StepScalars s, unsigned epoch)
{
    static_assert((PRE & PRE_MASK) == PRE_NONE, "gradient pre-processing keeps the two-pass route");
    // the classical blend (Eq. 16) comes after the base direction
    constexpr int kStatNest = (NEST == NOVAK_NESTEROV_APPROX) ? NOVAK_NESTEROV_APPROX
                                                              : NOVAK_NESTEROV_NONE;
    __shared__ double sh[kTrustWarps];
    __shared__ int sh_flag;

    grid_dependency_release();
    const int it = blockIdx.x;
    if (it >= n_items) return;
    // The item tables and the records are written by copies only, never by a
    // kernel: read before the previous kernel on the stream has finished.
    const int code = item_code[it];
    const Chunk ch = item_chunk[it];
    const int c = code & 0x7fffffff;                    // the entry's index in the chunk table
    const TensorRec r = recs[ch.tensor];
    grid_dependency_wait();

    PreArgs pre;
    pre.factor = 1.0f;
    pre.mean = nullptr;
    pre.row_len = 0u;
    pre.elem0 = static_cast<uint32_t>(ch.offset);

    if (code >= 0) {
        // ---- S item: this entry's two sums of squares
        const int c0 = tensor_first[ch.tensor], c1 = tensor_first[ch.tensor + 1];
        pre.step = 0.0f;
        pre.copy = nullptr;
        double tp, tu;
        entry_trust_sums<kStatNest, GT, PRE, LD_KEEP>(ch, r, s, pre, sh, tp, tu);
        if (threadIdx.x == 0) {
            chunk_p2[c] = tp;
            chunk_u2[c] = tu;
            __threadfence();                 // the sums before the arrival
            const unsigned last = static_cast<unsigned>(c1 - c0) - 1u;
            // wraps to 0 with the tensor's last entry, ready for the next launch
            sh_flag = atomicInc(&arrived[ch.tensor], last) == last ? 1 : 0;
        }
        __syncthreads();
        if (sh_flag == 0) return;
        // the tensor's last entry: every sum is there
        __threadfence();
        const float eta = tensor_trust_ratio(chunk_p2, chunk_u2, c0, c1, sh);
        if (threadIdx.x == 0) {
            trust[ch.tensor] = eta;          // for novak_get_trust_ratios
            store_release(&ready[ch.tensor], pack_ratio(epoch, eta));
        }
        return;
    }

    // ---- U item: the ordinary step over this entry, stretched by the tensor's ratio.
    // Lane 0 of every warp polls; the warp goes on as soon as it has the ratio.
    unsigned long long word = 0ull;
    if ((threadIdx.x & 31u) == 0u) {
        word = wait_for_ratio(&ready[ch.tensor], epoch, &ctl->error);
        if (word == 0ull) {
            atomicExch(&ctl->error, 1u);
            *reinterpret_cast<volatile unsigned *>(host_error) = 1u;
        }
    }
    word = __shfl_sync(0xffffffffu, word, 0);
    if (word == 0ull) return;            // (the update below has no CTA-wide barrier)
    pre.step = s.step * __uint_as_float(static_cast<unsigned>(word));      // Eq. 24a
    pre.copy = ((PRE & PRE_COPY16) != 0) ? r.p16 + ch.offset : nullptr;
    run_entry<NEST, GT, LA, PRE>(ch, r, s, pre);
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

// Every instantiation for one mode (PRE_NONE with or without PRE_COPY16 and PRE_MOM16).
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
