// Gradient statistics pass of phase 2 (Section 5.1, Table 2; Section 5.8) for
// sm_100a: ONE read of the gradient produces
//   - the global L2 norm of the raw gradient over every tensor of the group and
//     the clip factor c_clip/||g|| (1 when ||g|| <= c_clip), and
//   - for tensors that have rows, the mean of every row (Eq. 26: the mean over
//     dimensions 1..d for each index of dimension 0).
// Both stay in device memory; the step kernel that follows on the stream reads
// them there, so the host never waits for a reduction.
//
// Decomposition: one CTA per 4 consecutive chunk-table entries (the table of the
// step kernel); per entry when row means are wanted.
// All sums are carried in double precision and combined in a fixed order (warp
// shuffle tree, then warps in index order, then chunks in index order), so the
// result is bit-identical from run to run; there are no floating-point atomics.
// A row that spans several entries leaves one partial sum per entry; a second,
// small kernel (one thread per entry) adds those up in entry order and reduces
// the per-entry sums of squares; its last CTA (an integer ticket counter)
// writes the norm and the clip factor.  Nothing spins: every CTA does a bounded
// amount of work and returns.
//
// Row means need chunk-table entries of at most 2048 elements (the host checks).
#include "novak_internal.h"

#include "novak.h"

namespace novak {
namespace {

constexpr int kStatsBlock = 256;
constexpr int kStatsWarps = kStatsBlock / 32;

__device__ __forceinline__ void grid_dependency_release()
{
    asm volatile("griddepcontrol.launch_dependents;");
}
__device__ __forceinline__ void grid_dependency_wait()
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

// Gradient element i of a tensor as fp32 (bf16 widens exactly).  Default cache
// policy: the step kernel reads the same bytes next, and a gradient of up to
// ~100 MB is still in L2 then.
template <int GT>
__device__ __forceinline__ float grad_at(const void *g, uint32_t i)
{
    if constexpr (GT == NOVAK_GRAD_F32) {
        return __ldg(static_cast<const float *>(g) + i);
    } else {
        const unsigned short t = __ldg(static_cast<const unsigned short *>(g) + i);
        return __uint_as_float(static_cast<unsigned>(t) << 16);
    }
}

// Sum over the warp in a fixed tree order; lane 0 holds the total.
__device__ __forceinline__ double warp_sum(double x)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_down_sync(0xffffffffu, x, o);
    return x;
}

// Sum over the CTA (warps in index order); thread 0 holds the total.
__device__ __forceinline__ double block_sum(double x, double *sh)
{
    x = warp_sum(x);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    __syncthreads();                 // sh may still be read from an earlier call
    if (lane == 0) sh[warp] = x;
    __syncthreads();
    double t = 0.0;
    if (threadIdx.x == 0) {
#pragma unroll
        for (int w = 0; w < kStatsWarps; ++w) t += sh[w];
    }
    return t;
}

// Largest chunk-table entry the row-mean path handles: one shared-memory slot
// per 4-element vector, two vectors per thread.
constexpr int kStatsMaxChunk = 2048;
constexpr int kStatsMaxVec = kStatsMaxChunk / 4;

// Up to 4 consecutive gradient elements starting at element `i` of `g` (which
// points at the entry's first element), as fp32; n < 4 at a tensor's end (the
// rest reads as 0), n = 0 loads nothing.
template <int GT>
__device__ __forceinline__ void load_quad(const void *g, bool aligned, uint32_t i, uint32_t n,
                                          float (&x)[4])
{
    if (aligned && n == 4u) {
        if constexpr (GT == NOVAK_GRAD_F32) {
            const float4 t = __ldg(reinterpret_cast<const float4 *>(
                static_cast<const float *>(g) + i));
            x[0] = t.x; x[1] = t.y; x[2] = t.z; x[3] = t.w;
        } else {
            const uint2 t = __ldg(reinterpret_cast<const uint2 *>(
                static_cast<const unsigned short *>(g) + i));
            x[0] = __uint_as_float(t.x << 16);
            x[1] = __uint_as_float(t.x & 0xffff0000u);
            x[2] = __uint_as_float(t.y << 16);
            x[3] = __uint_as_float(t.y & 0xffff0000u);
        }
    } else {
#pragma unroll
        for (uint32_t j = 0; j < 4u; ++j) x[j] = (j < n) ? grad_at<GT>(g, i + j) : 0.0f;
    }
}

// Four squares are added in fp32 (relative rounding error ~1e-7 on a sum of
// positive terms, unbiased), everything beyond that in double.
__device__ __forceinline__ double sum_squares(const float (&x)[4], double sq)
{
    float s = x[0] * x[0];
    s = fmaf(x[1], x[1], s);
    s = fmaf(x[2], x[2], s);
    s = fmaf(x[3], x[3], s);
    return sq + double(s);
}

// Splits a vector's sum at the end of the row of its first element, which sits
// `rem` elements into a row of length L >= 4 (a vector touches at most two
// rows).  Row sums are carried in double from the first addition on: an
// absolute error in a row mean becomes an absolute error in every centred
// gradient of the row, and the update direction m^/(sqrt(v^)+eps) amplifies
// such an error by up to 1/eps where the centred gradient is below eps.
__device__ __forceinline__ void split_at_row_end(const float (&x)[4], uint32_t rem, uint32_t L,
                                                 double *lo, double *hi)
{
    const uint32_t left = L - rem;                         // elements up to the row's end
    double a = 0.0, b = 0.0;
#pragma unroll
    for (uint32_t j = 0; j < 4u; ++j) {
        if (j < left) a += double(x[j]); else b += double(x[j]);
    }
    *lo = a;
    *hi = b;
}

// A row mean as an unevaluated sum of two floats (hi + lo carries ~48 bits).
__device__ __forceinline__ float2 split_mean(double sum, uint32_t L)
{
    const double mu = sum / double(L);
    const float hi = static_cast<float>(mu);
    return make_float2(hi, static_cast<float>(mu - double(hi)));
}

// Entries one CTA of the first kernel takes (consecutive in the table).  All
// their table reads, then all their gradient loads, are issued together, so a
// CTA pays the table -> record -> data latency chain once per 32 KB, not per 8 KB.
#ifndef NOVAK_STATS_ROWS_ENTRIES
#define NOVAK_STATS_ROWS_ENTRIES 1
#endif
constexpr int kStatsEntries = 4;                          // no tensor has rows
constexpr int kStatsEntriesRows = NOVAK_STATS_ROWS_ENTRIES;   // row means: more registers per entry

// Sums of one row piece [s0, s1) of `row`, to the row mean if the piece is the
// whole row, else to the entry's first / last partial sum.
__device__ __forceinline__ void store_row_piece(const TensorRec &rec, uint32_t row, uint32_t r0,
                                                bool whole, double sum, uint32_t L,
                                                double *seg_first, double *seg_last, int c)
{
    if (whole)
        rec.mean[row] = split_mean(sum, L);   // whole row inside the entry
    else if (row == r0)
        seg_first[c] = sum;     // row began before this entry, or runs past it
    else
        seg_last[c] = sum;      // last row of the entry, continues in the next
}

template <int GT, bool ROWS>
__global__ void __launch_bounds__(kStatsBlock)
novak_grad_stats_kernel(const Chunk *__restrict__ chunks, int n_chunks,
                        const TensorRec *__restrict__ recs,
                        double *__restrict__ chunk_sq, double *__restrict__ seg_first,
                        double *__restrict__ seg_last)
{
    __shared__ double sh[kStatsWarps];
    // per 4-element vector of an entry: the sum of the elements that belong to
    // the row of its first element, and of those already in the next row
    __shared__ double vec_lo[ROWS ? kStatsMaxVec : 1];
    __shared__ double vec_hi[ROWS ? kStatsMaxVec : 1];
    constexpr uint32_t kElemBytes = (GT == NOVAK_GRAD_BF16) ? 2u : 4u;
    constexpr int K = ROWS ? kStatsEntriesRows : kStatsEntries;

    grid_dependency_release();
    const int c0 = blockIdx.x * K;
    Chunk ch[K];
    TensorRec rec[K];
#pragma unroll
    for (int k = 0; k < K; ++k) ch[k] = chunks[min(c0 + k, n_chunks - 1)];
#pragma unroll
    for (int k = 0; k < K; ++k) rec[k] = recs[ch[k].tensor];
    grid_dependency_wait();          // the gradient may come from the previous kernel

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const void *g[K];
    bool aligned[K], fast[K];
    uint32_t ia[K], ib[K], na[K], nb[K];
    float xa[K][4], xb[K][4];
    // ---- every entry's first two vectors per thread, all loads in flight at once
#pragma unroll
    for (int k = 0; k < K; ++k) {
        const uintptr_t addr = reinterpret_cast<uintptr_t>(rec[k].g) +
                               static_cast<uintptr_t>(ch[k].offset) * kElemBytes;
        g[k] = reinterpret_cast<const void *>(addr);          // the entry's first element
        aligned[k] = (addr & (4u * kElemBytes - 1u)) == 0;
        const uint32_t len = static_cast<uint32_t>(ch[k].len);
        const bool short_rows = ROWS && rec[k].mean != nullptr && rec[k].row_len < 4u;
        fast[k] = (c0 + k < n_chunks) && !short_rows;
        const uint32_t nvec = (len + 3u) >> 2;
        const uint32_t va = threadIdx.x, vb = va + kStatsBlock;
        ia[k] = va << 2;
        ib[k] = vb << 2;
        na[k] = (fast[k] && va < nvec) ? (len - ia[k] < 4u ? len - ia[k] : 4u) : 0u;
        nb[k] = (fast[k] && vb < nvec) ? (len - ib[k] < 4u ? len - ib[k] : 4u) : 0u;
        load_quad<GT>(g[k], aligned[k], ia[k], na[k], xa[k]);
        load_quad<GT>(g[k], aligned[k], ib[k], nb[k], xb[k]);
    }

    double sq = 0.0;
#pragma unroll
    for (int k = 0; k < K; ++k) {
        if (c0 + k >= n_chunks) break;
        const int c = c0 + k;
        const uint32_t len = static_cast<uint32_t>(ch[k].len);
        const bool rows = ROWS && rec[k].mean != nullptr;
        const uint32_t L = rec[k].row_len;
        const uint32_t off = static_cast<uint32_t>(ch[k].offset);   // used with rows only (< 2^31)
        const uint32_t end = off + len;

        if (rows && L < 4u) {
            // ---- rows of 1 to 3 elements: a thread per row, straight from global memory
            const uint32_t r0 = off / L, r1 = (end - 1u) / L;
            for (uint32_t row = r0 + threadIdx.x; row <= r1; row += kStatsBlock) {
                const uint32_t row_begin = row * L, row_end = row_begin + L;
                const uint32_t s0 = row_begin > off ? row_begin : off;
                const uint32_t s1 = row_end < end ? row_end : end;
                double sum = 0.0;
                for (uint32_t e = s0; e < s1; ++e) {
                    const float x = grad_at<GT>(rec[k].g, e);
                    sum += double(x);
                    sq = fma(double(x), double(x), sq);
                }
                store_row_piece(rec[k], row, r0, s0 == row_begin && s1 == row_end, sum, L,
                                seg_first, seg_last, c);
            }
            continue;
        }

        // ---- pass 1: squares of the vectors already loaded and, for a tensor with
        // rows, each vector's sum split at the row boundary
        sq = sum_squares(xa[k], sq);
        sq = sum_squares(xb[k], sq);
        if (rows) {                     // entries of tensors with rows have at most 512 vectors
            // where in its row each of this thread's two vectors starts: one division,
            // the second vector lies 4 x 256 elements further on
            const uint32_t ea = off + ia[k];
            const uint32_t rem_a = ea - (ea / L) * L;
            uint32_t rem_b = rem_a + 4u * kStatsBlock;
            if (rem_b >= L) rem_b = (L >= 4u * kStatsBlock) ? rem_b - L : rem_b % L;
            if (na[k]) split_at_row_end(xa[k], rem_a, L, &vec_lo[threadIdx.x], &vec_hi[threadIdx.x]);
            if (nb[k]) split_at_row_end(xb[k], rem_b, L, &vec_lo[threadIdx.x + kStatsBlock],
                                        &vec_hi[threadIdx.x + kStatsBlock]);
        } else {
            // entries longer than 2048 elements (no rows): the rest of the vectors
            const uint32_t nvec = (len + 3u) >> 2;
            for (uint32_t v = threadIdx.x + 2u * kStatsBlock; v < nvec; v += kStatsBlock) {
                float x[4];
                const uint32_t i = v << 2;
                load_quad<GT>(g[k], aligned[k], i, len - i < 4u ? len - i : 4u, x);
                sq = sum_squares(x, sq);
            }
        }
        if (rows) {
            // ---- pass 2: the pieces of rows inside this entry, summed in vector
            // order.  Rows of 128 elements or more take a warp each, shorter ones
            // a thread each.
            __syncthreads();
            const uint32_t r0 = off / L, r1 = (end - 1u) / L;
            const bool by_warp = L >= 128u;
            const uint32_t first = by_warp ? warp : threadIdx.x;
            const uint32_t stride = by_warp ? kStatsWarps : kStatsBlock;
            for (uint32_t row = r0 + first; row <= r1; row += stride) {
                const uint32_t row_begin = row * L, row_end = row_begin + L;
                const uint32_t s0 = row_begin > off ? row_begin : off;
                const uint32_t s1 = row_end < end ? row_end : end;
                const uint32_t vb = (s0 - off + 3u) >> 2, ve = (s1 - off + 3u) >> 2;
                double sum = 0.0;
                if (by_warp) {
                    for (uint32_t v = vb + lane; v < ve; v += 32u) sum += vec_lo[v];
                    sum = warp_sum(sum);
                } else {
                    for (uint32_t v = vb; v < ve; ++v) sum += vec_lo[v];
                }
                if (!by_warp || lane == 0) {
                    if (((s0 - off) & 3u) != 0u) sum += vec_hi[vb - 1u];   // row starts mid-vector
                    store_row_piece(rec[k], row, r0, s0 == row_begin && s1 == row_end, sum, L,
                                    seg_first, seg_last, c);
                }
            }
            __syncthreads();            // the slots are reused by the next entry
        }
    }

    // one sum of squares per CTA, filed under its first entry
    const double total = block_sum(sq, sh);
    if (threadIdx.x == 0) {
        chunk_sq[c0] = total;
#pragma unroll
        for (int k = 1; k < K; ++k)
            if (c0 + k < n_chunks) chunk_sq[c0 + k] = 0.0;
    }
}

// Sum of squares of the parameters (for ||theta_t|| of Eq. 21): one CTA per 4
// chunk-table entries, one sum per CTA filed under its first entry.  Launched
// only when the automatic learning-rate scaling is on.
__global__ void __launch_bounds__(kStatsBlock)
novak_param_sumsq_kernel(const Chunk *__restrict__ chunks, int n_chunks,
                         const TensorRec *__restrict__ recs, double *__restrict__ chunk_psq)
{
    __shared__ double sh[kStatsWarps];
    constexpr int K = kStatsEntries;
    grid_dependency_release();
    const int c0 = blockIdx.x * K;
    Chunk ch[K];
    const float *p[K];
#pragma unroll
    for (int k = 0; k < K; ++k) ch[k] = chunks[min(c0 + k, n_chunks - 1)];
#pragma unroll
    for (int k = 0; k < K; ++k) p[k] = recs[ch[k].tensor].p + ch[k].offset;
    grid_dependency_wait();          // the parameters come from the previous step
    double sq = 0.0;
#pragma unroll
    for (int k = 0; k < K; ++k) {
        if (c0 + k >= n_chunks) break;
        const uint32_t len = static_cast<uint32_t>(ch[k].len);
        const bool aligned = (reinterpret_cast<uintptr_t>(p[k]) & 15u) == 0;
        const uint32_t nvec = (len + 3u) >> 2;
        for (uint32_t v = threadIdx.x; v < nvec; v += kStatsBlock) {
            float x[4];
            const uint32_t i = v << 2;
            load_quad<NOVAK_GRAD_F32>(p[k], aligned, i, len - i < 4u ? len - i : 4u, x);
            sq = sum_squares(x, sq);
        }
    }
    const double total = block_sum(sq, sh);
    if (threadIdx.x == 0) {
        chunk_psq[c0] = total;
#pragma unroll
        for (int k = 1; k < K; ++k)
            if (c0 + k < n_chunks) chunk_psq[c0 + k] = 0.0;
    }
}

// Second kernel of the pass, one THREAD per chunk-table entry: puts together the
// rows that entry boundaries cut (the thread of the entry in which such a row
// BEGINS adds the pieces in entry order; the table lists a tensor's entries
// consecutively, in element order), and sums the entries' sums of squares: per
// CTA first, then the CTA that takes the last ticket adds the CTAs' sums in
// index order and writes the norm and the clip factor.
template <bool ROWS>
__global__ void __launch_bounds__(kStatsBlock)
novak_grad_stats_finish_kernel(const Chunk *__restrict__ chunks, int n_chunks,
                               const TensorRec *__restrict__ recs, double c_clip,
                               double auto_gamma, const double *__restrict__ chunk_sq,
                               const double *__restrict__ chunk_psq,
                               const double *__restrict__ seg_first,
                               const double *__restrict__ seg_last,
                               double *__restrict__ cta_sq, PrepOut *__restrict__ out)
{
    __shared__ double sh[kStatsWarps];
    __shared__ unsigned sh_last;

    grid_dependency_release();
    grid_dependency_wait();          // everything below is the first kernel's output
    const int i = blockIdx.x * kStatsBlock + threadIdx.x;
    double sq = 0.0, psq = 0.0;
    if (i < n_chunks) {
        sq = chunk_sq[i];
        if (chunk_psq != nullptr) psq = chunk_psq[i];
        if constexpr (ROWS) {
            const Chunk ci = chunks[i];
            const TensorRec ri = recs[ci.tensor];
            if (ri.mean != nullptr) {
                const uint32_t L = ri.row_len;
                const uint32_t o = static_cast<uint32_t>(ci.offset);
                const uint32_t e = o + static_cast<uint32_t>(ci.len);
                const uint32_t row = (e - 1u) / L;
                const uint32_t row_begin = row * L, row_end = row_begin + L;
                // the entry's last row runs past it, and began inside it
                if (row_end > e && row_begin >= o) {
                    double sum = (row == o / L) ? seg_first[i] : seg_last[i];
                    for (int j = i + 1; j < n_chunks; ++j) {
                        const Chunk cj = chunks[j];
                        if (cj.tensor != ci.tensor) break;
                        sum += seg_first[j];
                        if (static_cast<uint32_t>(cj.offset) + static_cast<uint32_t>(cj.len) >= row_end)
                            break;
                    }
                    ri.mean[row] = split_mean(sum, L);
                }
            }
        }
    }
    const double total = block_sum(sq, sh);
    const double ptotal = chunk_psq != nullptr ? block_sum(psq, sh) : 0.0;
    if (threadIdx.x == 0) {
        cta_sq[blockIdx.x] = total;
        if (chunk_psq != nullptr) cta_sq[gridDim.x + blockIdx.x] = ptotal;
        __threadfence();             // this CTA's sums before its ticket
        // wraps to 0 after the last CTA, ready for the next launch
        const unsigned ticket = atomicInc(&out->ticket, static_cast<unsigned>(gridDim.x) - 1u);
        sh_last = (ticket == static_cast<unsigned>(gridDim.x) - 1u) ? 1u : 0u;
    }
    __syncthreads();
    if (sh_last == 0u) return;

    // ---- the CTA that finished last: every CTA's sum is complete
    __threadfence();
    double t = 0.0, tp = 0.0;
    for (unsigned b = threadIdx.x; b < gridDim.x; b += kStatsBlock) {
        t += __ldcg(cta_sq + b);
        if (chunk_psq != nullptr) tp += __ldcg(cta_sq + gridDim.x + b);
    }
    const double sumsq = block_sum(t, sh);
    const double psumsq = chunk_psq != nullptr ? block_sum(tp, sh) : 0.0;
    if (threadIdx.x == 0) {
        const double norm = sqrt(sumsq);
        // Table 2: clipping is active when ||g|| > c_clip
        const double factor = (c_clip > 0.0 && norm > c_clip) ? c_clip / norm : 1.0;
        out->norm = norm;
        out->factor = static_cast<float>(factor);
        float scale = 1.0f;
        if (chunk_psq != nullptr && auto_gamma > 0.0) {
            // Eq. 20-22 on the norm of the gradient as given and of theta_t
            const double pnorm = sqrt(psumsq);
            const double g_bar = auto_gamma * norm + (1.0 - auto_gamma) * out->g_bar;
            const double theta_bar = auto_gamma * pnorm + (1.0 - auto_gamma) * out->theta_bar;
            double a = 1.0;              // 0/0: undefined, taken as 1
            if (!(g_bar == 0.0 && theta_bar == 0.0)) {
                a = g_bar / theta_bar;
                a = a < 0.1 ? 0.1 : (a > 2.0 ? 2.0 : a);
            }
            out->pnorm = pnorm;
            out->g_bar = g_bar;
            out->theta_bar = theta_bar;
            scale = static_cast<float>(a);
        }
        out->auto_scale = scale;
    }
}

}  // namespace

namespace {

cudaError_t launch_pdl(const void *fn, unsigned grid, void **args, bool pdl, cudaStream_t stream)
{
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(grid);
    lc.blockDim = dim3(kStatsBlock);
    lc.dynamicSmemBytes = 0;
    lc.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelExC(&lc, fn, args);
}

}  // namespace

int grad_stats_ctas(int n_chunks) { return (n_chunks + kStatsBlock - 1) / kStatsBlock; }

cudaError_t launch_grad_stats(const Chunk *d_chunks, int n_chunks, const TensorRec *d_recs,
                              int grad_dtype, double c_clip, double auto_gamma, double *chunk_sq,
                              double *chunk_psq, double *seg_first, double *seg_last,
                              double *cta_sq, PrepOut *prep, bool any_rows, int pdl,
                              cudaStream_t stream)
{
    if (auto_gamma > 0.0 && !chunk_psq) return cudaErrorInvalidValue;
    if (n_chunks <= 0 || !d_chunks || !d_recs || !chunk_sq || !cta_sq || !prep)
        return cudaErrorInvalidValue;
    if (any_rows && (!seg_first || !seg_last)) return cudaErrorInvalidValue;
    const void *first = nullptr;
    switch (grad_dtype) {
    case NOVAK_GRAD_F32:
        first = any_rows ? reinterpret_cast<const void *>(novak_grad_stats_kernel<NOVAK_GRAD_F32, true>)
                         : reinterpret_cast<const void *>(novak_grad_stats_kernel<NOVAK_GRAD_F32, false>);
        break;
    case NOVAK_GRAD_BF16:
        first = any_rows ? reinterpret_cast<const void *>(novak_grad_stats_kernel<NOVAK_GRAD_BF16, true>)
                         : reinterpret_cast<const void *>(novak_grad_stats_kernel<NOVAK_GRAD_BF16, false>);
        break;
    default: return cudaErrorInvalidValue;
    }
    const void *second = any_rows ? reinterpret_cast<const void *>(novak_grad_stats_finish_kernel<true>)
                                  : reinterpret_cast<const void *>(novak_grad_stats_finish_kernel<false>);
    void *args1[] = {&d_chunks, &n_chunks, &d_recs, &chunk_sq, &seg_first, &seg_last};
    const int per_cta = any_rows ? kStatsEntriesRows : kStatsEntries;
    const unsigned grid1 = static_cast<unsigned>((n_chunks + per_cta - 1) / per_cta);
    cudaError_t e = launch_pdl(first, grid1, args1, (pdl & 2) != 0, stream);
    if (e != cudaSuccess) return e;
    const double *c_psq = nullptr;
    if (auto_gamma > 0.0) {
        void *args_p[] = {&d_chunks, &n_chunks, &d_recs, &chunk_psq};
        const unsigned grid_p = static_cast<unsigned>((n_chunks + kStatsEntries - 1) / kStatsEntries);
        e = launch_pdl(reinterpret_cast<const void *>(novak_param_sumsq_kernel), grid_p, args_p,
                       (pdl & 2) != 0, stream);
        if (e != cudaSuccess) return e;
        c_psq = chunk_psq;
    }
    const double *c_sq = chunk_sq, *c_first = seg_first, *c_last = seg_last;
    void *args2[] = {&d_chunks, &n_chunks, &d_recs, &c_clip, &auto_gamma, &c_sq, &c_psq,
                     &c_first, &c_last, &cta_sq, &prep};
    return launch_pdl(second, static_cast<unsigned>(grad_stats_ctas(n_chunks)), args2, (pdl & 4) != 0, stream);
}

}  // namespace novak
