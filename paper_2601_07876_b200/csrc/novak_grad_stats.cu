// Gradient statistics pass of phase 2 (Section 5.1, Table 2; Section 5.8) for
// sm_100a: ONE read of the gradient produces
//   - the global L2 norm of the raw gradient over every tensor of the group and
//     the clip factor c_clip/||g|| (1 when ||g|| <= c_clip), and
//   - for tensors that have rows, the mean of every row (Eq. 26: the mean over
//     dimensions 1..d for each index of dimension 0).
// Both stay in device memory; the step kernel that follows on the stream reads
// them there, so the host never waits for a reduction.
//
// Decomposition.  Tensors without rows: one CTA per 4 consecutive chunk-table
// entries (the table of the step kernel), sum of squares only.  Tensors with
// rows: a table of row units built on the host, aligned to ROWS, not to the
// chunk table: a unit is a group of whole rows of up to 8192 elements (a warp
// streams each row; half a warp for rows of up to 1024 elements, eight lanes
// below 128, a thread below 32), or a slice of at most 16384 elements of a
// longer row (the whole CTA).  No shared-memory
// staging, no per-vector row arithmetic: a lane only ever adds along one row.
// All sums are carried in double precision and combined in a fixed order (per
// lane, warp shuffle tree, warps in index order, CTAs in index order), so the
// result is bit-identical from run to run; there are no floating-point atomics.
// A second, small kernel adds the slices of long rows in order and reduces the
// CTAs' sums of squares; its last CTA (an integer ticket counter) writes the
// norm and the clip factor.  Nothing spins: every CTA does a bounded amount of
// work and returns.
#include "novak_internal.h"

#include "novak.h"

namespace novak {
namespace {

// Resident CTAs per SM the first kernel of the pass is compiled for.
#ifndef NOVAK_STATS_MIN_CTAS
#define NOVAK_STATS_MIN_CTAS 6
#endif

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

// Up to 4 consecutive gradient elements starting at element `i` of `g`, as
// fp32; n < 4 at a ragged end (the rest reads as 0), n = 0 loads nothing.
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

// Row sums are carried in double from the first addition on: an absolute error
// in a row mean becomes an absolute error in every centred gradient of the row,
// and the update direction m^/(sqrt(v^)+eps) amplifies such an error by up to
// 1/eps where the centred gradient is below eps.
__device__ __forceinline__ double sum_four(const float (&x)[4], double sum)
{
    return sum + ((double(x[0]) + double(x[1])) + (double(x[2]) + double(x[3])));
}

// A row mean as an unevaluated sum of two floats (hi + lo carries ~48 bits).
__device__ __forceinline__ float2 split_mean(double sum, uint32_t L)
{
    const double mu = sum / double(L);
    const float hi = static_cast<float>(mu);
    return make_float2(hi, static_cast<float>(mu - double(hi)));
}

// Chunk-table entries one CTA of the plain path takes (consecutive in the
// list).  All their table reads, then all their gradient loads, are issued
// together, so a CTA pays the table -> record -> data latency chain once per
// 32 KB, not per 8 KB.
constexpr int kStatsEntries = 4;

// Entries per CTA of the plain path: bf16 entries are half as many bytes, so a
// CTA takes twice as many (with 128-bit loads) to keep the same bytes in
// flight.  Where row units share the kernel the plain entries are the small
// tensors only, and the lean generic path keeps the registers for the rows.
template <int GT, bool ROWS>
struct PlainEntries {
    static constexpr bool wide = (GT == NOVAK_GRAD_BF16) && !ROWS;
    static constexpr int value = wide ? 2 * kStatsEntries : kStatsEntries;
};

// Squares of 8 bf16 values packed in 16 bytes.
__device__ __forceinline__ double sum_squares_bf16x8(const uint4 t, double sq)
{
    const unsigned w[4] = {t.x, t.y, t.z, t.w};
    float s = 0.0f;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const float lo = __uint_as_float(w[j] << 16), hi = __uint_as_float(w[j] & 0xffff0000u);
        s = fmaf(lo, lo, s);
        s = fmaf(hi, hi, s);
    }
    return sq + double(s);
}

// ---- tensors without rows, bf16 gradients: 8 consecutive entries, 128-bit loads
__device__ __forceinline__ double plain_entries_bf16(const Chunk *__restrict__ plain, int n_plain,
                                                     const TensorRec *__restrict__ recs, int c0)
{
    constexpr int K = PlainEntries<NOVAK_GRAD_BF16, false>::value;
    Chunk ch[K];
    const void *base[K];
#pragma unroll
    for (int k = 0; k < K; ++k) ch[k] = plain[min(c0 + k, n_plain - 1)];
#pragma unroll
    for (int k = 0; k < K; ++k) base[k] = recs[ch[k].tensor].g;
    grid_dependency_wait();          // the gradient may come from the previous kernel

    const unsigned short *g[K];
    bool wide[K];
    uint4 x[K];
    // one 16-byte vector (8 elements) per thread and entry, all loads in flight at once
#pragma unroll
    for (int k = 0; k < K; ++k) {
        g[k] = static_cast<const unsigned short *>(base[k]) + ch[k].offset;
        const uint32_t len = (c0 + k < n_plain) ? static_cast<uint32_t>(ch[k].len) : 0u;
        wide[k] = (reinterpret_cast<uintptr_t>(g[k]) & 15u) == 0;
        x[k] = make_uint4(0u, 0u, 0u, 0u);
        if (wide[k] && (threadIdx.x + 1u) * 8u <= len)
            x[k] = __ldg(reinterpret_cast<const uint4 *>(g[k]) + threadIdx.x);
    }
    double sq = 0.0;
#pragma unroll
    for (int k = 0; k < K; ++k) {
        if (c0 + k >= n_plain) break;
        sq = sum_squares_bf16x8(x[k], sq);
        // what the one vector per thread did not cover: an unaligned entry, a ragged
        // end, or an entry longer than 2048 elements
        const uint32_t len = static_cast<uint32_t>(ch[k].len);
        const uint32_t done = wide[k] ? min(len & ~7u, 8u * kStatsBlock) : 0u;
        for (uint32_t e = done + threadIdx.x; e < len; e += kStatsBlock) {
            const float v = grad_at<NOVAK_GRAD_BF16>(g[k], e);
            sq = fma(double(v), double(v), sq);
        }
    }
    return sq;
}

// ---- tensors without rows: the sum of squares of 4 consecutive entries
template <int GT, bool WIDE>
__device__ __forceinline__ double plain_entries(const Chunk *__restrict__ plain, int n_plain,
                                                const TensorRec *__restrict__ recs, int c0)
{
    if constexpr (WIDE) return plain_entries_bf16(plain, n_plain, recs, c0);
    constexpr uint32_t kElemBytes = (GT == NOVAK_GRAD_BF16) ? 2u : 4u;
    constexpr int K = kStatsEntries;
    Chunk ch[K];
    const void *base[K];
#pragma unroll
    for (int k = 0; k < K; ++k) ch[k] = plain[min(c0 + k, n_plain - 1)];
#pragma unroll
    for (int k = 0; k < K; ++k) base[k] = recs[ch[k].tensor].g;
    grid_dependency_wait();          // the gradient may come from the previous kernel

    const void *g[K];
    bool aligned[K];
    float xa[K][4], xb[K][4];
    // every entry's first two vectors per thread, all loads in flight at once
#pragma unroll
    for (int k = 0; k < K; ++k) {
        const uintptr_t addr = reinterpret_cast<uintptr_t>(base[k]) +
                               static_cast<uintptr_t>(ch[k].offset) * kElemBytes;
        g[k] = reinterpret_cast<const void *>(addr);          // the entry's first element
        aligned[k] = (addr & (4u * kElemBytes - 1u)) == 0;
        const uint32_t len = (c0 + k < n_plain) ? static_cast<uint32_t>(ch[k].len) : 0u;
        const uint32_t nvec = (len + 3u) >> 2;
        const uint32_t va = threadIdx.x, vb = va + kStatsBlock;
        const uint32_t ia = va << 2, ib = vb << 2;
        load_quad<GT>(g[k], aligned[k], ia, va < nvec ? (len - ia < 4u ? len - ia : 4u) : 0u, xa[k]);
        load_quad<GT>(g[k], aligned[k], ib, vb < nvec ? (len - ib < 4u ? len - ib : 4u) : 0u, xb[k]);
    }
    double sq = 0.0;
#pragma unroll
    for (int k = 0; k < K; ++k) {
        if (c0 + k >= n_plain) break;
        sq = sum_squares(xa[k], sq);
        sq = sum_squares(xb[k], sq);
        // entries longer than 2048 elements: the rest of the vectors
        const uint32_t len = static_cast<uint32_t>(ch[k].len);
        const uint32_t nvec = (len + 3u) >> 2;
        for (uint32_t v = threadIdx.x + 2u * kStatsBlock; v < nvec; v += kStatsBlock) {
            float x[4];
            const uint32_t i = v << 2;
            load_quad<GT>(g[k], aligned[k], i, len - i < 4u ? len - i : 4u, x);
            sq = sum_squares(x, sq);
        }
    }
    return sq;
}

// One aligned vector of 4 gradient elements as fp32.
template <int GT>
__device__ __forceinline__ void load_vec(const void *g, uint32_t v, float (&x)[4])
{
    if constexpr (GT == NOVAK_GRAD_F32) {
        const float4 t = __ldg(static_cast<const float4 *>(g) + v);
        x[0] = t.x; x[1] = t.y; x[2] = t.z; x[3] = t.w;
    } else {
        const uint2 t = __ldg(static_cast<const uint2 *>(g) + v);
        x[0] = __uint_as_float(t.x << 16);
        x[1] = __uint_as_float(t.x & 0xffff0000u);
        x[2] = __uint_as_float(t.y << 16);
        x[3] = __uint_as_float(t.y & 0xffff0000u);
    }
}

// Sum and sum of squares of elements [e0, e0 + n) of a tensor's gradient, the
// calling threads (`nthreads` of them, this one being number `t`) striding over
// 4-element vectors: 128-bit / 64-bit loads, four of them in flight per thread,
// where the span is aligned; element by element otherwise.
template <int GT>
__device__ __forceinline__ void span_sums(const void *g_tensor, uint32_t e0, uint32_t n, uint32_t t,
                                          uint32_t nthreads, double &sum, double &sq)
{
    constexpr uint32_t kElemBytes = (GT == NOVAK_GRAD_BF16) ? 2u : 4u;
    const uintptr_t addr = reinterpret_cast<uintptr_t>(g_tensor) + uintptr_t(e0) * kElemBytes;
    const void *g = reinterpret_cast<const void *>(addr);
    if ((addr & (4u * kElemBytes - 1u)) == 0) {
        const uint32_t nfull = n >> 2;
        uint32_t v = t;
        for (; v + 3u * nthreads < nfull; v += 4u * nthreads) {
            float x0[4], x1[4], x2[4], x3[4];
            load_vec<GT>(g, v, x0);
            load_vec<GT>(g, v + nthreads, x1);
            load_vec<GT>(g, v + 2u * nthreads, x2);
            load_vec<GT>(g, v + 3u * nthreads, x3);
            sum = sum_four(x0, sum); sq = sum_squares(x0, sq);
            sum = sum_four(x1, sum); sq = sum_squares(x1, sq);
            sum = sum_four(x2, sum); sq = sum_squares(x2, sq);
            sum = sum_four(x3, sum); sq = sum_squares(x3, sq);
        }
        if (v < nfull) {
            // up to three more vectors, again loaded together
            float x0[4] = {0.f, 0.f, 0.f, 0.f}, x1[4] = {0.f, 0.f, 0.f, 0.f}, x2[4] = {0.f, 0.f, 0.f, 0.f};
            load_vec<GT>(g, v, x0);
            if (v + nthreads < nfull) load_vec<GT>(g, v + nthreads, x1);
            if (v + 2u * nthreads < nfull) load_vec<GT>(g, v + 2u * nthreads, x2);
            sum = sum_four(x0, sum); sq = sum_squares(x0, sq);
            sum = sum_four(x1, sum); sq = sum_squares(x1, sq);
            sum = sum_four(x2, sum); sq = sum_squares(x2, sq);
        }
        const uint32_t e = (nfull << 2) + t;                  // ragged end: < 4 elements
        if (e < n) {
            const float x = grad_at<GT>(g, e);
            sum += double(x);
            sq = fma(double(x), double(x), sq);
        }
    } else {
#pragma unroll 4
        for (uint32_t e = t; e < n; e += nthreads) {
            const float x = grad_at<GT>(g, e);
            sum += double(x);
            sq = fma(double(x), double(x), sq);
        }
    }
}

// Whole rows [row0, row0 + n_rows) of length L, LANES lanes per row (8, 16 or
// 32), so that a warp works on 32 / LANES rows at a time: the loads of several
// rows are in flight together and a lane's share of a short row still fills a
// batch of four loads.  Row means are written; the squares go into sq.
template <int GT, int LANES>
__device__ __forceinline__ void rows_by_lane_group(const TensorRec &rec, uint32_t row0, uint32_t n_rows,
                                                   uint32_t L, double &sq)
{
    constexpr uint32_t kPerWarp = 32u / LANES;
    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31u;
    const uint32_t sub = lane / LANES, l = lane % LANES;
    const uint32_t end = row0 + n_rows;
    for (uint32_t r0 = row0 + warp * kPerWarp; r0 < end; r0 += kStatsWarps * kPerWarp) {
        const uint32_t r = r0 + sub;
        const bool live = r < end;
        double sum = 0.0;
        span_sums<GT>(rec.g, live ? r * L : 0u, live ? L : 0u, l, LANES, sum, sq);
#pragma unroll
        for (int o = LANES / 2; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
        if (live && l == 0u) rec.mean[r] = split_mean(sum, L);
    }
}

// ---- tensors with rows: one unit of the row table (see RowUnit)
template <int GT>
__device__ __forceinline__ double row_unit(const RowUnit u, const TensorRec rec,
                                           double *__restrict__ part_sum, int unit_index,
                                           double *sh)
{
    const uint32_t L = rec.row_len;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    double sq = 0.0;
    if (u.part_len != 0u) {
        // a slice of one long row for the whole CTA: the whole row, or a piece whose
        // sum the second kernel adds to its neighbours'
        double sum = 0.0;
        span_sums<GT>(rec.g, u.row0 * L + u.part_off, u.part_len, threadIdx.x, kStatsBlock, sum, sq);
        const double total = block_sum(sum, sh);
        if (threadIdx.x == 0) {
            if (u.n_parts == 1u) rec.mean[u.row0] = split_mean(total, L);
            else part_sum[unit_index] = total;
        }
    } else if (L > kRowHalfWarpMax) {
        rows_by_lane_group<GT, 32>(rec, u.row0, u.n_rows, L, sq);     // a warp per row
    } else if (L >= 128u) {
        rows_by_lane_group<GT, 16>(rec, u.row0, u.n_rows, L, sq);     // two rows per warp
    } else if (L >= 32u) {
        // (a thread per row would read its row as a chain of dependent scalar loads)
        rows_by_lane_group<GT, 8>(rec, u.row0, u.n_rows, L, sq);      // four rows per warp
    } else {
        // very short rows, a thread each
        const uint32_t r = u.row0 + threadIdx.x;
        if (threadIdx.x < u.n_rows) {
            double sum = 0.0;
#pragma unroll 4
            for (uint32_t e = r * L; e < (r + 1u) * L; ++e) {
                const float x = grad_at<GT>(rec.g, e);
                sum += double(x);
                sq = fma(double(x), double(x), sq);
            }
            rec.mean[r] = split_mean(sum, L);
        }
    }
    return sq;
}

// First kernel of the pass.  CTAs [0, ceil(n_plain / 4)) take 4 chunk-table
// entries each of the tensors without rows; the following n_units CTAs take one
// row unit each.  Every CTA leaves one sum of squares in part_sq[blockIdx.x].
template <int GT, bool ROWS>
__global__ void __launch_bounds__(kStatsBlock, NOVAK_STATS_MIN_CTAS)
novak_grad_stats_kernel(const Chunk *__restrict__ plain, int n_plain,
                        const RowUnit *__restrict__ units, int n_units,
                        const TensorRec *__restrict__ recs, double *__restrict__ part_sq,
                        double *__restrict__ part_sum)
{
    __shared__ double sh[kStatsWarps];
    grid_dependency_release();
    using Per = PlainEntries<GT, ROWS>;
    const int plain_ctas = (n_plain + Per::value - 1) / Per::value;
    double sq;
    if (!ROWS || static_cast<int>(blockIdx.x) < plain_ctas) {
        sq = plain_entries<GT, Per::wide>(plain, n_plain, recs, blockIdx.x * Per::value);
    } else {
        const int ui = blockIdx.x - plain_ctas;
        const RowUnit u = units[ui];
        const TensorRec rec = recs[u.tensor];
        grid_dependency_wait();      // the gradient may come from the previous kernel
        sq = row_unit<GT>(u, rec, part_sum, ui, sh);
    }
    const double total = block_sum(sq, sh);
    if (threadIdx.x == 0) part_sq[blockIdx.x] = total;
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
    for (int k = 0; k < K; ++k) p[k] = recs[ch[k].tensor].p_in + ch[k].offset;
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

// From the sums of squares to what the step kernel reads: the norm of the
// gradient and the clip factor (Table 2: active when ||g|| > c_clip), and,
// with has_p, the averages and the factor of Eq. 20-22 on the norm of the
// gradient as given and of theta_t.  One thread.
__device__ __forceinline__ void write_scalars(PrepOut *out, double sumsq, double psumsq,
                                              double c_clip, double auto_gamma, bool has_p)
{
    const double norm = sqrt(sumsq);
    const double factor = (c_clip > 0.0 && norm > c_clip) ? c_clip / norm : 1.0;
    out->norm = norm;
    out->factor = static_cast<float>(factor);
    float scale = 1.0f;
    if (has_p && auto_gamma > 0.0) {
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

// For a group that is sharded over several processes: the sums of squares of
// the WHOLE group (this process's local_sums, all-reduced by the caller) turned
// into norm, clip factor and Eq. 20-22.  One thread.
__global__ void novak_grad_norm_scalar_kernel(PrepOut *out, const double *totals, double c_clip,
                                              double auto_gamma, int has_p)
{
    grid_dependency_release();
    grid_dependency_wait();
    if (blockIdx.x == 0 && threadIdx.x == 0)
        write_scalars(out, totals[0], totals[1], c_clip, auto_gamma, has_p != 0);
}

// Second kernel of the pass, one THREAD per sum of the first: completes the
// means of the long rows that were cut into slices (the thread of a row's first
// slice adds the slices in order) and adds up the sums of squares: per CTA
// first, then the CTA that takes the last ticket adds the CTAs' sums in index
// order and writes the norm, the clip factor and, when asked, Eq. 20-22.
// The sums it reads are written by kernels that may still run while this grid
// is resident (dependent launch): they are not declared read-only.
__global__ void __launch_bounds__(kStatsBlock)
novak_grad_stats_finish_kernel(const RowUnit *__restrict__ units, int n_units,
                               const TensorRec *__restrict__ recs, int n_work,
                               const double *part_sq, const double *part_sum, int n_chunks,
                               const double *chunk_psq, double c_clip,
                               double auto_gamma, int finalize, double *cta_sq, PrepOut *out)
{
    __shared__ double sh[kStatsWarps];
    __shared__ unsigned sh_last;

    grid_dependency_release();
    grid_dependency_wait();          // everything below is the earlier kernels' output
    const int i = blockIdx.x * kStatsBlock + threadIdx.x;
    double sq = 0.0, psq = 0.0;
    if (i < n_work) sq = part_sq[i];
    if (chunk_psq != nullptr && i < n_chunks) psq = chunk_psq[i];
    if (i < n_units) {
        const RowUnit u = units[i];
        if (u.n_parts > 1u && u.part_idx == 0u) {
            double sum = 0.0;
            for (uint32_t j = 0; j < u.n_parts; ++j) sum += part_sum[i + j];
            const TensorRec r = recs[u.tensor];
            r.mean[u.row0] = split_mean(sum, r.row_len);
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
        // what this process saw; a sharded group all-reduces these two before the scalars
        out->local_sums[0] = sumsq;
        out->local_sums[1] = psumsq;
        if (finalize) write_scalars(out, sumsq, psumsq, c_clip, auto_gamma, chunk_psq != nullptr);
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

int grad_stats_work(int n_plain, int n_units, int grad_dtype)
{
    const int per = (grad_dtype == NOVAK_GRAD_BF16 && n_units == 0)
                        ? PlainEntries<NOVAK_GRAD_BF16, false>::value : kStatsEntries;
    return (n_plain + per - 1) / per + n_units;
}

int grad_stats_ctas(int n_work, int n_chunks)
{
    const int n = n_work > n_chunks ? n_work : n_chunks;
    return (n + kStatsBlock - 1) / kStatsBlock;
}

cudaError_t launch_grad_norm_scalars(PrepOut *prep, const double *d_totals, double c_clip,
                                     double auto_gamma, int pdl, cudaStream_t stream)
{
    if (!prep || !d_totals) return cudaErrorInvalidValue;
    int has_p = auto_gamma > 0.0 ? 1 : 0;
    void *args[] = {&prep, &d_totals, &c_clip, &auto_gamma, &has_p};
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(1);
    lc.blockDim = dim3(32);
    lc.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = (pdl & 4) ? 1 : 0;
    return cudaLaunchKernelExC(&lc, reinterpret_cast<const void *>(novak_grad_norm_scalar_kernel), args);
}

cudaError_t launch_grad_stats(const StatsPlan &w, int grad_dtype, double c_clip, double auto_gamma,
                              bool finalize, int pdl, cudaStream_t stream)
{
    const int n_work = grad_stats_work(w.n_plain, w.n_units, grad_dtype);
    if (n_work <= 0 || !w.recs || !w.part_sq || !w.cta_sq || !w.prep) return cudaErrorInvalidValue;
    if (w.n_plain > 0 && !w.plain) return cudaErrorInvalidValue;
    if (w.n_units > 0 && (!w.units || !w.part_sum)) return cudaErrorInvalidValue;
    if (auto_gamma > 0.0 && (!w.chunks || !w.chunk_psq || w.n_chunks <= 0)) return cudaErrorInvalidValue;
    const void *first = nullptr;
    switch (grad_dtype) {
    case NOVAK_GRAD_F32:
        first = w.n_units > 0 ? reinterpret_cast<const void *>(novak_grad_stats_kernel<NOVAK_GRAD_F32, true>)
                              : reinterpret_cast<const void *>(novak_grad_stats_kernel<NOVAK_GRAD_F32, false>);
        break;
    case NOVAK_GRAD_BF16:
        first = w.n_units > 0 ? reinterpret_cast<const void *>(novak_grad_stats_kernel<NOVAK_GRAD_BF16, true>)
                              : reinterpret_cast<const void *>(novak_grad_stats_kernel<NOVAK_GRAD_BF16, false>);
        break;
    default: return cudaErrorInvalidValue;
    }
    StatsPlan a = w;
    void *args1[] = {&a.plain, &a.n_plain, &a.units, &a.n_units, &a.recs, &a.part_sq, &a.part_sum};
    cudaError_t e = launch_pdl(first, static_cast<unsigned>(n_work), args1, (pdl & 2) != 0, stream);
    if (e != cudaSuccess) return e;
    const double *c_psq = nullptr;
    if (auto_gamma > 0.0) {
        void *args_p[] = {&a.chunks, &a.n_chunks, &a.recs, &a.chunk_psq};
        const unsigned grid_p = static_cast<unsigned>((a.n_chunks + kStatsEntries - 1) / kStatsEntries);
        e = launch_pdl(reinterpret_cast<const void *>(novak_param_sumsq_kernel), grid_p, args_p,
                       (pdl & 2) != 0, stream);
        if (e != cudaSuccess) return e;
        c_psq = a.chunk_psq;
    }
    int work = n_work;
    int fin = finalize ? 1 : 0;
    const double *c_sq = a.part_sq, *c_sum = a.part_sum;
    void *args2[] = {&a.units, &a.n_units, &a.recs, &work, &c_sq, &c_sum, &a.n_chunks, &c_psq,
                     &c_clip, &auto_gamma, &fin, &a.cta_sq, &a.prep};
    return launch_pdl(reinterpret_cast<const void *>(novak_grad_stats_finish_kernel),
                      static_cast<unsigned>(grad_stats_ctas(n_work, c_psq ? a.n_chunks : 0)), args2,
                      (pdl & 4) != 0, stream);
}

}  // namespace novak
