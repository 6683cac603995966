// True Nesterov momentum (Section 4.4, Eq. 10-12): the two passes around the
// caller's closure.  novak_look_kernel<false, .> saves theta_{t-1} and moves the
// parameters to theta~ = theta_{t-1} + beta_N m_{t-1} (Eq. 10);
// novak_look_kernel<true, .> puts theta_{t-1} back (Section 5.8's steps 1, 2 and
// 4).  Both walk the step kernel's chunk table, 128 bits per access where the
// parameters, the first moment and the save buffer share 16-byte alignment.
// HBM-bound: 16 B per element (theta and m read, save and theta written; 14 B
// with bf16 moments) and 8 B per element (save read, theta written).
#include "novak.h"
#include "novak_internal.h"

namespace novak {
namespace {

constexpr int kLookThreads = 256;

__device__ __forceinline__ float4 ld_stream(const float *p)
{
    float4 v;
    asm volatile("ld.global.cs.v4.f32 {%0,%1,%2,%3}, [%4];"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
    return v;
}

__device__ __forceinline__ void st_stream(float *p, float4 v)
{
    asm volatile("st.global.cs.v4.f32 [%0], {%1,%2,%3,%4};"
                 :: "l"(p), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
}

// Four first moments as stored: fp32, or bf16 widened exactly.
template <bool M16>
__device__ __forceinline__ float4 ld_moment4(const void *m, int vec)
{
    if constexpr (M16) {
        uint2 t;
        asm volatile("ld.global.cs.v2.u32 {%0,%1}, [%2];"
                     : "=r"(t.x), "=r"(t.y) : "l"(static_cast<const uint2 *>(m) + vec));
        return make_float4(__uint_as_float(t.x << 16), __uint_as_float(t.x & 0xffff0000u),
                           __uint_as_float(t.y << 16), __uint_as_float(t.y & 0xffff0000u));
    } else {
        return ld_stream(static_cast<const float *>(m) + 4 * vec);
    }
}

template <bool M16>
__device__ __forceinline__ float ld_moment1(const void *m, int idx)
{
    if constexpr (M16)
        return __uint_as_float(static_cast<unsigned>(static_cast<const unsigned short *>(m)[idx]) << 16);
    else
        return static_cast<const float *>(m)[idx];
}

// RESTORE = false: save <- theta, theta <- theta + beta_N m.
// RESTORE = true:  theta <- save (m_region is not read).
// M16: the first moment is stored as bf16.
template <bool RESTORE, bool M16>
__global__ void __launch_bounds__(kLookThreads)
novak_look_kernel(const Chunk *__restrict__ chunks, int n_chunks, const LookRec *__restrict__ recs,
                  const void *__restrict__ m_region, float *__restrict__ save_region, float beta_n)
{
    constexpr int kMomBytes = M16 ? 2 : 4;
    // Programmatic dependent launch: CTAs become resident and read their first
    // work-table entry (written by copies only) while the previous kernel on
    // the stream drains; no tensor is touched before it has completed.
    asm volatile("griddepcontrol.launch_dependents;");
    int c = blockIdx.x;
    if (c >= n_chunks) return;
    Chunk ch = chunks[c];
    LookRec r = recs[ch.tensor];
    asm volatile("griddepcontrol.wait;" ::: "memory");
    for (;;) {
        float *p = r.p + ch.offset;
        float *sv = save_region + r.state_off + ch.offset;
        const void *m = RESTORE ? nullptr
                                : static_cast<const char *>(m_region) + (r.state_off + ch.offset) * kMomBytes;
        uintptr_t bits = reinterpret_cast<uintptr_t>(p) | reinterpret_cast<uintptr_t>(sv);
        if (!RESTORE) bits |= reinterpret_cast<uintptr_t>(m) << (M16 ? 1 : 0);
        if ((bits & 15u) == 0) {
            const int nvec = ch.len >> 2;
            // two vectors per thread and pass: all loads first, then the stores
            for (int i = threadIdx.x; i < nvec; i += 2 * kLookThreads) {
                const int j = i + kLookThreads;
                const bool two = j < nvec;
                if (RESTORE) {
                    const float4 a = ld_stream(sv + 4 * i);
                    float4 b = a;
                    if (two) b = ld_stream(sv + 4 * j);
                    st_stream(p + 4 * i, a);
                    if (two) st_stream(p + 4 * j, b);
                } else {
                    const float4 a = ld_stream(p + 4 * i);
                    const float4 ma = ld_moment4<M16>(m, i);
                    float4 b = a, mb = ma;
                    if (two) {
                        b = ld_stream(p + 4 * j);
                        mb = ld_moment4<M16>(m, j);
                    }
                    st_stream(sv + 4 * i, a);
                    st_stream(p + 4 * i, make_float4(fmaf(beta_n, ma.x, a.x), fmaf(beta_n, ma.y, a.y),
                                                     fmaf(beta_n, ma.z, a.z), fmaf(beta_n, ma.w, a.w)));
                    if (two) {
                        st_stream(sv + 4 * j, b);
                        st_stream(p + 4 * j, make_float4(fmaf(beta_n, mb.x, b.x), fmaf(beta_n, mb.y, b.y),
                                                         fmaf(beta_n, mb.z, b.z), fmaf(beta_n, mb.w, b.w)));
                    }
                }
            }
            // ragged tail of a tensor: at most 3 elements
            const int idx = (nvec << 2) + threadIdx.x;
            if (idx < ch.len) {
                if (RESTORE) {
                    p[idx] = sv[idx];
                } else {
                    const float a = p[idx];
                    sv[idx] = a;
                    p[idx] = fmaf(beta_n, ld_moment1<M16>(m, idx), a);
                }
            }
        } else {
            for (int i = threadIdx.x; i < ch.len; i += kLookThreads) {
                if (RESTORE) {
                    p[i] = sv[i];
                } else {
                    const float a = p[i];
                    sv[i] = a;
                    p[i] = fmaf(beta_n, ld_moment1<M16>(m, i), a);
                }
            }
        }
        c += gridDim.x;
        if (c >= n_chunks) break;
        ch = chunks[c];
        r = recs[ch.tensor];
    }
}

template <typename Kernel, typename... Args>
cudaError_t launch_look(Kernel kernel, int grid, int pdl, cudaStream_t stream, Args... args)
{
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(static_cast<unsigned>(grid));
    lc.blockDim = dim3(kLookThreads);
    lc.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = (pdl & 1) ? 1 : 0;
    return cudaLaunchKernelEx(&lc, kernel, args...);
}

}  // namespace

cudaError_t launch_extrapolate(const Chunk *d_chunks, int n_chunks, const LookRec *d_recs,
                               const void *m_region, int moments_bf16, float *save_region,
                               float beta_n, int grid, int pdl, cudaStream_t stream)
{
    if (n_chunks <= 0) return cudaSuccess;
    if (grid < 1 || grid > n_chunks) grid = n_chunks;
    if (moments_bf16)
        return launch_look(novak_look_kernel<false, true>, grid, pdl, stream, d_chunks, n_chunks, d_recs,
                           m_region, save_region, beta_n);
    return launch_look(novak_look_kernel<false, false>, grid, pdl, stream, d_chunks, n_chunks, d_recs,
                       m_region, save_region, beta_n);
}

cudaError_t launch_restore(const Chunk *d_chunks, int n_chunks, const LookRec *d_recs,
                           const float *save_region, int grid, int pdl, cudaStream_t stream)
{
    if (n_chunks <= 0) return cudaSuccess;
    if (grid < 1 || grid > n_chunks) grid = n_chunks;
    // the kernel only reads the save buffer when restoring
    const void *no_moments = nullptr;
    return launch_look(novak_look_kernel<true, false>, grid, pdl, stream, d_chunks, n_chunks, d_recs,
                       no_moments, const_cast<float *>(save_region), 0.0f);
}

}  // namespace novak
