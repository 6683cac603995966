// Launch side of the step kernel: picks the instantiation for the step's modes
// and launches it; also owns the statically allocated work table of
// novak_step_noalloc.
#include "novak_internal.h"

#include "novak.h"

#include <mutex>

#ifndef NOVAK_BLOCK
#define NOVAK_BLOCK 256
#endif

namespace novak {

// novak_step_inst.cu, compiled once per gradient pre-processing mode, holds the
// kernels; mode N (the PRE_* bits as a number) exports step_kernel_mode<N>.
#define NOVAK_FOR_EACH_PRE_MODE(X) \
    X(0) X(1) X(2) X(3) X(4) X(5) X(6) X(7) X(8) X(9) X(10) X(11) X(12) X(13) X(14) X(15)
#define NOVAK_DECLARE(N) void *step_kernel_mode##N(int nesterov, int grad_dtype, int la);
NOVAK_FOR_EACH_PRE_MODE(NOVAK_DECLARE)
#undef NOVAK_DECLARE

namespace {

constexpr int kBlock = NOVAK_BLOCK;

using StepKernelFn = void (*)(const Chunk *, int, const TensorRec *, const PrepOut *,
                              const float *, StepScalars, int);

using StepRowsKernelFn = void (*)(const Chunk *, int, const RowUnit *, int, const TensorRec *,
                                  StepScalars);

void *pick_kernel_raw(int nesterov, int grad_dtype, int la, int pre)
{
    void *fn = nullptr;
    switch (pre) {
#define NOVAK_CASE(N) case N: fn = step_kernel_mode##N(nesterov, grad_dtype, la); break;
        NOVAK_FOR_EACH_PRE_MODE(NOVAK_CASE)
#undef NOVAK_CASE
    default: break;
    }
    return fn;
}

StepKernelFn pick_kernel(int nesterov, int grad_dtype, int la, int pre)
{
    if ((pre & PRE_MASK) == PRE_CENTER_ROWS) return nullptr;     // another signature
    return reinterpret_cast<StepKernelFn>(pick_kernel_raw(nesterov, grad_dtype, la, pre));
}

}  // namespace

// Work table of novak_step_noalloc: tensor records followed by the chunk table,
// resident in every GPU that loads this library until the process exits
// (320 KiB + 2 MiB).  In host code this name is only a handle for
// cudaGetSymbolAddress, never a device address.
struct NoAllocTable {
    TensorRec recs[kNoAllocMaxTensors];
    Chunk chunks[kNoAllocMaxChunks];
};
static __device__ __align__(256) unsigned char g_noalloc_table[sizeof(NoAllocTable)];

cudaError_t noalloc_table(TensorRec **d_recs, Chunk **d_chunks)
{
    constexpr int kMaxDevices = 64;
    static void *resolved[kMaxDevices] = {};
    static std::mutex resolved_mutex;   // host threads may make their first call together
    std::lock_guard<std::mutex> lock(resolved_mutex);
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    if (!resolved[dev]) {
        void *ptr = nullptr;
        e = cudaGetSymbolAddress(&ptr, g_noalloc_table);  // address on the current device
        if (e != cudaSuccess) return e;
        resolved[dev] = ptr;
    }
    NoAllocTable *t = static_cast<NoAllocTable *>(resolved[dev]);
    *d_recs = t->recs;
    *d_chunks = t->chunks;
    return cudaSuccess;
}

int step_block_threads() { return kBlock; }

cudaError_t step_occupancy(int nesterov, int grad_dtype, int la, int pre, int *ctas_per_sm)
{
    void *fn = pick_kernel_raw(nesterov, grad_dtype, la, pre);
    if (!fn) return cudaErrorInvalidValue;
    return cudaOccupancyMaxActiveBlocksPerMultiprocessor(ctas_per_sm, fn, kBlock, 0);
}

cudaError_t launch_step_rows(const Chunk *d_rest, int n_rest, const RowUnit *d_units, int n_units,
                             const TensorRec *d_recs, const StepScalars &s, int nesterov,
                             int grad_dtype, int la, const LaunchCfg &cfg, cudaStream_t stream)
{
    if ((cfg.pre & PRE_MASK) != PRE_CENTER_ROWS || n_rest < 0 || n_units < 0 || n_rest + n_units <= 0)
        return cudaErrorInvalidValue;
    StepRowsKernelFn fn = reinterpret_cast<StepRowsKernelFn>(pick_kernel_raw(nesterov, grad_dtype, la, cfg.pre));
    if (!fn) return cudaErrorInvalidValue;
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(static_cast<unsigned>(n_rest + n_units));
    lc.blockDim = dim3(kOwnBlockThreads);
    lc.dynamicSmemBytes = 0;
    lc.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = (cfg.pdl & 1) ? 1 : 0;
    return cudaLaunchKernelEx(&lc, fn, d_rest, n_rest, d_units, n_units, d_recs, s);
}

cudaError_t launch_step(const Chunk *d_chunks, int n_chunks, const TensorRec *d_recs,
                        const PrepOut *prep, const float *trust, const StepScalars &s, int nesterov,
                        int grad_dtype, int la, const LaunchCfg &cfg, cudaStream_t stream)
{
    StepKernelFn fn = pick_kernel(nesterov, grad_dtype, la, cfg.pre);
    if (!fn || n_chunks <= 0 || cfg.grid <= 0) return cudaErrorInvalidValue;
    if ((cfg.pre & PRE_MASK) != PRE_NONE && prep == nullptr) return cudaErrorInvalidValue;
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(static_cast<unsigned>(cfg.grid));
    lc.blockDim = dim3(kBlock);
    lc.dynamicSmemBytes = 0;
    lc.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = (cfg.pdl & 1) ? 1 : 0;
    return cudaLaunchKernelEx(&lc, fn, d_chunks, n_chunks, d_recs, prep, trust, s, cfg.reverse);
}

}  // namespace novak
