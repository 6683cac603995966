// Launch side of the step kernel: picks the instantiation for the step's modes
// and launches it; also owns the statically allocated work table of
// novak_step_noalloc.
#include "novak_internal.h"

#include "novak.h"

#ifndef NOVAK_BLOCK
#define NOVAK_BLOCK 256
#endif

namespace novak {

// One translation unit per gradient pre-processing mode holds the kernels.
void *step_kernel_pre0(int nesterov, int grad_dtype, int la);
void *step_kernel_pre1(int nesterov, int grad_dtype, int la);
void *step_kernel_pre2(int nesterov, int grad_dtype, int la);
void *step_kernel_pre0_copy(int nesterov, int grad_dtype, int la);
void *step_kernel_pre1_copy(int nesterov, int grad_dtype, int la);
void *step_kernel_pre2_copy(int nesterov, int grad_dtype, int la);
void *step_kernel_pre0_mom16(int nesterov, int grad_dtype, int la);
void *step_kernel_pre1_mom16(int nesterov, int grad_dtype, int la);
void *step_kernel_pre2_mom16(int nesterov, int grad_dtype, int la);
void *step_kernel_pre0_copy_mom16(int nesterov, int grad_dtype, int la);
void *step_kernel_pre1_copy_mom16(int nesterov, int grad_dtype, int la);
void *step_kernel_pre2_copy_mom16(int nesterov, int grad_dtype, int la);

namespace {

constexpr int kBlock = NOVAK_BLOCK;

using StepKernelFn = void (*)(const Chunk *, int, const TensorRec *, const PrepOut *,
                              const float *, StepScalars, int);

StepKernelFn pick_kernel(int nesterov, int grad_dtype, int la, int pre)
{
    void *fn = nullptr;
    switch (pre) {
    case PRE_NONE: fn = step_kernel_pre0(nesterov, grad_dtype, la); break;
    case PRE_SCALE: fn = step_kernel_pre1(nesterov, grad_dtype, la); break;
    case PRE_CENTER: fn = step_kernel_pre2(nesterov, grad_dtype, la); break;
    case PRE_NONE | PRE_COPY16: fn = step_kernel_pre0_copy(nesterov, grad_dtype, la); break;
    case PRE_SCALE | PRE_COPY16: fn = step_kernel_pre1_copy(nesterov, grad_dtype, la); break;
    case PRE_CENTER | PRE_COPY16: fn = step_kernel_pre2_copy(nesterov, grad_dtype, la); break;
    case PRE_NONE | PRE_MOM16: fn = step_kernel_pre0_mom16(nesterov, grad_dtype, la); break;
    case PRE_SCALE | PRE_MOM16: fn = step_kernel_pre1_mom16(nesterov, grad_dtype, la); break;
    case PRE_CENTER | PRE_MOM16: fn = step_kernel_pre2_mom16(nesterov, grad_dtype, la); break;
    case PRE_NONE | PRE_COPY16 | PRE_MOM16: fn = step_kernel_pre0_copy_mom16(nesterov, grad_dtype, la); break;
    case PRE_SCALE | PRE_COPY16 | PRE_MOM16: fn = step_kernel_pre1_copy_mom16(nesterov, grad_dtype, la); break;
    case PRE_CENTER | PRE_COPY16 | PRE_MOM16: fn = step_kernel_pre2_copy_mom16(nesterov, grad_dtype, la); break;
    default: break;
    }
    return reinterpret_cast<StepKernelFn>(fn);
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
    StepKernelFn fn = pick_kernel(nesterov, grad_dtype, la, pre);
    if (!fn) return cudaErrorInvalidValue;
    return cudaOccupancyMaxActiveBlocksPerMultiprocessor(ctas_per_sm, fn, kBlock, 0);
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
