// The optimizer handle behind the C ABI and what the host translation units
// (novak_host.cpp, novak_host_device.cpp, novak_host_step.cpp) share: the
// hyperparameters, the per-step scalar plan and the helpers that cross files.
// Private to the library.
#pragma once

#include "novak.h"
#include "novak_internal.h"
#include "novak_plan.h"

#include <cstdint>
#include <string>
#include <vector>

namespace novak_host {

using novak::Chunk;
using novak::PrepOut;
using novak::RowUnit;
using novak::StepScalars;
using novak::TensorRec;

constexpr int kRing = 4;                       // pinned staging slots for tensor records
constexpr int kRecTables = 8;                  // device record tables kept per handle
constexpr int64_t kSlotAlign = 32;             // elements: 128-byte slots
constexpr uint64_t kMetaMagic = 0x4e4f56414b763037ull;  // "NOVAKv07"
constexpr int64_t kDefaultChunkElems = 2048;
constexpr int kDefaultCtasPerSm = 0;
constexpr int64_t kDefaultHostSegmentElems = 4 << 20;  // elements per pipelined segment
constexpr int kMaxHostSegments = 32;

struct Handle {
    Hyper h{};
    uint32_t warnings = 0;
    int64_t chunk_elems = kDefaultChunkElems;
    int ctas_per_sm = kDefaultCtasPerSm;
    int serpentine = 0;
    int pdl = 7;                       // bit 0: step kernel, 1: statistics, 2: its second kernel
    int64_t host_segment_elems = kDefaultHostSegmentElems;

    // state layout (fixed by novak_attach_state)
    bool attached = false;
    char *d_state = nullptr;
    int n = 0;
    int n_arrays = 0;
    int64_t region_elems = 0;
    int64_t total_numel = 0;
    std::vector<int64_t> numel, slot_off;
    std::vector<int32_t> phase;
    std::vector<int64_t> rows, row_off;   // dimension 0 of each tensor (0: none), prefix sums
    int64_t total_rows = 0;
    std::vector<void *> copies;           // bf16 copies of the parameters the step also writes

    // counters
    int64_t t = 0, n_syncs = 0, last_sync = 0, launches = 0;
    Plan last_plan{};
    int last_grid = 0;

    // device work table
    Chunk *d_chunks = nullptr;
    std::vector<Chunk> h_chunks;       // host copy of the device chunk table
    int n_chunks = 0;
    TensorRec *d_recs = nullptr;       // kRecTables tables of n records each
    TensorRec *h_recs[kRing] = {nullptr, nullptr, nullptr, nullptr};
    cudaEvent_t ring_ev[kRing] = {nullptr, nullptr, nullptr, nullptr};
    int ring_pos = 0;
    // Which (parameter, gradient) pointer lists the device tables hold.  A
    // caller that rotates through a few gradient buffers finds its table
    // already resident and the step enqueues nothing but the kernel.
    struct RecTable {
        std::vector<void *> p;
        std::vector<const void *> g;
        const void *save = nullptr;   // save buffer theta_{t-1} is read from (NULL: the parameters)
        int gdtype = -1;
        uint64_t hash = 0;
        int64_t last_use = 0;
    };
    RecTable tables[kRecTables];
    int cur_table = -1;
    int64_t table_clock = 0;
    int64_t record_uploads = 0;
    int sms = 0;

    // Scratch of the gradient statistics pass (one allocation): its result, one
    // sum of squares and two row-piece sums per chunk-table entry, the row means.
    char *d_prep = nullptr;
    PrepOut *prep_out = nullptr;
    double *part_sq = nullptr, *part_sum = nullptr, *cta_sq = nullptr, *chunk_psq = nullptr;
    Chunk *d_plain = nullptr;           // entries of the tensors without rows (NULL: all of them)
    RowUnit *d_units = nullptr;
    int n_plain = 0, n_units = 0;
    // step kernel that forms the row means itself (PRE_CENTER_ROWS): the chunk-table
    // entries of the tensors it does not own rows of, and its units of whole rows
    int center_in_step = 1;             // NOVAK_OPT_CENTRALIZE_IN_STEP
    Chunk *d_rest = nullptr;
    RowUnit *d_own = nullptr;
    RowUnit *d_long_units = nullptr;    // statistics units of the tensors with rows too long to own
    int n_rest = 0, n_own = 0, n_long_units = 0;
    int64_t rows_gen = 0;               // bumped whenever the row settings change
    int64_t prep_key = -1;              // rows_gen and centring the scratch was laid out for
    // the averages of Eq. 20-21 live in the scratch; values waiting to be written there
    // a step taken in two halves (novak_step_begin / novak_step_finish)
    bool half_open = false;
    int half_launches = 0;
    alignas(8) unsigned char half_ctx[256] = {};   // the StepCtx of the open step
    int device = -1;                    // CUDA device of the attached state buffer (-1: unknown)

    // graph-capturable step: the counters and the plan in device memory
    int dyn = 0;
    novak::DevPlan *d_plan = nullptr;
    bool dyn_upload_counters = true, dyn_upload_rates = true;
    bool extrapolated = false;          // between novak_nesterov_extrapolate and _restore
    novak::LookRec *d_look = nullptr;   // device records of the two look-ahead helpers
    novak::LookRec *h_look = nullptr;   // pinned staging of those records
    cudaEvent_t look_ev = nullptr;      // the staging buffer's last upload
    std::vector<void *> look_p;         // the parameter list the device records hold
    void *look_save = nullptr;          // save buffer of the open look-ahead
    bool ema_pending = false;
    double pending_g_bar = 0.0, pending_theta_bar = 0.0;
    float2 *row_mean = nullptr;

    // Scratch of layer adaptation (one allocation): two sums of squares per
    // chunk-table entry, where each tensor's entries start, the trust ratios.
    char *d_trust = nullptr;
    double *chunk_u2 = nullptr, *chunk_p2 = nullptr;
    int *tensor_first = nullptr;
    float *trust = nullptr;
    std::vector<int> h_tensor_first;
    // layer adaptation and step in one launch: the item list, the kernel's counters
    // and per-tensor words (one allocation), the directions of one step (another), a
    // host-mapped error word
    int adapt_in_step = 1;              // NOVAK_OPT_LAYER_ADAPTATION_IN_STEP
    int64_t adapt_lead_elems = 0;          // NOVAK_OPT_LAYER_ADAPTATION_LEAD
    int adapt_group = 4;                   // NOVAK_OPT_LAYER_ADAPTATION_GROUP
    char *d_adapt = nullptr;
    int *d_item_code = nullptr;         // every item's first chunk-table entry
    Chunk *d_item_chunk = nullptr;
    int n_items = 0;
    int adapt_lag = 0;                  // CTA b updates item b - adapt_lag
    novak::AdaptCtl *adapt_ctl = nullptr;
    unsigned *adapt_arrived = nullptr;
    unsigned long long *adapt_ready = nullptr;
    unsigned *h_adapt_error = nullptr;  // pinned, mapped; written by the kernel
    unsigned *d_adapt_error = nullptr;  // its device address
    unsigned adapt_epoch = 0;
    float *adapt_direction = nullptr;   // one slot of adapt_slot_elems floats per chunk-table entry
    int adapt_slot_elems = 0;

    // novak_step_host: the chunk table cut into segments, each with the element
    // ranges it covers, two copy streams and the events that order them.
    struct Range { int tensor; int64_t off, len; };
    struct Segment { int c0, c1; std::vector<Range> ranges; };
    std::vector<Segment> segments;
    int64_t segments_for = -1;          // host_segment_elems the segments were cut for
    cudaStream_t up_stream = nullptr, down_stream = nullptr;
    std::vector<cudaEvent_t> host_ev;   // [0] start, [1] end, then (uploaded, stepped) per segment

    // host copies of the work table for novak_step_noalloc (no device memory of ours)
    std::vector<Chunk> na_chunks;
    std::vector<TensorRec> na_recs;
    std::vector<void *> na_p;
    std::vector<const void *> na_g;
    int na_gdtype = -1;
    uint64_t na_token = 0;       // identifies this handle's upload in the shared table

    std::string err;
};

}  // namespace novak_host

struct novak_opt : novak_host::Handle {};

namespace novak_host {

// Planner helpers (novak_host.cpp); the scalar plan itself is in novak_plan.h.
int64_t round_up(int64_t x, int64_t a);
void build_chunks(const int64_t *numel, const int32_t *phase, int n, int64_t chunk_elems,
                  std::vector<Chunk> &out);
void build_row_units(const int64_t *numel, const int64_t *rows, int n, std::vector<RowUnit> &out);
// Units of the step kernel that owns rows: whole rows of the tensors whose rows
// have at most novak::kOwnRowMax elements, about novak::kOwnUnitElems elements
// and at most novak::kOwnUnitRows rows per unit.
void build_own_units(const int64_t *numel, const int64_t *rows, int n, std::vector<RowUnit> &out);
int check_hyper(const Hyper &h, const char **why);

// The variant the kernels are instantiated for: a true step's gradient needs no
// correction (Eq. 11's gradient is given), so it runs as variant none.
inline int kernel_variant(const Plan &p)
{
    return p.nesterov == NOVAK_NESTEROV_TRUE ? NOVAK_NESTEROV_NONE : p.nesterov;
}

// Makes the handle's device current for the lifetime of the object when it is
// not (a process that drives several GPUs); restores the caller's device.
struct DeviceGuard {
    int prev = -1;
    bool switched = false;
    explicit DeviceGuard(int want)
    {
        if (want < 0 || cudaGetDevice(&prev) != cudaSuccess || prev == want) return;
        switched = cudaSetDevice(want) == cudaSuccess;
    }
    ~DeviceGuard()
    {
        if (switched) cudaSetDevice(prev);
    }
    DeviceGuard(const DeviceGuard &) = delete;
    DeviceGuard &operator=(const DeviceGuard &) = delete;
};

// Error reporting: store the message in the handle, return the code.
int fail(novak_opt *o, int code, const char *fmt, ...);
int fail_cuda(novak_opt *o, cudaError_t e, const char *what);

// State layout and mode helpers.
int n_state_arrays(const Hyper &h);
// Start of tensor i inside state array `array` (0 m, 1 v, 2 slow, 3 running
// sum): m and v hold fp32 or bf16 elements, the lookahead arrays fp32.
void *slice(const novak_opt *o, int array, int i);
inline int moment_bytes(const Hyper &h) { return h.mom16 ? 2 : 4; }
// Bytes of the whole state for a region of `region_elems` padded elements.
size_t state_bytes_for(const Hyper &h, int64_t region_elems);
int pre_mode(const novak_opt *o);
// The mode a step actually runs in: pre_mode, or PRE_CENTER_ROWS where the step
// kernel can centralize by itself (whole_table: the step is one launch over the
// whole group, as in novak_step).
int step_pre_mode(const novak_opt *o, bool whole_table);
int prepare_prep(novak_opt *o, cudaStream_t stream);
void fill_info(const novak_opt *o, const Plan &p, novak_info *out);

// Device work tables (novak_host_device.cpp).
void release_device(novak_opt *o);
int prepare_device(novak_opt *o, cudaStream_t stream);
void invalidate_tables(novak_opt *o);
int prepare_trust(novak_opt *o, cudaStream_t stream);
// The item list and counters of the one-launch form of layer adaptation.
int prepare_adapt(novak_opt *o, cudaStream_t stream);
// Items of that kernel, in tensor order.  An item is a run of consecutive chunk-
// table entries of one tensor: the tensor's first entry alone, the others in
// runs of `group`.  items[k] is the item's first entry, counts[k] its number of
// entries.  Returns the lag: CTA b takes the statistics of item b and the update
// of item b - lag; the longest tensor's items minus one (so that an update only
// ever waits for CTAs with a lower index) plus lead_entries / group.
int64_t build_adapt_items(const std::vector<int> &tensor_first, int n, int64_t lead_entries, int group,
                          std::vector<int32_t> &items, std::vector<int32_t> &counts);
uint64_t hash_pointers(void *const *d_params, const void *const *d_grads, int n, int grad_dtype,
                       const void *save);
// `save`: NULL, or the save buffer of an open look-ahead, from which the step
// then reads theta_{t-1} (the parameter tensors hold Eq. 10's point).
int refresh_records(novak_opt *o, void *const *d_params, const void *const *d_grads,
                    int grad_dtype, const void *save, cudaStream_t stream);
// Device records of the look-ahead helpers for this parameter list (uploaded
// only when the list differs from the one the device holds).
int prepare_look(novak_opt *o, void *const *d_params, cudaStream_t stream);
// Device-resident plan of the graph-capturable step: allocated on first use;
// counters and rates are uploaded when the host has changed them.
int prepare_dyn(novak_opt *o, cudaStream_t stream);
// The device-resident plan copied to the host (synchronises the device).
int read_dyn(const novak_opt *o, novak::DevPlan *out);

}  // namespace novak_host
