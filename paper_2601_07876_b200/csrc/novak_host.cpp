// Host side of the NOVAK step library: the C ABI, hyperparameter validation,
// the per-step scalar plan (double precision), the state layout, the
// multi-tensor chunk table and the launch.  Declarations and argument
// contracts are in include/novak.h.
#include "novak.h"
#include "novak_internal.h"

#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <vector>

using novak::Chunk;
using novak::PrepOut;
using novak::RowUnit;
using novak::StepScalars;
using novak::TensorRec;

namespace {

constexpr int kRing = 4;                       // pinned staging slots for tensor records
constexpr int kRecTables = 8;                  // device record tables kept per handle
constexpr int64_t kSlotAlign = 32;             // elements: 128-byte slots
constexpr uint64_t kMetaMagic = 0x4e4f56414b763036ull;  // "NOVAKv06"
constexpr int64_t kDefaultChunkElems = 2048;
constexpr int kDefaultCtasPerSm = 0;
constexpr int64_t kDefaultHostSegmentElems = 4 << 20;  // elements per pipelined segment
constexpr int kMaxHostSegments = 32;

struct Hyper {
    double lr, beta1, beta2, eps, wd, beta_n, la_alpha;
    double clip;            // c_clip of the global-norm clipping, 0: off
    int nesterov, la_k, la_mode, rectified, bias1_power;
    int centralize;         // Eq. 26 on tensors that were given rows
    int layer_adapt;        // Eq. 19 / 25: one trust ratio per tensor
    int adaptive_beta;      // Eq. 3-4
    double tau1, tau2;      // warm-up time scales of beta1, beta2
    double sparse_tau;      // tau of Eq. 27, 0: no mask
    int auto_lr;            // Eq. 20-22
    double auto_gamma;      // gamma of Eq. 20-21
};

struct Plan {
    double bc1, bc2, rho_inf, rho_t, r_t, step_size, decay;
    double beta1_t, beta2_t;   // coefficients of Eq. 1-2 at this step (Eq. 3-4 when warmed up)
    int rect_branch, is_sync;
};

// Eq. 5-9 and 18 for the 1-based step index t.  1 - beta^t is evaluated as
// -expm1(t log beta) for every t (Section 5.8 gives the log form for large t).
Plan make_plan(const Hyper &h, int64_t t)
{
    Plan p;
    const double td = static_cast<double>(t);
    const double l1 = h.beta1 > 0.0 ? td * std::log(h.beta1) : -INFINITY;
    const double l2 = h.beta2 > 0.0 ? td * std::log(h.beta2) : -INFINITY;
    p.bc1 = -std::expm1(l1);
    p.bc2 = -std::expm1(l2);
    const double b2t = std::exp(l2);
    p.rho_inf = 2.0 / (1.0 - h.beta2) - 1.0;
    p.rho_t = p.rho_inf - 2.0 * td * b2t / p.bc2;
    p.rect_branch = (h.rectified && p.rho_t >= 5.0) ? 1 : 0;
    p.r_t = 1.0;
    if (p.rect_branch) {
        const double a = (p.rho_t - 4.0) / (p.rho_inf - 4.0);
        const double b = (p.rho_t - 2.0) / (p.rho_inf - 2.0);
        p.r_t = std::sqrt(a * b * (p.rho_inf / p.rho_t));
    }
    p.step_size = h.lr * p.r_t;
    if (h.bias1_power == 2) p.step_size /= p.bc1;
    p.decay = 1.0 - h.lr * h.wd;
    p.is_sync = (h.la_k > 0 && t % h.la_k == 0) ? 1 : 0;
    // Phase 3, Eq. 3-4: only the moment updates see the warmed-up coefficients.
    p.beta1_t = h.beta1;
    p.beta2_t = h.beta2;
    if (h.adaptive_beta) {
        p.beta1_t = h.beta1 * -std::expm1(-td / h.tau1);
        p.beta2_t = h.beta2 * -std::expm1(-td / h.tau2);
    }
    return p;
}

int lookahead_action(const Hyper &h, int64_t t)
{
    using namespace novak;
    if (h.la_k <= 0) return LA_NONE;
    const bool first_step = (t == 1);
    const bool sync = (t % h.la_k == 0);
    const bool first_of_window = ((t - 1) % h.la_k == 0);
    const bool traj = (h.la_mode == NOVAK_LOOKAHEAD_TRAJ_MEAN && h.la_k > 1);
    int la = 0;
    if (first_step) la |= LA_S_INIT | LA_S_WRITE;
    if (sync) {
        la |= LA_SYNC | LA_S_WRITE;
        if (!first_step) la |= LA_S_READ;
    }
    if (traj) {
        if (!first_of_window) la |= LA_A_READ;
        if (sync) la |= LA_TRAJ; else la |= LA_A_WRITE;
    }
    return la;
}

int64_t round_up(int64_t x, int64_t a) { return (x + a - 1) / a * a; }

// Splits tensors into chunk-table entries; see novak_build_chunks in novak.h.
void build_chunks(const int64_t *numel, const int32_t *phase, int n, int64_t chunk_elems,
                  std::vector<Chunk> &out)
{
    out.clear();
    for (int i = 0; i < n; ++i) {
        int64_t off = 0;
        const int32_t ph = phase ? phase[i] : 0;
        if (ph != 0) {
            const int64_t head = std::min<int64_t>(numel[i], kSlotAlign - ph);
            out.push_back(Chunk{i, static_cast<int32_t>(head), 0});
            off = head;
        }
        while (off < numel[i]) {
            const int64_t len = std::min<int64_t>(chunk_elems, numel[i] - off);
            out.push_back(Chunk{i, static_cast<int32_t>(len), off});
            off += len;
        }
    }
}

// Cuts the tensors that have rows into units of the statistics pass; see
// novak_build_row_units in novak.h and RowUnit.
void build_row_units(const int64_t *numel, const int64_t *rows, int n, std::vector<RowUnit> &out)
{
    out.clear();
    for (int i = 0; i < n; ++i) {
        if (rows[i] <= 0) continue;
        const uint32_t R = static_cast<uint32_t>(rows[i]);
        const uint32_t L = static_cast<uint32_t>(numel[i] / rows[i]);
        if (L > novak::kRowWarpMax) {
            // a CTA per slice of at most kRowUnitElems elements (one slice for most rows)
            const uint32_t parts = (L + novak::kRowUnitElems - 1) / novak::kRowUnitElems;
            for (uint32_t r = 0; r < R; ++r)
                for (uint32_t p = 0; p < parts; ++p) {
                    const uint32_t off = p * novak::kRowUnitElems;
                    out.push_back(RowUnit{i, r, 1u, off, std::min(novak::kRowUnitElems, L - off),
                                          parts, p, 0u});
                }
        } else {
            // a warp per row from 128 elements on (at least one row for each of the
            // CTA's 8 warps), else a thread per row
            // (rows per unit a multiple of 8, so that no warp idles while others take a
            // second row)
            const uint32_t per = L >= 128u ? std::max(8u, novak::kRowUnitElems / L / 8u * 8u)
                                           : novak::kRowUnitThreads;
            for (uint32_t r = 0; r < R; r += per)
                out.push_back(RowUnit{i, r, std::min(per, R - r), 0u, 0u, 1u, 0u, 0u});
        }
    }
}

}  // namespace

struct novak_opt {
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
    int64_t rows_gen = 0;               // bumped whenever the row settings change
    int64_t prep_key = -1;              // rows_gen and centring the scratch was laid out for
    // the averages of Eq. 20-21 live in the scratch; values waiting to be written there
    // a step taken in two halves (novak_step_begin / novak_step_finish)
    bool half_open = false;
    int half_launches = 0;
    alignas(8) unsigned char half_ctx[256] = {};   // the StepCtx of the open step
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

namespace {

int fail(novak_opt *o, int code, const char *fmt, ...)
{
    if (o) {
        char buf[512];
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(buf, sizeof buf, fmt, ap);
        va_end(ap);
        o->err = buf;
    }
    return code;
}

int fail_cuda(novak_opt *o, cudaError_t e, const char *what)
{
    return fail(o, NOVAK_ECUDA, "%s: %s", what, cudaGetErrorString(e));
}

bool in_unit(double x) { return x >= 0.0 && x < 1.0; }  // false for NaN

int n_state_arrays(const Hyper &h)
{
    int a = 2;
    if (h.la_k > 0) a += 1;
    if (h.la_k > 0 && h.la_mode == NOVAK_LOOKAHEAD_TRAJ_MEAN) a += 1;
    return a;
}

float *slice(const novak_opt *o, int array, int i)
{
    return reinterpret_cast<float *>(o->d_state) + array * o->region_elems + o->slot_off[i] +
           o->phase[i];
}

int pre_mode(const novak_opt *o)
{
    if (o->h.centralize && o->total_rows > 0) return novak::PRE_CENTER;
    if (o->h.clip > 0.0 || o->h.auto_lr) return novak::PRE_SCALE;
    return novak::PRE_NONE;
}

void fill_info(const novak_opt *o, const Plan &p, novak_info *out)
{
    std::memset(out, 0, sizeof *out);
    out->t = o->t;
    out->n_syncs = o->n_syncs;
    out->last_sync_step = o->last_sync;
    out->total_numel = o->total_numel;
    out->launches = o->launches;
    out->record_uploads = o->record_uploads;
    out->bc1 = p.bc1; out->bc2 = p.bc2;
    out->rho_inf = p.rho_inf; out->rho_t = p.rho_t;
    out->r_t = p.r_t; out->step_size = p.step_size; out->decay = p.decay;
    out->rect_branch = p.rect_branch; out->is_sync = p.is_sync;
    out->nesterov_variant = o->h.nesterov;
    out->lookahead_mode = o->h.la_mode;
    out->lookahead_k = o->h.la_k;
    out->n_tensors = o->n;
    out->n_chunks = o->n_chunks;
    out->grid = o->last_grid;
    out->block = novak::step_block_threads();
    out->warnings = o->warnings;
    out->grad_processing = pre_mode(o);
    out->layer_adaptation = o->h.layer_adapt;
    out->beta1_t = p.beta1_t;
    out->beta2_t = p.beta2_t;
}

void release_device(novak_opt *o)
{
    if (o->d_chunks) cudaFree(o->d_chunks);
    if (o->d_recs) cudaFree(o->d_recs);
    for (int i = 0; i < kRing; ++i) {
        if (o->h_recs[i]) cudaFreeHost(o->h_recs[i]);
        if (o->ring_ev[i]) cudaEventDestroy(o->ring_ev[i]);
        o->h_recs[i] = nullptr;
        o->ring_ev[i] = nullptr;
    }
    if (o->d_trust) cudaFree(o->d_trust);
    o->d_trust = nullptr;
    o->chunk_u2 = o->chunk_p2 = nullptr;
    o->tensor_first = nullptr;
    o->trust = nullptr;
    if (o->d_prep) cudaFree(o->d_prep);
    o->d_prep = nullptr;
    o->prep_out = nullptr;
    o->part_sq = o->part_sum = o->cta_sq = o->chunk_psq = nullptr;
    o->d_plain = nullptr;
    o->d_units = nullptr;
    o->n_plain = o->n_units = 0;
    o->prep_key = -1;
    o->row_mean = nullptr;
    for (cudaEvent_t ev : o->host_ev) cudaEventDestroy(ev);
    o->host_ev.clear();
    if (o->up_stream) cudaStreamDestroy(o->up_stream);
    if (o->down_stream) cudaStreamDestroy(o->down_stream);
    o->up_stream = o->down_stream = nullptr;
    o->segments.clear();
    o->segments_for = -1;
    o->h_chunks.clear();
    o->d_chunks = nullptr;
    o->d_recs = nullptr;
    o->n_chunks = 0;
    for (auto &tb : o->tables) {
        tb.p.clear();
        tb.g.clear();
        tb.gdtype = -1;
        tb.last_use = 0;
    }
    o->cur_table = -1;
}

// First step: chunk table and record buffers on the device.
int prepare_device(novak_opt *o, cudaStream_t stream)
{
    cudaError_t e;
    int dev = 0;
    if ((e = cudaGetDevice(&dev)) != cudaSuccess) return fail_cuda(o, e, "cudaGetDevice");
    if ((e = cudaDeviceGetAttribute(&o->sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess)
        return fail_cuda(o, e, "cudaDeviceGetAttribute");

    std::vector<Chunk> chunks;
    build_chunks(o->numel.data(), o->phase.data(), o->n, o->chunk_elems, chunks);
    if (chunks.size() > static_cast<size_t>(INT32_MAX)) return fail(o, NOVAK_EINVAL, "too many chunks");

    const size_t cbytes = chunks.size() * sizeof(Chunk);
    const size_t rbytes = static_cast<size_t>(o->n) * sizeof(TensorRec);
    if ((e = cudaMalloc(reinterpret_cast<void **>(&o->d_chunks), cbytes)) != cudaSuccess) {
        release_device(o);
        return fail(o, NOVAK_ENOMEM, "cudaMalloc(chunk table, %zu B): %s", cbytes, cudaGetErrorString(e));
    }
    if ((e = cudaMalloc(reinterpret_cast<void **>(&o->d_recs), rbytes * kRecTables)) != cudaSuccess) {
        release_device(o);
        return fail(o, NOVAK_ENOMEM, "cudaMalloc(tensor records, %zu B): %s", rbytes * kRecTables, cudaGetErrorString(e));
    }
    for (int i = 0; i < kRing; ++i) {
        if ((e = cudaHostAlloc(reinterpret_cast<void **>(&o->h_recs[i]), rbytes, cudaHostAllocDefault)) != cudaSuccess ||
            (e = cudaEventCreateWithFlags(&o->ring_ev[i], cudaEventDisableTiming)) != cudaSuccess) {
            release_device(o);
            return fail(o, NOVAK_ENOMEM, "pinned record ring: %s", cudaGetErrorString(e));
        }
    }
    // The table is built once: a blocking copy keeps the host vector's
    // lifetime trivial.  Ordered before the first launch by the stream sync.
    if ((e = cudaMemcpyAsync(o->d_chunks, chunks.data(), cbytes, cudaMemcpyHostToDevice, stream)) != cudaSuccess ||
        (e = cudaStreamSynchronize(stream)) != cudaSuccess) {
        release_device(o);
        return fail_cuda(o, e, "chunk table upload");
    }
    o->n_chunks = static_cast<int>(chunks.size());
    o->h_chunks.swap(chunks);
    return NOVAK_OK;
}

// Forget which pointer lists the device record tables hold (their contents
// depend on the centralization settings as well as on the pointers).
void invalidate_tables(novak_opt *o)
{
    for (auto &tb : o->tables) {
        tb.p.clear();
        tb.g.clear();
        tb.gdtype = -1;
        tb.last_use = 0;
    }
    o->cur_table = -1;
}

// Scratch of the statistics pass, laid out when a step first needs it and
// again when the row settings change.
int prepare_prep(novak_opt *o, cudaStream_t stream)
{
    const bool centre = o->h.centralize && o->total_rows > 0;
    const int64_t key = o->rows_gen * 2 + (centre ? 1 : 0);
    if (o->d_prep && o->prep_key == key) return NOVAK_OK;
    cudaError_t e;
    if (o->d_prep) {
        // sizes changed: keep the averages of Eq. 20-21 (the copy waits for the device)
        if (!o->ema_pending) {
            PrepOut old;
            if ((e = cudaMemcpy(&old, o->prep_out, sizeof old, cudaMemcpyDeviceToHost)) != cudaSuccess)
                return fail_cuda(o, e, "cudaMemcpy(gradient statistics)");
            o->pending_g_bar = old.g_bar;
            o->pending_theta_bar = old.theta_bar;
            o->ema_pending = true;
        }
        cudaFree(o->d_prep);
        o->d_prep = nullptr;
        invalidate_tables(o);
    }
    // work of the pass: row units for the tensors with rows, chunk-table entries for the rest
    std::vector<RowUnit> units;
    std::vector<Chunk> plain;
    if (centre) {
        build_row_units(o->numel.data(), o->rows.data(), o->n, units);
        for (const Chunk &c : o->h_chunks)
            if (o->rows[c.tensor] <= 0) plain.push_back(c);
    }
    const size_t n_plain = centre ? plain.size() : static_cast<size_t>(o->n_chunks);
    if (units.size() > static_cast<size_t>(INT32_MAX) / 2) return fail(o, NOVAK_EINVAL, "too many rows");
    // sized for fp32 gradients; bf16 gradients take more entries per CTA and need less
    const size_t n_work = static_cast<size_t>(novak::grad_stats_work(
        static_cast<int>(n_plain), static_cast<int>(units.size()), NOVAK_GRAD_F32));
    const size_t nc = static_cast<size_t>(o->n_chunks);
    const size_t ctas = static_cast<size_t>(novak::grad_stats_ctas(static_cast<int>(n_work), o->n_chunks));
    size_t off = 256;
    const size_t off_sq = off;      off += n_work * sizeof(double);
    const size_t off_sum = off;     off += units.size() * sizeof(double);
    const size_t off_psq = off;     off += nc * sizeof(double);
    const size_t off_cta = off;     off += 2 * ctas * sizeof(double);
    off = (off + 15) / 16 * 16;
    const size_t off_plain = off;   off += plain.size() * sizeof(Chunk);
    const size_t off_units = off;   off += units.size() * sizeof(RowUnit);
    const size_t off_mean = off;    off += static_cast<size_t>(o->total_rows) * sizeof(float2);
    const size_t bytes = off + 16;
    if ((e = cudaMalloc(reinterpret_cast<void **>(&o->d_prep), bytes)) != cudaSuccess) {
        o->d_prep = nullptr;
        return fail(o, NOVAK_ENOMEM, "cudaMalloc(gradient statistics, %zu B): %s", bytes, cudaGetErrorString(e));
    }
    if ((e = cudaMemsetAsync(o->d_prep, 0, bytes, stream)) != cudaSuccess)
        return fail_cuda(o, e, "cudaMemsetAsync(gradient statistics)");
    o->prep_out = reinterpret_cast<PrepOut *>(o->d_prep);
    o->part_sq = reinterpret_cast<double *>(o->d_prep + off_sq);
    o->part_sum = reinterpret_cast<double *>(o->d_prep + off_sum);
    o->chunk_psq = reinterpret_cast<double *>(o->d_prep + off_psq);
    o->cta_sq = reinterpret_cast<double *>(o->d_prep + off_cta);
    o->d_plain = centre ? reinterpret_cast<Chunk *>(o->d_prep + off_plain) : nullptr;
    o->d_units = reinterpret_cast<RowUnit *>(o->d_prep + off_units);
    o->row_mean = reinterpret_cast<float2 *>(o->d_prep + off_mean);
    o->n_plain = static_cast<int>(n_plain);
    o->n_units = static_cast<int>(units.size());
    // The tables are built once per layout: blocking copies keep the host
    // vectors' lifetime trivial.
    if (!plain.empty() &&
        (e = cudaMemcpyAsync(o->d_plain, plain.data(), plain.size() * sizeof(Chunk),
                             cudaMemcpyHostToDevice, stream)) != cudaSuccess)
        return fail_cuda(o, e, "statistics table upload");
    if (!units.empty() &&
        (e = cudaMemcpyAsync(o->d_units, units.data(), units.size() * sizeof(RowUnit),
                             cudaMemcpyHostToDevice, stream)) != cudaSuccess)
        return fail_cuda(o, e, "row unit upload");
    if ((e = cudaStreamSynchronize(stream)) != cudaSuccess) return fail_cuda(o, e, "statistics table upload");
    o->prep_key = key;
    invalidate_tables(o);              // records carry pointers into this scratch
    return NOVAK_OK;
}

// Scratch of layer adaptation, allocated when a step first needs it.
int prepare_trust(novak_opt *o, cudaStream_t stream)
{
    if (o->d_trust) return NOVAK_OK;
    const size_t nc = static_cast<size_t>(o->n_chunks), n = static_cast<size_t>(o->n);
    const size_t off_p2 = nc * sizeof(double);
    const size_t off_first = 2 * nc * sizeof(double);
    const size_t off_trust = off_first + (n + 1) * sizeof(int);
    const size_t bytes = off_trust + n * sizeof(float) + 16;
    cudaError_t e;
    if ((e = cudaMalloc(reinterpret_cast<void **>(&o->d_trust), bytes)) != cudaSuccess) {
        o->d_trust = nullptr;
        return fail(o, NOVAK_ENOMEM, "cudaMalloc(layer adaptation, %zu B): %s", bytes, cudaGetErrorString(e));
    }
    o->chunk_u2 = reinterpret_cast<double *>(o->d_trust);
    o->chunk_p2 = reinterpret_cast<double *>(o->d_trust + off_p2);
    o->tensor_first = reinterpret_cast<int *>(o->d_trust + off_first);
    o->trust = reinterpret_cast<float *>(o->d_trust + off_trust);
    // the table lists a tensor's entries consecutively, tensors in order
    o->h_tensor_first.assign(n + 1, o->n_chunks);
    for (int c = o->n_chunks - 1; c >= 0; --c) o->h_tensor_first[o->h_chunks[c].tensor] = c;
    if ((e = cudaMemcpyAsync(o->tensor_first, o->h_tensor_first.data(), (n + 1) * sizeof(int),
                             cudaMemcpyHostToDevice, stream)) != cudaSuccess ||
        (e = cudaStreamSynchronize(stream)) != cudaSuccess)
        return fail_cuda(o, e, "layer adaptation table upload");
    return NOVAK_OK;
}

uint64_t hash_pointers(void *const *d_params, const void *const *d_grads, int n, int grad_dtype)
{
    uint64_t h = 0xcbf29ce484222325ull ^ static_cast<uint64_t>(grad_dtype);
    for (int i = 0; i < n; ++i) {
        h = (h ^ reinterpret_cast<uintptr_t>(d_params[i])) * 0x100000001b3ull;
        h = (h ^ reinterpret_cast<uintptr_t>(d_grads[i])) * 0x100000001b3ull;
    }
    return h;
}

// Selects the device record table that holds the caller's pointer lists,
// uploading them (in stream order, into the least recently used table) when
// none does.
int refresh_records(novak_opt *o, void *const *d_params, const void *const *d_grads,
                    int grad_dtype, cudaStream_t stream)
{
    const int n = o->n;
    const uint64_t hash = hash_pointers(d_params, d_grads, n, grad_dtype);
    int lru = 0;
    for (int k = 0; k < kRecTables; ++k) {
        novak_opt::RecTable &tb = o->tables[k];
        if (tb.gdtype == grad_dtype && tb.hash == hash && !tb.p.empty() &&
            std::memcmp(tb.p.data(), d_params, n * sizeof(void *)) == 0 &&
            std::memcmp(tb.g.data(), d_grads, n * sizeof(void *)) == 0) {
            tb.last_use = ++o->table_clock;
            o->cur_table = k;
            return NOVAK_OK;
        }
        if (tb.last_use < o->tables[lru].last_use) lru = k;
    }

    const uintptr_t gmask = grad_dtype == NOVAK_GRAD_BF16 ? 1u : 3u;
    const uintptr_t gvec = grad_dtype == NOVAK_GRAD_BF16 ? 8u : 16u;
    bool scalar_path = false;
    for (int i = 0; i < n; ++i) {
        const uintptr_t p = reinterpret_cast<uintptr_t>(d_params[i]);
        const uintptr_t g = reinterpret_cast<uintptr_t>(d_grads[i]);
        if (!p || !g) return fail(o, NOVAK_EINVAL, "tensor %d: NULL pointer", i);
        if ((p & 3u) || (g & gmask)) return fail(o, NOVAK_EINVAL, "tensor %d: pointer not aligned to its element size", i);
        // 128-bit path needs parameter, state and gradient congruent mod 16 B.
        const uintptr_t m = reinterpret_cast<uintptr_t>(slice(o, 0, i));
        if (((p ^ m) & 15u) || (((p & 15u) / 4u) != ((g % gvec) / (gvec / 4u))) || (g % (gvec / 4u)))
            scalar_path = true;
        // the bf16 copy is stored 4 elements (8 bytes) at a time beside 16-byte parameters
        if (!o->copies.empty() &&
            ((p & 15u) >> 1) != (reinterpret_cast<uintptr_t>(o->copies[i]) & 7u))
            scalar_path = true;
    }
    const int slot = o->ring_pos;
    cudaError_t e;
    if ((e = cudaEventSynchronize(o->ring_ev[slot])) != cudaSuccess)
        return fail_cuda(o, e, "cudaEventSynchronize(record ring)");
    TensorRec *h = o->h_recs[slot];
    const bool la = o->h.la_k > 0;
    const bool traj = la && o->h.la_mode == NOVAK_LOOKAHEAD_TRAJ_MEAN;
    for (int i = 0; i < n; ++i) {
        h[i].p = static_cast<float *>(d_params[i]);
        h[i].g = d_grads[i];
        h[i].m = slice(o, 0, i);
        h[i].v = slice(o, 1, i);
        h[i].slow = la ? slice(o, 2, i) : nullptr;
        h[i].acc = traj ? slice(o, 3, i) : nullptr;
        const bool rows = o->h.centralize && o->row_mean && !o->rows.empty() && o->rows[i] > 0;
        h[i].mean = rows ? o->row_mean + o->row_off[i] : nullptr;
        h[i].row_len = rows ? static_cast<uint32_t>(o->numel[i] / o->rows[i]) : 0u;
        h[i].p16 = o->copies.empty() ? nullptr : static_cast<__nv_bfloat16 *>(o->copies[i]);
        h[i].reserved = 0;
    }
    // Stream order puts this copy behind every earlier launch that read the
    // table being replaced.
    novak_opt::RecTable &tb = o->tables[lru];
    tb.p.clear();
    if ((e = cudaMemcpyAsync(o->d_recs + static_cast<size_t>(lru) * n, h, n * sizeof(TensorRec),
                             cudaMemcpyHostToDevice, stream)) != cudaSuccess)
        return fail_cuda(o, e, "tensor record upload");
    if ((e = cudaEventRecord(o->ring_ev[slot], stream)) != cudaSuccess)
        return fail_cuda(o, e, "cudaEventRecord(record ring)");
    o->ring_pos = (slot + 1) % kRing;
    tb.p.assign(d_params, d_params + n);
    tb.g.assign(d_grads, d_grads + n);
    tb.gdtype = grad_dtype;
    tb.hash = hash;
    tb.last_use = ++o->table_clock;
    o->cur_table = lru;
    o->record_uploads += 1;
    if (scalar_path) o->warnings |= NOVAK_WARN_SCALAR_PATH;
    return NOVAK_OK;
}

int check_hyper(const Hyper &h, const char **why)
{
    *why = "";
    if (!(h.lr > 0.0) || !std::isfinite(h.lr)) { *why = "lr must be > 0"; return 0; }
    if (!in_unit(h.beta1)) { *why = "beta1 must be in [0,1)"; return 0; }
    if (!in_unit(h.beta2)) { *why = "beta2 must be in [0,1)"; return 0; }
    if (!(h.beta2 < 1.0 - 1e-8)) { *why = "beta2 must be < 1 - 1e-8 (rho_inf)"; return 0; }
    if (!(h.eps > 0.0) || !std::isfinite(h.eps)) { *why = "eps must be > 0"; return 0; }
    if (!(h.wd >= 0.0) || !std::isfinite(h.wd)) { *why = "weight_decay must be >= 0"; return 0; }
    if (!in_unit(h.beta_n)) { *why = "nesterov beta must be in [0,1)"; return 0; }
    if (h.nesterov < NOVAK_NESTEROV_NONE || h.nesterov > NOVAK_NESTEROV_CLASSICAL) { *why = "unknown nesterov_variant"; return 0; }
    if (h.la_k < 0) { *why = "lookahead_k must be >= 0"; return 0; }
    if (h.la_k > 0 && !(h.la_alpha > 0.0 && h.la_alpha < 1.0)) { *why = "lookahead_alpha must be in (0,1)"; return 0; }
    if (h.la_mode != NOVAK_LOOKAHEAD_LAST && h.la_mode != NOVAK_LOOKAHEAD_TRAJ_MEAN) { *why = "unknown lookahead mode"; return 0; }
    if (h.bias1_power != 1 && h.bias1_power != 2) { *why = "bias1_power must be 1 or 2"; return 0; }
    if (!(h.clip >= 0.0) || !std::isfinite(h.clip)) { *why = "clip threshold must be >= 0"; return 0; }
    if (h.centralize != 0 && h.centralize != 1) { *why = "centralize must be 0 or 1"; return 0; }
    if (h.auto_lr != 0 && h.auto_lr != 1) { *why = "auto_lr must be 0 or 1"; return 0; }
    if (!(h.auto_gamma > 0.0 && h.auto_gamma <= 1.0)) { *why = "auto_lr gamma must be in (0, 1]"; return 0; }
    if (!(h.sparse_tau >= 0.0) || !std::isfinite(h.sparse_tau)) { *why = "sparse threshold must be >= 0"; return 0; }
    if (h.layer_adapt != 0 && h.layer_adapt != 1) { *why = "layer_adaptation must be 0 or 1"; return 0; }
    if (h.adaptive_beta != 0 && h.adaptive_beta != 1) { *why = "adaptive_beta must be 0 or 1"; return 0; }
    if (!(h.tau1 > 0.0) || !std::isfinite(h.tau1) || !(h.tau2 > 0.0) || !std::isfinite(h.tau2)) { *why = "warm-up time scales must be > 0"; return 0; }
    return 1;
}

}  // namespace

extern "C" {

int novak_create(novak_opt **out, double lr, double beta1, double beta2, double eps,
                 double weight_decay, int nesterov_variant, int lookahead_k,
                 double lookahead_alpha)
{
    if (!out) return NOVAK_EINVAL;
    *out = nullptr;
    Hyper h{};
    h.lr = lr; h.beta1 = beta1; h.beta2 = beta2; h.eps = eps; h.wd = weight_decay;
    h.beta_n = beta1;
    h.la_alpha = lookahead_alpha;
    h.la_k = lookahead_k;
    h.la_mode = NOVAK_LOOKAHEAD_LAST;
    h.rectified = 1;
    h.bias1_power = 1;
    h.clip = 0.0;
    h.centralize = 0;
    h.layer_adapt = 0;
    h.sparse_tau = 0.0;
    h.auto_lr = 0;
    h.auto_gamma = 0.1;    // Section 4.6
    h.adaptive_beta = 0;
    h.tau1 = 1000.0;       // Section 4.2's values
    h.tau2 = 5000.0;
    uint32_t warn = 0;
    h.nesterov = nesterov_variant;
    if (nesterov_variant == NOVAK_NESTEROV_TRUE) {
        h.nesterov = NOVAK_NESTEROV_APPROX;  // no closure on this path: downgrade, warn
        warn |= NOVAK_WARN_TRUE_DOWNGRADED;
    }
    const char *why;
    if (!check_hyper(h, &why)) return NOVAK_EINVAL;
    novak_opt *o = new (std::nothrow) novak_opt();
    if (!o) return NOVAK_ENOMEM;
    o->h = h;
    o->warnings = warn;
    o->last_plan = make_plan(h, 1);
    *out = o;
    return NOVAK_OK;
}

void novak_destroy(novak_opt *opt)
{
    if (!opt) return;
    release_device(opt);
    delete opt;
}

int novak_set_option(novak_opt *o, int key, double value)
{
    if (!o) return NOVAK_EINVAL;
    Hyper h = o->h;
    const char *why = "";
    switch (key) {
    case NOVAK_OPT_NESTEROV_BETA: h.beta_n = value; break;
    case NOVAK_OPT_LOOKAHEAD_MODE:
        if (o->attached) return fail(o, NOVAK_ESTATE, "lookahead mode changes the state layout: set it before attach");
        if (value != 0.0 && value != 1.0) return fail(o, NOVAK_EINVAL, "unknown lookahead mode");
        h.la_mode = static_cast<int>(value);
        break;
    case NOVAK_OPT_RECTIFIED:
        if (value != 0.0 && value != 1.0) return fail(o, NOVAK_EINVAL, "rectified must be 0 or 1");
        h.rectified = static_cast<int>(value);
        break;
    case NOVAK_OPT_LR: h.lr = value; break;
    case NOVAK_OPT_WEIGHT_DECAY: h.wd = value; break;
    case NOVAK_OPT_BIAS1_POWER:
        if (value != 1.0 && value != 2.0) return fail(o, NOVAK_EINVAL, "bias1_power must be 1 or 2");
        h.bias1_power = static_cast<int>(value);
        break;
    case NOVAK_OPT_SPARSE_THRESHOLD: h.sparse_tau = value; break;
    case NOVAK_OPT_AUTO_LR:
        if (value != 0.0 && value != 1.0) return fail(o, NOVAK_EINVAL, "auto_lr must be 0 or 1");
        h.auto_lr = static_cast<int>(value);
        break;
    case NOVAK_OPT_AUTO_LR_GAMMA: h.auto_gamma = value; break;
    case NOVAK_OPT_LAYER_ADAPTATION:
        if (value != 0.0 && value != 1.0) return fail(o, NOVAK_EINVAL, "layer_adaptation must be 0 or 1");
        h.layer_adapt = static_cast<int>(value);
        break;
    case NOVAK_OPT_ADAPTIVE_BETA:
        if (value != 0.0 && value != 1.0) return fail(o, NOVAK_EINVAL, "adaptive_beta must be 0 or 1");
        h.adaptive_beta = static_cast<int>(value);
        break;
    case NOVAK_OPT_BETA1_TAU: h.tau1 = value; break;
    case NOVAK_OPT_BETA2_TAU: h.tau2 = value; break;
    case NOVAK_OPT_CLIP_THRESHOLD: h.clip = value; break;
    case NOVAK_OPT_CENTRALIZE:
        if (value != 0.0 && value != 1.0) return fail(o, NOVAK_EINVAL, "centralize must be 0 or 1");
        if (h.centralize != static_cast<int>(value)) invalidate_tables(o);
        h.centralize = static_cast<int>(value);
        break;
    case NOVAK_OPT_CHUNK_ELEMS: {
        if (o->d_chunks || !o->na_chunks.empty())
            return fail(o, NOVAK_ESTATE, "chunk size is fixed once a step was taken");
        const int64_t c = static_cast<int64_t>(value);
        if (!(value >= 1024.0 && value <= 16777216.0) || c % 1024 != 0 || static_cast<double>(c) != value)
            return fail(o, NOVAK_EINVAL, "chunk_elems must be a multiple of 1024 in [1024, 2^24]");
        o->chunk_elems = c;
        return NOVAK_OK;
    }
    case NOVAK_OPT_CTAS_PER_SM:
        if (o->d_chunks) return fail(o, NOVAK_ESTATE, "grid policy is fixed once a step was taken");
        if (!(value >= 0.0 && value <= 32.0) || value != std::floor(value))
            return fail(o, NOVAK_EINVAL, "ctas_per_sm must be an integer in [0, 32]");
        o->ctas_per_sm = static_cast<int>(value);
        return NOVAK_OK;
    case NOVAK_OPT_SERPENTINE:
        if (value != 0.0 && value != 1.0) return fail(o, NOVAK_EINVAL, "serpentine must be 0 or 1");
        o->serpentine = static_cast<int>(value);
        return NOVAK_OK;
    case NOVAK_OPT_DEPENDENT_LAUNCH:
        if (!(value >= 0.0 && value <= 7.0) || value != std::floor(value))
            return fail(o, NOVAK_EINVAL, "dependent_launch must be an integer in [0, 7]");
        o->pdl = static_cast<int>(value);
        return NOVAK_OK;
    case NOVAK_OPT_HOST_SEGMENT_ELEMS:
        if (!(value >= 0.0 && value <= 4294967296.0) || value != std::floor(value))
            return fail(o, NOVAK_EINVAL, "host_segment_elems must be an integer in [0, 2^32]");
        o->host_segment_elems = static_cast<int64_t>(value);
        return NOVAK_OK;
    default:
        return fail(o, NOVAK_EINVAL, "unknown option key %d", key);
    }
    if (!check_hyper(h, &why)) return fail(o, NOVAK_EINVAL, "%s", why);
    o->h = h;
    return NOVAK_OK;
}

int novak_get_option(const novak_opt *o, int key, double *value)
{
    if (!o || !value) return NOVAK_EINVAL;
    switch (key) {
    case NOVAK_OPT_NESTEROV_BETA: *value = o->h.beta_n; break;
    case NOVAK_OPT_LOOKAHEAD_MODE: *value = o->h.la_mode; break;
    case NOVAK_OPT_RECTIFIED: *value = o->h.rectified; break;
    case NOVAK_OPT_LR: *value = o->h.lr; break;
    case NOVAK_OPT_WEIGHT_DECAY: *value = o->h.wd; break;
    case NOVAK_OPT_BIAS1_POWER: *value = o->h.bias1_power; break;
    case NOVAK_OPT_SPARSE_THRESHOLD: *value = o->h.sparse_tau; break;
    case NOVAK_OPT_AUTO_LR: *value = o->h.auto_lr; break;
    case NOVAK_OPT_AUTO_LR_GAMMA: *value = o->h.auto_gamma; break;
    case NOVAK_OPT_LAYER_ADAPTATION: *value = o->h.layer_adapt; break;
    case NOVAK_OPT_ADAPTIVE_BETA: *value = o->h.adaptive_beta; break;
    case NOVAK_OPT_BETA1_TAU: *value = o->h.tau1; break;
    case NOVAK_OPT_BETA2_TAU: *value = o->h.tau2; break;
    case NOVAK_OPT_CLIP_THRESHOLD: *value = o->h.clip; break;
    case NOVAK_OPT_CENTRALIZE: *value = o->h.centralize; break;
    case NOVAK_OPT_CHUNK_ELEMS: *value = static_cast<double>(o->chunk_elems); break;
    case NOVAK_OPT_CTAS_PER_SM: *value = o->ctas_per_sm; break;
    case NOVAK_OPT_SERPENTINE: *value = o->serpentine; break;
    case NOVAK_OPT_DEPENDENT_LAUNCH: *value = o->pdl; break;
    case NOVAK_OPT_HOST_SEGMENT_ELEMS: *value = static_cast<double>(o->host_segment_elems); break;
    default: return NOVAK_EINVAL;
    }
    return NOVAK_OK;
}

size_t novak_state_bytes(const novak_opt *o, const int64_t *numel, int n)
{
    if (!o || !numel || n <= 0) return 0;
    int64_t region = 0;
    for (int i = 0; i < n; ++i) {
        if (numel[i] <= 0) return 0;
        region += round_up(numel[i] + kSlotAlign - 1, kSlotAlign);
    }
    return static_cast<size_t>(region) * sizeof(float) * n_state_arrays(o->h);
}

int novak_attach_state(novak_opt *o, void *d_state, size_t bytes, void *const *d_params,
                       const int64_t *numel, int n, void *stream)
{
    if (!o) return NOVAK_EINVAL;
    if (!d_state || !numel || n <= 0) return fail(o, NOVAK_EINVAL, "attach: NULL buffer or empty tensor list");
    if (reinterpret_cast<uintptr_t>(d_state) & 255u) return fail(o, NOVAK_EINVAL, "attach: state buffer must be 256-byte aligned");
    const size_t need = novak_state_bytes(o, numel, n);
    if (need == 0) return fail(o, NOVAK_EINVAL, "attach: every numel must be > 0");
    if (bytes < need) return fail(o, NOVAK_EINVAL, "attach: state buffer has %zu B, needs %zu B", bytes, need);
    std::vector<int32_t> phase(n, 0);
    if (d_params) {
        for (int i = 0; i < n; ++i) {
            const uintptr_t p = reinterpret_cast<uintptr_t>(d_params[i]);
            if (!p || (p & 3u)) return fail(o, NOVAK_EINVAL, "attach: parameter %d is NULL or not 4-byte aligned", i);
            phase[i] = static_cast<int32_t>((p % (kSlotAlign * 4)) / 4);
        }
    }
    cudaError_t e = cudaMemsetAsync(d_state, 0, need, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return fail_cuda(o, e, "cudaMemsetAsync(state)");

    release_device(o);
    o->na_chunks.clear();
    o->na_p.clear();
    o->na_token = 0;
    o->d_state = static_cast<char *>(d_state);
    o->n = n;
    o->n_arrays = n_state_arrays(o->h);
    o->numel.assign(numel, numel + n);
    o->phase = phase;
    o->slot_off.resize(n);
    int64_t off = 0, total = 0;
    for (int i = 0; i < n; ++i) {
        o->slot_off[i] = off;
        off += round_up(numel[i] + kSlotAlign - 1, kSlotAlign);
        total += numel[i];
    }
    o->region_elems = off;
    o->total_numel = total;
    o->rows.assign(n, 0);
    o->row_off.assign(n, 0);
    o->total_rows = 0;
    o->copies.clear();
    o->half_open = false;
    o->ema_pending = false;
    o->t = 0; o->n_syncs = 0; o->last_sync = 0;
    o->attached = true;
    o->err.clear();
    return NOVAK_OK;
}

}  // extern "C"

namespace {

StepScalars make_scalars(const Hyper &h, const Plan &p)
{
    StepScalars s;
    s.beta1 = static_cast<float>(p.beta1_t);
    s.omb1 = static_cast<float>(1.0 - p.beta1_t);
    s.beta2 = static_cast<float>(p.beta2_t);
    s.omb2 = static_cast<float>(1.0 - p.beta2_t);
    s.blend_b1 = static_cast<float>(h.beta1);
    s.blend_omb1 = static_cast<float>(1.0 - h.beta1);
    s.beta_n = static_cast<float>(h.beta_n);
    s.inv_bc1 = static_cast<float>(1.0 / p.bc1);
    s.inv_bc2 = static_cast<float>(1.0 / p.bc2);
    s.eps = static_cast<float>(h.eps);
    s.decay = static_cast<float>(p.decay);
    s.step = static_cast<float>(p.step_size);
    s.la_alpha = static_cast<float>(h.la_alpha);
    s.k = static_cast<float>(h.la_k > 0 ? h.la_k : 1);
    s.sparse_tau = h.sparse_tau > 0.0 ? static_cast<float>(h.sparse_tau) : -1.0f;
    return s;
}

// Everything one step needs, fixed before anything is enqueued.
struct StepCtx {
    int64_t t;
    Plan plan;
    int la;
    int grad_dtype;
    StepScalars s;
    const TensorRec *d_recs;
    int reverse;
    int pre;                 // novak::PRE_*
    const float *trust;      // per-tensor factors of Eq. 25, NULL without layer adaptation
};

int check_step_args(novak_opt *o, const char *who, void *const *d_params,
                    const void *const *d_grads, const int64_t *numel, int n, int grad_dtype)
{
    if (!o->attached) return fail(o, NOVAK_ESTATE, "%s: no state attached", who);
    if (o->half_open && std::strcmp(who, "step_begin") != 0)
        return fail(o, NOVAK_ESTATE, "%s: a step begun with novak_step_begin is still open", who);
    if (!d_params || !d_grads || !numel) return fail(o, NOVAK_EINVAL, "%s: NULL argument", who);
    if (grad_dtype != NOVAK_GRAD_F32 && grad_dtype != NOVAK_GRAD_BF16)
        return fail(o, NOVAK_EINVAL, "%s: unknown grad_dtype %d", who, grad_dtype);
    if (n != o->n || std::memcmp(numel, o->numel.data(), n * sizeof(int64_t)) != 0)
        return fail(o, NOVAK_ESTATE, "%s: tensor list differs from the attached layout", who);
    return NOVAK_OK;
}

// Work table on the device, records for these pointers, the scalar plan of step t+1.
int begin_step(novak_opt *o, void *const *d_params, const void *const *d_grads, int grad_dtype,
               cudaStream_t stream, StepCtx *ctx)
{
    int rc;
    if (!o->d_chunks && (rc = prepare_device(o, stream)) != NOVAK_OK) return rc;
    ctx->pre = pre_mode(o);
    if (ctx->pre != novak::PRE_NONE && (rc = prepare_prep(o, stream)) != NOVAK_OK) return rc;
    if (o->ema_pending && o->prep_out) {
        // averages set by the caller (or saved over a reallocation) go into the scratch
        const double ema[2] = {o->pending_g_bar, o->pending_theta_bar};
        cudaError_t e = cudaMemcpyAsync(&o->prep_out->g_bar, ema, sizeof ema, cudaMemcpyHostToDevice, stream);
        if (e != cudaSuccess) return fail_cuda(o, e, "upload of the auto-LR averages");
        o->ema_pending = false;
    }
    if (o->h.layer_adapt && (rc = prepare_trust(o, stream)) != NOVAK_OK) return rc;
    ctx->trust = o->h.layer_adapt ? o->trust : nullptr;
    if ((rc = refresh_records(o, d_params, d_grads, grad_dtype, stream)) != NOVAK_OK) return rc;
    ctx->t = o->t + 1;
    ctx->plan = make_plan(o->h, ctx->t);
    ctx->la = lookahead_action(o->h, ctx->t);
    ctx->grad_dtype = grad_dtype;
    ctx->s = make_scalars(o->h, ctx->plan);
    ctx->d_recs = o->d_recs + static_cast<size_t>(o->cur_table) * o->n;
    ctx->reverse = (o->serpentine && (ctx->t % 2 == 0)) ? 1 : 0;
    // After a statistics pass the END of the gradient is what L2 still holds:
    // the step kernel then walks the table from the end.
    if (ctx->pre != novak::PRE_NONE || ctx->trust) ctx->reverse = 1;
    return NOVAK_OK;
}

// Everything that has to see the whole group before the first element is
// updated: phase 2's statistics, then phase 7's trust ratios.  Returns the
// number of kernels launched through *launches.
cudaError_t launch_stats(novak_opt *o, const StepCtx &ctx, bool finalize, cudaStream_t stream);
cudaError_t launch_statistics(novak_opt *o, const StepCtx &ctx, bool finalize, cudaStream_t stream,
                              int *launches, const char **what)
{
    if (ctx.pre == novak::PRE_NONE) return cudaSuccess;
    *what = "gradient statistics kernel launch";
    const cudaError_t e = launch_stats(o, ctx, finalize, stream);
    if (e == cudaSuccess) *launches += o->h.auto_lr ? 3 : 2;
    return e;
}

cudaError_t launch_trust(novak_opt *o, const StepCtx &ctx, cudaStream_t stream, int *launches,
                         const char **what)
{
    cudaError_t e;
    if (ctx.trust) {
        *what = "layer adaptation kernel launch";
        e = novak::launch_trust_stats(o->d_chunks, o->n_chunks, ctx.d_recs, o->n, o->tensor_first,
                                      o->prep_out, ctx.s, o->h.nesterov, ctx.grad_dtype, ctx.pre,
                                      o->chunk_u2, o->chunk_p2, o->trust, o->pdl, stream);
        if (e != cudaSuccess) return e;
        *launches += 2;
    }
    return cudaSuccess;
}

cudaError_t launch_prepasses(novak_opt *o, const StepCtx &ctx, cudaStream_t stream, int *launches,
                             const char **what)
{
    const cudaError_t e = launch_statistics(o, ctx, true, stream, launches, what);
    return e != cudaSuccess ? e : launch_trust(o, ctx, stream, launches, what);
}

// Phase 2's statistics pass over the whole group: global norm, clip factor, row means.
cudaError_t launch_stats(novak_opt *o, const StepCtx &ctx, bool finalize, cudaStream_t stream)
{
    novak::StatsPlan plan;
    plan.plain = o->d_plain ? o->d_plain : o->d_chunks;
    plan.n_plain = o->n_plain;
    plan.units = o->d_units;
    plan.n_units = o->n_units;
    plan.recs = ctx.d_recs;
    plan.chunks = o->d_chunks;
    plan.n_chunks = o->n_chunks;
    plan.part_sq = o->part_sq;
    plan.part_sum = o->part_sum;
    plan.chunk_psq = o->chunk_psq;
    plan.cta_sq = o->cta_sq;
    plan.prep = o->prep_out;
    return novak::launch_grad_stats(plan, ctx.grad_dtype, o->h.clip,
                                    o->h.auto_lr ? o->h.auto_gamma : 0.0, finalize, o->pdl, stream);
}

// One launch over chunk-table entries [c0, c1).
cudaError_t launch_range(novak_opt *o, const StepCtx &ctx, int c0, int c1, cudaStream_t stream)
{
    novak::LaunchCfg cfg;
    const int count = c1 - c0;
    cfg.grid = count;
    if (o->ctas_per_sm > 0) cfg.grid = std::min(count, o->sms * o->ctas_per_sm);
    cfg.reverse = ctx.reverse;
    cfg.pdl = o->pdl;
    cfg.pre = ctx.pre | (o->copies.empty() ? 0 : novak::PRE_COPY16);
    o->last_grid = cfg.grid;
    return novak::launch_step(o->d_chunks + c0, count, ctx.d_recs, o->prep_out, ctx.trust, ctx.s,
                              o->h.nesterov, ctx.grad_dtype, ctx.la, cfg, stream);
}

void commit_step(novak_opt *o, const StepCtx &ctx, int launches)
{
    o->t = ctx.t;
    o->launches += launches;
    o->last_plan = ctx.plan;
    if (ctx.plan.is_sync) { o->n_syncs += 1; o->last_sync = ctx.t; }
}

// Cuts the chunk table into runs of about host_segment_elems elements and lists,
// per run, the element ranges of the tensors it covers.
void build_segments(novak_opt *o)
{
    o->segments.clear();
    o->segments_for = o->host_segment_elems;
    int64_t want = o->host_segment_elems;
    if (want <= 0) want = INT64_MAX;
    else want = std::max<int64_t>(want, (o->total_numel + kMaxHostSegments - 1) / kMaxHostSegments);
    novak_opt::Segment seg{0, 0, {}};
    int64_t have = 0;
    auto add = [&](const Chunk &c) {
        if (!seg.ranges.empty() && seg.ranges.back().tensor == c.tensor &&
            seg.ranges.back().off + seg.ranges.back().len == c.offset)
            seg.ranges.back().len += c.len;
        else
            seg.ranges.push_back({c.tensor, c.offset, c.len});
    };
    for (int c = 0; c < o->n_chunks; ++c) {
        add(o->h_chunks[c]);
        have += o->h_chunks[c].len;
        seg.c1 = c + 1;
        if (have >= want && c + 1 < o->n_chunks) {
            o->segments.push_back(seg);
            seg = novak_opt::Segment{c + 1, c + 1, {}};
            have = 0;
        }
    }
    o->segments.push_back(seg);
}

int prepare_host_pipeline(novak_opt *o)
{
    cudaError_t e;
    if (!o->up_stream &&
        (e = cudaStreamCreateWithFlags(&o->up_stream, cudaStreamNonBlocking)) != cudaSuccess)
        return fail_cuda(o, e, "cudaStreamCreate(upload)");
    if (!o->down_stream &&
        (e = cudaStreamCreateWithFlags(&o->down_stream, cudaStreamNonBlocking)) != cudaSuccess)
        return fail_cuda(o, e, "cudaStreamCreate(download)");
    const size_t need = 2 + 2 * o->segments.size();
    while (o->host_ev.size() < need) {
        cudaEvent_t ev;
        if ((e = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming)) != cudaSuccess)
            return fail_cuda(o, e, "cudaEventCreate(host pipeline)");
        o->host_ev.push_back(ev);
    }
    return NOVAK_OK;
}

// Copies the ranges of one segment between host and device tensors, merging
// ranges that are adjacent on both sides into one copy.
cudaError_t copy_ranges(const novak_opt::Segment &seg, void *const *dst, const void *const *src,
                        size_t elem_bytes, cudaMemcpyKind kind, cudaStream_t stream)
{
    size_t i = 0;
    const size_t n = seg.ranges.size();
    while (i < n) {
        const novak_opt::Range &r = seg.ranges[i];
        char *d = static_cast<char *>(dst[r.tensor]) + r.off * elem_bytes;
        const char *sr = static_cast<const char *>(src[r.tensor]) + r.off * elem_bytes;
        size_t bytes = static_cast<size_t>(r.len) * elem_bytes;
        size_t j = i + 1;
        while (j < n) {
            const novak_opt::Range &q = seg.ranges[j];
            if (static_cast<char *>(dst[q.tensor]) + q.off * elem_bytes != d + bytes ||
                static_cast<const char *>(src[q.tensor]) + q.off * elem_bytes != sr + bytes)
                break;
            bytes += static_cast<size_t>(q.len) * elem_bytes;
            ++j;
        }
        const cudaError_t e = cudaMemcpyAsync(d, sr, bytes, kind, stream);
        if (e != cudaSuccess) return e;
        i = j;
    }
    return cudaSuccess;
}

}  // namespace

extern "C" {

int novak_step(novak_opt *o, void *const *d_params, const void *const *d_grads,
               const int64_t *numel, int n, int grad_dtype, void *stream_)
{
    if (!o) return NOVAK_EINVAL;
    int rc = check_step_args(o, "step", d_params, d_grads, numel, n, grad_dtype);
    if (rc != NOVAK_OK) return rc;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    StepCtx ctx;
    if ((rc = begin_step(o, d_params, d_grads, grad_dtype, stream, &ctx)) != NOVAK_OK) return rc;
    cudaError_t e;
    int launches = 1;
    const char *what = "";
    if ((e = launch_prepasses(o, ctx, stream, &launches, &what)) != cudaSuccess)
        return fail_cuda(o, e, what);
    if ((e = launch_range(o, ctx, 0, o->n_chunks, stream)) != cudaSuccess)
        return fail_cuda(o, e, "step kernel launch");
    commit_step(o, ctx, launches);
    return NOVAK_OK;
}

int novak_step_begin(novak_opt *o, void *const *d_params, const void *const *d_grads,
                     const int64_t *numel, int n, int grad_dtype, void *stream_)
{
    static_assert(sizeof(StepCtx) <= sizeof(o->half_ctx), "room for the open step");
    if (!o) return NOVAK_EINVAL;
    int rc = check_step_args(o, "step_begin", d_params, d_grads, numel, n, grad_dtype);
    if (rc != NOVAK_OK) return rc;
    if (o->half_open) return fail(o, NOVAK_ESTATE, "step_begin: the previous step was not finished");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    StepCtx ctx;
    if ((rc = begin_step(o, d_params, d_grads, grad_dtype, stream, &ctx)) != NOVAK_OK) return rc;
    if (ctx.pre == novak::PRE_CENTER || ctx.trust)
        return fail(o, NOVAK_ESTATE, "step_begin: centralization and layer adaptation need whole "
                    "tensors and are not available for a group cut across processes");
    int launches = 0;
    const char *what = "";
    const cudaError_t e = launch_statistics(o, ctx, false, stream, &launches, &what);
    if (e != cudaSuccess) return fail_cuda(o, e, what);
    std::memcpy(o->half_ctx, &ctx, sizeof ctx);
    o->half_launches = launches;
    o->half_open = true;
    return NOVAK_OK;
}

int novak_local_sums(novak_opt *o, double **d_sums)
{
    if (!o || !d_sums) return NOVAK_EINVAL;
    if (!o->half_open) return fail(o, NOVAK_ESTATE, "local_sums: no step is open");
    *d_sums = o->prep_out ? o->prep_out->local_sums : nullptr;
    return NOVAK_OK;
}

int novak_copy_local_sums(novak_opt *o, double *d_dst, void *stream_)
{
    if (!o || !d_dst) return NOVAK_EINVAL;
    if (!o->half_open) return fail(o, NOVAK_ESTATE, "copy_local_sums: no step is open");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    cudaError_t e;
    if (o->prep_out)
        e = cudaMemcpyAsync(d_dst, o->prep_out->local_sums, 2 * sizeof(double),
                            cudaMemcpyDeviceToDevice, stream);
    else
        e = cudaMemsetAsync(d_dst, 0, 2 * sizeof(double), stream);   // no statistics: nothing to add
    if (e != cudaSuccess) return fail_cuda(o, e, "copy_local_sums");
    return NOVAK_OK;
}

int novak_step_finish(novak_opt *o, const double *d_total_sums, void *stream_)
{
    if (!o) return NOVAK_EINVAL;
    if (!o->half_open) return fail(o, NOVAK_ESTATE, "step_finish: no step is open");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    StepCtx ctx;
    std::memcpy(&ctx, o->half_ctx, sizeof ctx);
    int launches = o->half_launches + 1;
    cudaError_t e;
    if (ctx.pre != novak::PRE_NONE) {
        const double *totals = d_total_sums ? d_total_sums : o->prep_out->local_sums;
        e = novak::launch_grad_norm_scalars(o->prep_out, totals, o->h.clip,
                                            o->h.auto_lr ? o->h.auto_gamma : 0.0, o->pdl, stream);
        if (e != cudaSuccess) return fail_cuda(o, e, "gradient norm kernel launch");
        ++launches;
    }
    if ((e = launch_range(o, ctx, 0, o->n_chunks, stream)) != cudaSuccess)
        return fail_cuda(o, e, "step kernel launch");
    o->half_open = false;
    commit_step(o, ctx, launches);
    return NOVAK_OK;
}

int novak_step_host(novak_opt *o, void *const *h_params, const void *const *h_grads,
                    void *const *d_params, void *const *d_grads, const int64_t *numel, int n,
                    int grad_dtype, void *stream_)
{
    if (!o) return NOVAK_EINVAL;
    if (!h_params || !h_grads) return fail(o, NOVAK_EINVAL, "step_host: NULL argument");
    int rc = check_step_args(o, "step_host", d_params, const_cast<const void *const *>(d_grads),
                             numel, n, grad_dtype);
    if (rc != NOVAK_OK) return rc;
    for (int i = 0; i < n; ++i)
        if (!h_params[i] || !h_grads[i] || !d_params[i] || !d_grads[i])
            return fail(o, NOVAK_EINVAL, "step_host: tensor %d has a NULL pointer", i);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const size_t gsz = grad_dtype == NOVAK_GRAD_BF16 ? 2 : 4;

    StepCtx ctx;
    if ((rc = begin_step(o, d_params, const_cast<const void *const *>(d_grads), grad_dtype, stream,
                         &ctx)) != NOVAK_OK)
        return rc;
    if (o->segments.empty() || o->segments_for != o->host_segment_elems) build_segments(o);
    if ((rc = prepare_host_pipeline(o)) != NOVAK_OK) return rc;

    // upload stream: gradients of segment i; caller's stream: kernel over segment
    // i once they have arrived; download stream: its parameters once the kernel
    // has run.  Both copy streams start behind the caller's earlier work and the
    // caller's stream ends behind the last download.
    const int n_seg = static_cast<int>(o->segments.size());
    cudaEvent_t ev_start = o->host_ev[0], ev_end = o->host_ev[1];
    cudaError_t e;
    const char *what = "host pipeline";
    int launched = 0, extra_launches = 0;
    bool forked = false;
    do {
        what = "cudaEventRecord(start)";
        if ((e = cudaEventRecord(ev_start, stream)) != cudaSuccess) break;
        if ((e = cudaStreamWaitEvent(o->up_stream, ev_start, 0)) != cudaSuccess) break;
        if ((e = cudaStreamWaitEvent(o->down_stream, ev_start, 0)) != cudaSuccess) break;
        forked = true;
        const bool stats = ctx.pre != novak::PRE_NONE || ctx.trust != nullptr;
        if (stats) {
            // The norm and the row means need the whole gradient: every run is
            // uploaded before the statistics kernel, and only kernels and
            // downloads of different runs overlap.
            what = "gradient upload";
            for (int i = 0; i < n_seg && e == cudaSuccess; ++i)
                e = copy_ranges(o->segments[i], d_grads, h_grads, gsz, cudaMemcpyHostToDevice, o->up_stream);
            if (e != cudaSuccess) break;
            if ((e = cudaEventRecord(o->host_ev[2], o->up_stream)) != cudaSuccess) break;
            if ((e = cudaStreamWaitEvent(stream, o->host_ev[2], 0)) != cudaSuccess) break;
            if ((e = launch_prepasses(o, ctx, stream, &extra_launches, &what)) != cudaSuccess) break;
        }
        for (int i = 0; i < n_seg && e == cudaSuccess; ++i) {
            const novak_opt::Segment &seg = o->segments[i];
            cudaEvent_t ev_up = o->host_ev[2 + 2 * i], ev_step = o->host_ev[3 + 2 * i];
            if (!stats) {
                what = "gradient upload";
                if ((e = copy_ranges(seg, d_grads, h_grads, gsz, cudaMemcpyHostToDevice, o->up_stream)) != cudaSuccess) break;
                if ((e = cudaEventRecord(ev_up, o->up_stream)) != cudaSuccess) break;
                if ((e = cudaStreamWaitEvent(stream, ev_up, 0)) != cudaSuccess) break;
            }
            what = "step kernel launch";
            if ((e = launch_range(o, ctx, seg.c0, seg.c1, stream)) != cudaSuccess) break;
            ++launched;
            if ((e = cudaEventRecord(ev_step, stream)) != cudaSuccess) break;
            if ((e = cudaStreamWaitEvent(o->down_stream, ev_step, 0)) != cudaSuccess) break;
            what = "parameter download";
            if ((e = copy_ranges(seg, h_params, const_cast<const void *const *>(d_params), 4,
                                 cudaMemcpyDeviceToHost, o->down_stream)) != cudaSuccess) break;
        }
    } while (false);
    if (forked) {
        // join even after a failure so that the caller's stream stays ordered
        // behind whatever the copy streams were given
        cudaError_t j;
        if ((j = cudaEventRecord(ev_end, o->down_stream)) == cudaSuccess)
            j = cudaStreamWaitEvent(stream, ev_end, 0);
        if (e == cudaSuccess && j != cudaSuccess) { e = j; what = "join of the copy streams"; }
    }
    if (launched == n_seg) commit_step(o, ctx, launched + extra_launches);
    if (e != cudaSuccess) return fail_cuda(o, e, what);
    return NOVAK_OK;
}

// ---------------------------------------------------------------------------
// novak_step_noalloc: the same step with its work table in the library's
// statically allocated device array instead of cudaMalloc'ed memory.
// ---------------------------------------------------------------------------
namespace {
// Which upload the shared table of each device currently holds (0 = none).
uint64_t g_noalloc_owner[64] = {};
uint64_t g_noalloc_next_token = 1;
}  // namespace

int novak_step_noalloc(novak_opt *o, void *const *d_params, const void *const *d_grads,
                       const int64_t *numel, int n, int grad_dtype, void *stream_)
{
    if (!o) return NOVAK_EINVAL;
    if (!o->attached) return fail(o, NOVAK_ESTATE, "step_noalloc: no state attached");
    if (!d_params || !d_grads || !numel) return fail(o, NOVAK_EINVAL, "step_noalloc: NULL argument");
    if (grad_dtype != NOVAK_GRAD_F32 && grad_dtype != NOVAK_GRAD_BF16)
        return fail(o, NOVAK_EINVAL, "step_noalloc: unknown grad_dtype %d", grad_dtype);
    if (n != o->n || std::memcmp(numel, o->numel.data(), n * sizeof(int64_t)) != 0)
        return fail(o, NOVAK_ESTATE, "step_noalloc: tensor list differs from the attached layout");
    if (pre_mode(o) != novak::PRE_NONE || o->h.layer_adapt)
        return fail(o, NOVAK_ESTATE, "step_noalloc: clipping, centralization and layer adaptation keep "
                    "scratch in allocated device memory; use novak_step, or switch them off");
    if (n > novak::kNoAllocMaxTensors)
        return fail(o, NOVAK_EINVAL, "step_noalloc: %d tensors exceed the static table's %d; "
                    "split the group or use novak_step", n, novak::kNoAllocMaxTensors);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);

    if (o->na_chunks.empty())
        build_chunks(o->numel.data(), o->phase.data(), o->n, o->chunk_elems, o->na_chunks);
    if (o->na_chunks.size() > static_cast<size_t>(novak::kNoAllocMaxChunks)) {
        const size_t need = o->na_chunks.size();
        o->na_chunks.clear();
        return fail(o, NOVAK_EINVAL, "step_noalloc: %zu chunk-table entries exceed the static "
                    "table's %d; raise NOVAK_OPT_CHUNK_ELEMS (now %lld) or use novak_step",
                    need, novak::kNoAllocMaxChunks, static_cast<long long>(o->chunk_elems));
    }

    // tensor records: rebuilt on the host when the caller's pointers changed
    bool changed = o->na_gdtype != grad_dtype || o->na_p.empty() ||
                   std::memcmp(o->na_p.data(), d_params, n * sizeof(void *)) != 0 ||
                   std::memcmp(o->na_g.data(), d_grads, n * sizeof(void *)) != 0;
    if (changed) {
        const uintptr_t gmask = grad_dtype == NOVAK_GRAD_BF16 ? 1u : 3u;
        for (int i = 0; i < n; ++i) {
            const uintptr_t p = reinterpret_cast<uintptr_t>(d_params[i]);
            const uintptr_t g = reinterpret_cast<uintptr_t>(d_grads[i]);
            if (!p || !g) return fail(o, NOVAK_EINVAL, "tensor %d: NULL pointer", i);
            if ((p & 3u) || (g & gmask))
                return fail(o, NOVAK_EINVAL, "tensor %d: pointer not aligned to its element size", i);
        }
        const bool la = o->h.la_k > 0;
        const bool traj = la && o->h.la_mode == NOVAK_LOOKAHEAD_TRAJ_MEAN;
        o->na_recs.resize(n);
        for (int i = 0; i < n; ++i) {
            TensorRec &r = o->na_recs[i];
            r.p = static_cast<float *>(d_params[i]);
            r.g = d_grads[i];
            r.m = slice(o, 0, i);
            r.v = slice(o, 1, i);
            r.slow = la ? slice(o, 2, i) : nullptr;
            r.acc = traj ? slice(o, 3, i) : nullptr;
            r.mean = nullptr;
            r.p16 = o->copies.empty() ? nullptr : static_cast<__nv_bfloat16 *>(o->copies[i]);
            r.row_len = 0;
            r.reserved = 0;
        }
        o->na_p.assign(d_params, d_params + n);
        o->na_g.assign(d_grads, d_grads + n);
        o->na_gdtype = grad_dtype;
        o->na_token = 0;  // forces an upload below
    }

    // The static table of the current device (first call on a device resolves
    // its address; nothing is allocated).
    TensorRec *d_recs = nullptr;
    Chunk *d_chunks = nullptr;
    int dev = 0;
    cudaError_t e;
    if ((e = cudaGetDevice(&dev)) != cudaSuccess) return fail_cuda(o, e, "cudaGetDevice");
    if ((e = novak::noalloc_table(&d_recs, &d_chunks)) != cudaSuccess)
        return fail_cuda(o, e, "cudaGetSymbolAddress(static work table)");
    if (o->na_token == 0 || g_noalloc_owner[dev] != o->na_token) {
        // Every handle shares the table: (re)write the part this step reads.
        // Copies from pageable memory are staged by the driver before the call
        // returns, so the host vectors may change afterwards.
        if ((e = cudaMemcpyAsync(d_recs, o->na_recs.data(), n * sizeof(TensorRec),
                                 cudaMemcpyHostToDevice, stream)) != cudaSuccess ||
            (e = cudaMemcpyAsync(d_chunks, o->na_chunks.data(), o->na_chunks.size() * sizeof(Chunk),
                                 cudaMemcpyHostToDevice, stream)) != cudaSuccess) {
            g_noalloc_owner[dev] = 0;
            return fail_cuda(o, e, "static work table upload");
        }
        o->na_token = g_noalloc_next_token++;
        g_noalloc_owner[dev] = o->na_token;
    }

    const int64_t t = o->t + 1;
    const Plan p = make_plan(o->h, t);
    const int la_action = lookahead_action(o->h, t);
    const StepScalars s = make_scalars(o->h, p);

    const int n_chunks = static_cast<int>(o->na_chunks.size());
    novak::LaunchCfg cfg;
    cfg.grid = n_chunks;
    cfg.reverse = (o->serpentine && (t % 2 == 0)) ? 1 : 0;
    cfg.pdl = o->pdl;
    cfg.pre = novak::PRE_NONE | (o->copies.empty() ? 0 : novak::PRE_COPY16);
    e = novak::launch_step(d_chunks, n_chunks, d_recs, nullptr, nullptr, s, o->h.nesterov, grad_dtype,
                           la_action, cfg, stream);
    if (e != cudaSuccess) return fail_cuda(o, e, "step kernel launch");

    o->t = t;
    o->launches += 1;
    o->last_plan = p;
    o->last_grid = cfg.grid;
    if (p.is_sync) { o->n_syncs += 1; o->last_sync = t; }
    return NOVAK_OK;
}

int novak_set_tensor_rows(novak_opt *o, const int64_t *rows, int n)
{
    if (!o) return NOVAK_EINVAL;
    if (!o->attached) return fail(o, NOVAK_ESTATE, "set_tensor_rows: attach the state first");
    if (!rows || n != o->n) return fail(o, NOVAK_EINVAL, "set_tensor_rows: NULL or wrong tensor count");
    int64_t total = 0;
    for (int i = 0; i < n; ++i) {
        if (rows[i] < 0) return fail(o, NOVAK_EINVAL, "set_tensor_rows: tensor %d has negative rows", i);
        if (rows[i] == 0) continue;
        if (o->numel[i] % rows[i] != 0)
            return fail(o, NOVAK_EINVAL, "set_tensor_rows: tensor %d: %lld elements are not a multiple of %lld rows",
                        i, static_cast<long long>(o->numel[i]), static_cast<long long>(rows[i]));
        if (o->numel[i] >= (int64_t(1) << 31))
            return fail(o, NOVAK_EINVAL, "set_tensor_rows: tensor %d has 2^31 or more elements", i);
        total += rows[i];
    }
    o->rows.assign(rows, rows + n);
    int64_t off = 0;
    for (int i = 0; i < n; ++i) { o->row_off[i] = off; off += o->rows[i]; }
    o->total_rows = total;
    o->rows_gen += 1;
    invalidate_tables(o);
    return NOVAK_OK;
}

int novak_set_param_copies(novak_opt *o, void *const *d_copies, int n)
{
    if (!o) return NOVAK_EINVAL;
    if (!o->attached) return fail(o, NOVAK_ESTATE, "set_param_copies: attach the state first");
    if (d_copies == nullptr) {
        o->copies.clear();
    } else {
        if (n != o->n) return fail(o, NOVAK_EINVAL, "set_param_copies: wrong tensor count");
        for (int i = 0; i < n; ++i) {
            const uintptr_t c = reinterpret_cast<uintptr_t>(d_copies[i]);
            if (!c || (c & 1u))
                return fail(o, NOVAK_EINVAL, "set_param_copies: copy %d is NULL or not 2-byte aligned", i);
        }
        o->copies.assign(d_copies, d_copies + n);
    }
    invalidate_tables(o);
    o->na_p.clear();              // the no-allocation path rebuilds its records too
    return NOVAK_OK;
}

int novak_get_grad_stats(novak_opt *o, double *norm, double *factor, void *stream_)
{
    if (!o) return NOVAK_EINVAL;
    if (!o->prep_out) return fail(o, NOVAK_ESTATE, "get_grad_stats: no step with clipping or centralization yet");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    PrepOut h;
    cudaError_t e;
    if ((e = cudaMemcpyAsync(&h, o->prep_out, sizeof h, cudaMemcpyDeviceToHost, stream)) != cudaSuccess ||
        (e = cudaStreamSynchronize(stream)) != cudaSuccess)
        return fail_cuda(o, e, "get_grad_stats");
    if (norm) *norm = h.norm;
    if (factor) *factor = static_cast<double>(h.factor);
    return NOVAK_OK;
}

int novak_get_auto_lr_state(novak_opt *o, double *g_bar, double *theta_bar, double *scale,
                            void *stream_)
{
    if (!o) return NOVAK_EINVAL;
    if (o->ema_pending || !o->prep_out) {
        // nothing on the device yet: what a resume put in, or the initial zeros
        if (g_bar) *g_bar = o->ema_pending ? o->pending_g_bar : 0.0;
        if (theta_bar) *theta_bar = o->ema_pending ? o->pending_theta_bar : 0.0;
        if (scale) *scale = 1.0;
        return NOVAK_OK;
    }
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    PrepOut h;
    cudaError_t e;
    if ((e = cudaMemcpyAsync(&h, o->prep_out, sizeof h, cudaMemcpyDeviceToHost, stream)) != cudaSuccess ||
        (e = cudaStreamSynchronize(stream)) != cudaSuccess)
        return fail_cuda(o, e, "get_auto_lr_state");
    if (g_bar) *g_bar = h.g_bar;
    if (theta_bar) *theta_bar = h.theta_bar;
    if (scale) *scale = static_cast<double>(h.auto_scale);
    return NOVAK_OK;
}

int novak_set_auto_lr_state(novak_opt *o, double g_bar, double theta_bar)
{
    if (!o) return NOVAK_EINVAL;
    if (!(g_bar >= 0.0) || !(theta_bar >= 0.0) || !std::isfinite(g_bar) || !std::isfinite(theta_bar))
        return fail(o, NOVAK_EINVAL, "set_auto_lr_state: averages of norms are finite and >= 0");
    o->pending_g_bar = g_bar;
    o->pending_theta_bar = theta_bar;
    o->ema_pending = true;
    return NOVAK_OK;
}

int novak_get_trust_ratios(novak_opt *o, float *h_out, int n, void *stream_)
{
    if (!o) return NOVAK_EINVAL;
    if (!h_out || n != o->n) return fail(o, NOVAK_EINVAL, "get_trust_ratios: NULL or wrong tensor count");
    if (!o->trust || o->t == 0) return fail(o, NOVAK_ESTATE, "get_trust_ratios: no step with layer adaptation yet");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    cudaError_t e;
    if ((e = cudaMemcpyAsync(h_out, o->trust, n * sizeof(float), cudaMemcpyDeviceToHost, stream)) != cudaSuccess ||
        (e = cudaStreamSynchronize(stream)) != cudaSuccess)
        return fail_cuda(o, e, "get_trust_ratios");
    return NOVAK_OK;
}

int novak_get_info(const novak_opt *o, novak_info *out)
{
    if (!o || !out) return NOVAK_EINVAL;
    fill_info(o, o->last_plan, out);
    return NOVAK_OK;
}

int novak_plan(const novak_opt *o, int64_t t, novak_info *out)
{
    if (!o || !out || t < 1) return NOVAK_EINVAL;
    fill_info(o, make_plan(o->h, t), out);
    return NOVAK_OK;
}

int novak_state_ptrs(const novak_opt *o, int tensor, void **d_m, void **d_v, void **d_slow,
                     void **d_acc)
{
    if (!o || !o->attached || tensor < 0 || tensor >= o->n) return NOVAK_EINVAL;
    if (d_m) *d_m = slice(o, 0, tensor);
    if (d_v) *d_v = slice(o, 1, tensor);
    if (d_slow) *d_slow = o->n_arrays > 2 ? slice(o, 2, tensor) : nullptr;
    if (d_acc) *d_acc = o->n_arrays > 3 ? slice(o, 3, tensor) : nullptr;
    return NOVAK_OK;
}

int novak_export_meta(const novak_opt *o, novak_meta *out)
{
    if (!o || !out) return NOVAK_EINVAL;
    std::memset(out, 0, sizeof *out);
    out->magic = kMetaMagic;
    out->t = o->t; out->n_syncs = o->n_syncs; out->last_sync_step = o->last_sync;
    out->total_numel = o->total_numel;
    out->lr = o->h.lr; out->beta1 = o->h.beta1; out->beta2 = o->h.beta2; out->eps = o->h.eps;
    out->weight_decay = o->h.wd; out->nesterov_beta = o->h.beta_n;
    out->lookahead_alpha = o->h.la_alpha;
    out->nesterov_variant = o->h.nesterov; out->lookahead_k = o->h.la_k;
    out->lookahead_mode = o->h.la_mode; out->rectified = o->h.rectified;
    out->bias1_power = o->h.bias1_power;
    out->clip_threshold = o->h.clip;
    out->centralize = o->h.centralize;
    out->adaptive_beta = o->h.adaptive_beta;
    out->layer_adaptation = o->h.layer_adapt;
    out->sparse_threshold = o->h.sparse_tau;
    out->auto_lr = o->h.auto_lr;
    out->auto_lr_gamma = o->h.auto_gamma;
    out->beta1_tau = o->h.tau1;
    out->beta2_tau = o->h.tau2;
    out->n_tensors = o->n;
    out->warnings = o->warnings;
    return NOVAK_OK;
}

int novak_import_meta(novak_opt *o, const novak_meta *in)
{
    if (!o || !in) return NOVAK_EINVAL;
    if (in->magic != kMetaMagic) return fail(o, NOVAK_EINVAL, "import: not a NOVAK meta record");
    if (!o->attached) return fail(o, NOVAK_ESTATE, "import: attach the state first");
    if (in->n_tensors != o->n || in->total_numel != o->total_numel ||
        in->lookahead_k != o->h.la_k || in->lookahead_mode != o->h.la_mode)
        return fail(o, NOVAK_ESTATE, "import: tensor list or lookahead layout differs");
    if (in->t < 0 || in->n_syncs < 0) return fail(o, NOVAK_EINVAL, "import: negative counter");
    Hyper h = o->h;
    h.lr = in->lr; h.beta1 = in->beta1; h.beta2 = in->beta2; h.eps = in->eps;
    h.wd = in->weight_decay; h.beta_n = in->nesterov_beta; h.la_alpha = in->lookahead_alpha;
    h.nesterov = in->nesterov_variant; h.rectified = in->rectified;
    h.bias1_power = in->bias1_power;
    h.clip = in->clip_threshold;
    h.adaptive_beta = in->adaptive_beta;
    h.layer_adapt = in->layer_adaptation;
    h.sparse_tau = in->sparse_threshold;
    h.auto_lr = in->auto_lr;
    h.auto_gamma = in->auto_lr_gamma;
    h.tau1 = in->beta1_tau;
    h.tau2 = in->beta2_tau;
    if (h.centralize != in->centralize) invalidate_tables(o);
    h.centralize = in->centralize;
    const char *why;
    if (!check_hyper(h, &why)) return fail(o, NOVAK_EINVAL, "import: %s", why);
    o->h = h;
    o->t = in->t; o->n_syncs = in->n_syncs; o->last_sync = in->last_sync_step;
    o->warnings |= in->warnings;
    o->last_plan = make_plan(h, in->t > 0 ? in->t : 1);
    return NOVAK_OK;
}

int64_t novak_build_row_units(const int64_t *numel, const int64_t *rows, int n, int32_t *tensor,
                              int64_t *row0, int64_t *n_rows, int64_t *part_off,
                              int64_t *part_len, int64_t cap)
{
    if (!numel || !rows || n <= 0 || cap < 0) return -1;
    for (int i = 0; i < n; ++i)
        if (numel[i] <= 0 || rows[i] < 0 || (rows[i] > 0 && (numel[i] % rows[i] != 0 ||
                                                             numel[i] >= (int64_t(1) << 31))))
            return -1;
    std::vector<RowUnit> units;
    build_row_units(numel, rows, n, units);
    const int64_t count = static_cast<int64_t>(units.size());
    for (int64_t i = 0; i < count && i < cap; ++i) {
        if (tensor) tensor[i] = units[i].tensor;
        if (row0) row0[i] = units[i].row0;
        if (n_rows) n_rows[i] = units[i].n_rows;
        if (part_off) part_off[i] = units[i].part_off;
        if (part_len) part_len[i] = units[i].part_len;
    }
    return count;
}

int64_t novak_build_chunks(const int64_t *numel, const int32_t *phase, int n,
                           int64_t chunk_elems, int32_t *tensor, int64_t *offset,
                           int32_t *len, int64_t cap)
{
    if (!numel || n <= 0 || chunk_elems < kSlotAlign || chunk_elems % kSlotAlign != 0 ||
        chunk_elems > INT32_MAX || cap < 0)
        return -1;
    for (int i = 0; i < n; ++i)
        if (numel[i] <= 0 || (phase && (phase[i] < 0 || phase[i] >= kSlotAlign))) return -1;
    std::vector<Chunk> chunks;
    build_chunks(numel, phase, n, chunk_elems, chunks);
    const int64_t count = static_cast<int64_t>(chunks.size());
    for (int64_t i = 0; i < count && i < cap; ++i) {
        if (tensor) tensor[i] = chunks[i].tensor;
        if (offset) offset[i] = chunks[i].offset;
        if (len) len[i] = chunks[i].len;
    }
    return count;
}

const char *novak_last_error(const novak_opt *o) { return o ? o->err.c_str() : ""; }

}  // extern "C"
