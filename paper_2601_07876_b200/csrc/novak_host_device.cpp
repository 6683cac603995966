// Host side of the NOVAK step library, part 2: the device work tables of a
// handle (chunk table, cached tensor-record tables with their pinned staging
// ring, scratch of the statistics and layer-adaptation passes).
#include "novak_handle.h"

#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>

using namespace novak_host;

namespace novak_host {

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
    if (o->d_plan) cudaFree(o->d_plan);
    o->d_plan = nullptr;
    o->dyn_upload_counters = o->dyn_upload_rates = true;
    if (o->d_look) cudaFree(o->d_look);
    if (o->h_look) cudaFreeHost(o->h_look);
    if (o->look_ev) cudaEventDestroy(o->look_ev);
    o->d_look = o->h_look = nullptr;
    o->look_ev = nullptr;
    o->look_p.clear();
    o->look_save = nullptr;
    o->extrapolated = false;
    if (o->d_adapt) cudaFree(o->d_adapt);
    if (o->adapt_direction) cudaFree(o->adapt_direction);
    o->adapt_direction = nullptr;
    if (o->h_adapt_error) cudaFreeHost(o->h_adapt_error);
    o->d_adapt = nullptr;
    o->d_item_code = nullptr;
    o->d_item_chunk = nullptr;
    o->n_items = 0;
    o->adapt_ctl = nullptr;
    o->adapt_arrived = nullptr;
    o->adapt_ready = nullptr;
    o->h_adapt_error = o->d_adapt_error = nullptr;
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
    o->d_rest = nullptr;
    o->d_own = o->d_long_units = nullptr;
    o->n_rest = o->n_own = o->n_long_units = 0;
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
    // Work of the statistics pass: row units for the tensors with rows, chunk-table
    // entries for the rest.  With centralization the same allocation also holds the
    // tables of the step kernel that owns rows (used by steps that need no statistic
    // of the whole gradient): its units of whole rows, the chunk-table entries of the
    // tensors it does not own (those without rows, and those with rows too long to
    // own), and the statistics units of the latter, which is all the pass then has to
    // do.  Both sets are built together, so a caller may alternate between entry points
    // that use one or the other without any reallocation.
    std::vector<RowUnit> units, own, long_units;
    std::vector<Chunk> plain, rest;
    if (centre) {
        build_row_units(o->numel.data(), o->rows.data(), o->n, units);
        for (const Chunk &c : o->h_chunks)
            if (o->rows[c.tensor] <= 0) plain.push_back(c);
        build_own_units(o->numel.data(), o->rows.data(), o->n, own);
        std::vector<int64_t> long_rows(o->rows.size(), 0);
        for (int i = 0; i < o->n; ++i)
            if (o->rows[i] > 0 && o->numel[i] / o->rows[i] > static_cast<int64_t>(novak::kOwnRowMax))
                long_rows[i] = o->rows[i];
        build_row_units(o->numel.data(), long_rows.data(), o->n, long_units);
        for (const Chunk &c : o->h_chunks)
            if (o->rows[c.tensor] <= 0 || long_rows[c.tensor] > 0) rest.push_back(c);
    }
    const size_t n_plain = centre ? plain.size() : static_cast<size_t>(o->n_chunks);
    if (units.size() > static_cast<size_t>(INT32_MAX) / 2 || own.size() > static_cast<size_t>(INT32_MAX) / 2)
        return fail(o, NOVAK_EINVAL, "too many rows");
    // sized for fp32 gradients; bf16 gradients take more entries per CTA and need less
    // (the pass over the long rows alone needs fewer sums than the pass over everything)
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
    const size_t off_rest = off;    off += rest.size() * sizeof(Chunk);
    const size_t off_units = off;   off += units.size() * sizeof(RowUnit);
    const size_t off_own = off;     off += own.size() * sizeof(RowUnit);
    const size_t off_long = off;    off += long_units.size() * sizeof(RowUnit);
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
    o->d_rest = reinterpret_cast<Chunk *>(o->d_prep + off_rest);
    o->d_units = reinterpret_cast<RowUnit *>(o->d_prep + off_units);
    o->d_own = reinterpret_cast<RowUnit *>(o->d_prep + off_own);
    o->d_long_units = reinterpret_cast<RowUnit *>(o->d_prep + off_long);
    o->row_mean = reinterpret_cast<float2 *>(o->d_prep + off_mean);
    o->n_plain = static_cast<int>(n_plain);
    o->n_units = static_cast<int>(units.size());
    o->n_rest = static_cast<int>(rest.size());
    o->n_own = static_cast<int>(own.size());
    o->n_long_units = static_cast<int>(long_units.size());
    // The tables are built once per layout: blocking copies keep the host
    // vectors' lifetime trivial.
    const struct { void *dst; const void *src; size_t bytes; } uploads[] = {
        {o->d_plain, plain.data(), plain.size() * sizeof(Chunk)},
        {o->d_rest, rest.data(), rest.size() * sizeof(Chunk)},
        {o->d_units, units.data(), units.size() * sizeof(RowUnit)},
        {o->d_own, own.data(), own.size() * sizeof(RowUnit)},
        {o->d_long_units, long_units.data(), long_units.size() * sizeof(RowUnit)},
    };
    for (const auto &u : uploads)
        if (u.bytes != 0 &&
            (e = cudaMemcpyAsync(u.dst, u.src, u.bytes, cudaMemcpyHostToDevice, stream)) != cudaSuccess)
            return fail_cuda(o, e, "statistics table upload");
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

// Item list, counters and flags of the kernel that adapts and steps in one
// launch; allocated when a step first needs them (after prepare_trust).
int prepare_adapt(novak_opt *o, cudaStream_t stream)
{
    if (o->d_adapt) return NOVAK_OK;
    std::vector<int32_t> codes, counts;
    const int64_t lead_entries = (o->adapt_lead_elems + o->chunk_elems - 1) / o->chunk_elems;
    const int64_t lag = build_adapt_items(o->h_tensor_first, o->n, lead_entries, o->adapt_group, codes, counts);
    if (codes.size() + static_cast<size_t>(lag) > static_cast<size_t>(INT32_MAX))
        return fail(o, NOVAK_EINVAL, "too many chunks");
    // an item's entries as one span: consecutive in their tensor, all but the last full
    std::vector<Chunk> entries(codes.size());
    for (size_t k = 0; k < codes.size(); ++k) {
        const int c = codes[k];
        Chunk span = o->h_chunks[c];
        for (int j = 1; j < counts[k]; ++j) {
            if (o->h_chunks[c + j - 1].len != o->chunk_elems || o->h_chunks[c + j].tensor != span.tensor)
                return fail(o, NOVAK_EINVAL, "layer adaptation items: a short entry inside a tensor");
            span.len += o->h_chunks[c + j].len;
        }
        entries[k] = span;
    }
    const size_t n = static_cast<size_t>(o->n);
    const size_t off_ready = 256;
    const size_t off_arrived = off_ready + n * sizeof(unsigned long long);
    const size_t off_chunk = (off_arrived + n * sizeof(unsigned) + 15) / 16 * 16;
    const size_t off_code = off_chunk + entries.size() * sizeof(Chunk);
    const size_t bytes = off_code + codes.size() * sizeof(int32_t) + 16;
    cudaError_t e;
    if (!o->h_adapt_error) {
        if ((e = cudaHostAlloc(reinterpret_cast<void **>(&o->h_adapt_error), sizeof(unsigned),
                               cudaHostAllocMapped)) != cudaSuccess) {
            o->h_adapt_error = nullptr;
            return fail(o, NOVAK_ENOMEM, "cudaHostAlloc(error word): %s", cudaGetErrorString(e));
        }
        *o->h_adapt_error = 0u;
        if ((e = cudaHostGetDevicePointer(reinterpret_cast<void **>(&o->d_adapt_error),
                                          o->h_adapt_error, 0)) != cudaSuccess)
            return fail_cuda(o, e, "cudaHostGetDevicePointer(error word)");
    }
    if ((e = cudaMalloc(reinterpret_cast<void **>(&o->d_adapt), bytes)) != cudaSuccess) {
        o->d_adapt = nullptr;
        return fail(o, NOVAK_ENOMEM, "cudaMalloc(layer adaptation items, %zu B): %s", bytes, cudaGetErrorString(e));
    }
    // the directions of one step, 4 B per element of the group: written by the S items,
    // read by the U items a few MB of traffic later
    o->adapt_slot_elems = static_cast<int>((o->chunk_elems + 3) / 4 * 4);
    const size_t dir_bytes = static_cast<size_t>(o->n_chunks) * o->adapt_slot_elems * sizeof(float);
    if ((e = cudaMalloc(reinterpret_cast<void **>(&o->adapt_direction), dir_bytes)) != cudaSuccess) {
        o->adapt_direction = nullptr;
        cudaFree(o->d_adapt);
        o->d_adapt = nullptr;
        return fail(o, NOVAK_ENOMEM, "cudaMalloc(layer adaptation directions, %zu B): %s", dir_bytes,
                    cudaGetErrorString(e));
    }
    o->adapt_ctl = reinterpret_cast<novak::AdaptCtl *>(o->d_adapt);
    o->adapt_arrived = reinterpret_cast<unsigned *>(o->d_adapt + off_arrived);
    o->adapt_ready = reinterpret_cast<unsigned long long *>(o->d_adapt + off_ready);
    o->d_item_chunk = reinterpret_cast<Chunk *>(o->d_adapt + off_chunk);
    o->d_item_code = reinterpret_cast<int *>(o->d_adapt + off_code);
    o->n_items = static_cast<int>(codes.size());
    o->adapt_lag = static_cast<int>(lag);
    // built once: blocking copies keep the host vectors' lifetime trivial
    if ((e = cudaMemsetAsync(o->d_adapt, 0, off_chunk, stream)) != cudaSuccess ||
        (e = cudaMemcpyAsync(o->d_item_chunk, entries.data(), entries.size() * sizeof(Chunk),
                             cudaMemcpyHostToDevice, stream)) != cudaSuccess ||
        (e = cudaMemcpyAsync(o->d_item_code, codes.data(), codes.size() * sizeof(int32_t),
                             cudaMemcpyHostToDevice, stream)) != cudaSuccess ||
        (e = cudaStreamSynchronize(stream)) != cudaSuccess)
        return fail_cuda(o, e, "layer adaptation item upload");
    return NOVAK_OK;
}

// Records of the look-ahead helpers (Eq. 10): allocated on first use, uploaded
// through one pinned buffer whenever the parameter list changes.
int prepare_look(novak_opt *o, void *const *d_params, cudaStream_t stream)
{
    const size_t n = static_cast<size_t>(o->n);
    cudaError_t e;
    // each of the three is created once; a call that failed half-way is completed here
    if (!o->d_look) {
        if ((e = cudaMalloc(reinterpret_cast<void **>(&o->d_look), n * sizeof(novak::LookRec))) != cudaSuccess) {
            o->d_look = nullptr;
            return fail(o, NOVAK_ENOMEM, "cudaMalloc(look-ahead records): %s", cudaGetErrorString(e));
        }
        o->look_p.clear();
    }
    if (!o->h_look &&
        (e = cudaMallocHost(reinterpret_cast<void **>(&o->h_look), n * sizeof(novak::LookRec))) != cudaSuccess) {
        o->h_look = nullptr;
        return fail(o, NOVAK_ENOMEM, "cudaMallocHost(look-ahead records): %s", cudaGetErrorString(e));
    }
    if (!o->look_ev &&
        (e = cudaEventCreateWithFlags(&o->look_ev, cudaEventDisableTiming)) != cudaSuccess) {
        o->look_ev = nullptr;
        return fail_cuda(o, e, "cudaEventCreate(look-ahead records)");
    }
    if (o->look_p.size() == n && std::memcmp(o->look_p.data(), d_params, n * sizeof(void *)) == 0)
        return NOVAK_OK;
    for (size_t i = 0; i < n; ++i) {
        const uintptr_t p = reinterpret_cast<uintptr_t>(d_params[i]);
        if (!p) return fail(o, NOVAK_EINVAL, "tensor %zu: NULL pointer", i);
        if (p & 3u) return fail(o, NOVAK_EINVAL, "tensor %zu: pointer not aligned to its element size", i);
    }
    // the previous upload may still be reading the staging buffer
    if (!o->look_p.empty() && (e = cudaEventSynchronize(o->look_ev)) != cudaSuccess)
        return fail_cuda(o, e, "look-ahead record staging");
    o->look_p.clear();
    for (size_t i = 0; i < n; ++i) {
        o->h_look[i].p = static_cast<float *>(d_params[i]);
        o->h_look[i].state_off = o->slot_off[i] + o->phase[i];
    }
    if ((e = cudaMemcpyAsync(o->d_look, o->h_look, n * sizeof(novak::LookRec), cudaMemcpyHostToDevice,
                             stream)) != cudaSuccess ||
        (e = cudaEventRecord(o->look_ev, stream)) != cudaSuccess)
        return fail_cuda(o, e, "look-ahead record upload");
    o->look_p.assign(d_params, d_params + n);
    return NOVAK_OK;
}

int prepare_dyn(novak_opt *o, cudaStream_t stream)
{
    cudaError_t e;
    if (!o->d_plan) {
        if ((e = cudaMalloc(reinterpret_cast<void **>(&o->d_plan), sizeof(novak::DevPlan))) != cudaSuccess) {
            o->d_plan = nullptr;
            return fail(o, NOVAK_ENOMEM, "cudaMalloc(device plan): %s", cudaGetErrorString(e));
        }
        if ((e = cudaMemsetAsync(o->d_plan, 0, sizeof(novak::DevPlan), stream)) != cudaSuccess)
            return fail_cuda(o, e, "cudaMemsetAsync(device plan)");
        o->dyn_upload_counters = o->dyn_upload_rates = true;
    }
    // Copies from the stack: staged by the driver before the call returns (not
    // possible while the stream is being captured: change options and import
    // checkpoints outside a capture).
    const bool arm = o->dyn_upload_counters || o->dyn_upload_rates;
    if (o->dyn_upload_counters) {
        // the device counts the step that runs next
        const long long c[3] = {o->t + 1, o->n_syncs, o->last_sync};
        if ((e = cudaMemcpyAsync(&o->d_plan->t, c, sizeof c, cudaMemcpyHostToDevice, stream)) != cudaSuccess)
            return fail_cuda(o, e, "upload of the step counters");
        o->dyn_upload_counters = false;
    }
    if (o->dyn_upload_rates) {
        const double r[2] = {o->h.lr, o->h.wd};
        if ((e = cudaMemcpyAsync(&o->d_plan->lr, r, sizeof r, cudaMemcpyHostToDevice, stream)) != cudaSuccess)
            return fail_cuda(o, e, "upload of learning rate and weight decay");
        o->dyn_upload_rates = false;
    }
    if (arm && (e = novak::launch_plan_arm(o->d_plan, &o->h, sizeof o->h, stream)) != cudaSuccess)
        return fail_cuda(o, e, "plan kernel launch");
    if (arm) o->launches += 1;
    return NOVAK_OK;
}

int read_dyn(const novak_opt *o, novak::DevPlan *out)
{
    if (!o->d_plan) return NOVAK_ESTATE;
    if (cudaDeviceSynchronize() != cudaSuccess) return NOVAK_ECUDA;
    if (cudaMemcpy(out, o->d_plan, sizeof *out, cudaMemcpyDeviceToHost) != cudaSuccess) return NOVAK_ECUDA;
    return NOVAK_OK;
}

uint64_t hash_pointers(void *const *d_params, const void *const *d_grads, int n, int grad_dtype,
                       const void *save)
{
    uint64_t h = 0xcbf29ce484222325ull ^ static_cast<uint64_t>(grad_dtype);
    h = (h ^ reinterpret_cast<uintptr_t>(save)) * 0x100000001b3ull;
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
                    int grad_dtype, const void *save, cudaStream_t stream)
{
    const int n = o->n;
    const uint64_t hash = hash_pointers(d_params, d_grads, n, grad_dtype, save);
    int lru = 0;
    for (int k = 0; k < kRecTables; ++k) {
        novak_opt::RecTable &tb = o->tables[k];
        if (tb.gdtype == grad_dtype && tb.hash == hash && tb.save == save && !tb.p.empty() &&
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
    bool scalar_path = false, narrow_grad = false;
    for (int i = 0; i < n; ++i) {
        const uintptr_t p = reinterpret_cast<uintptr_t>(d_params[i]);
        const uintptr_t g = reinterpret_cast<uintptr_t>(d_grads[i]);
        if (!p || !g) return fail(o, NOVAK_EINVAL, "tensor %d: NULL pointer", i);
        if ((p & 3u) || (g & gmask)) return fail(o, NOVAK_EINVAL, "tensor %d: pointer not aligned to its element size", i);
        // 128-bit path needs parameter and state congruent mod 16 B (bf16 moments:
        // 8-byte accesses at half the parameter's offset); the state slices (and the
        // save buffer's) share the phase the parameters had at attach.
        const uintptr_t m = reinterpret_cast<uintptr_t>(slice(o, 0, i));
        const bool m_ok = o->h.mom16 ? ((p & 15u) >> 1) == (m & 7u) : ((p ^ m) & 15u) == 0;
        if (!m_ok) scalar_path = true;
        // a gradient at another offset is fetched element by element, the rest stays wide
        if ((((p & 15u) / 4u) != ((g % gvec) / (gvec / 4u))) || (g % (gvec / 4u)))
            narrow_grad = true;
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
        // the save buffer is laid out like a state array: same slot, same phase
        h[i].p_in = save ? static_cast<const float *>(save) + o->slot_off[i] + o->phase[i] : h[i].p;
        h[i].g = d_grads[i];
        h[i].m = slice(o, 0, i);
        h[i].v = slice(o, 1, i);
        h[i].slow = la ? static_cast<float *>(slice(o, 2, i)) : nullptr;
        h[i].acc = traj ? static_cast<float *>(slice(o, 3, i)) : nullptr;
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
    tb.save = save;
    tb.gdtype = grad_dtype;
    tb.hash = hash;
    tb.last_use = ++o->table_clock;
    o->cur_table = lru;
    o->record_uploads += 1;
    if (scalar_path) o->warnings |= NOVAK_WARN_SCALAR_PATH;
    if (narrow_grad) o->warnings |= NOVAK_WARN_NARROW_GRADIENT;
    return NOVAK_OK;
}

}  // namespace novak_host
