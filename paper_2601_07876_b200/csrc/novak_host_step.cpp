// Host side of the NOVAK step library, part 3: the step itself (scalars,
// statistics and layer-adaptation passes, the fused kernel), the pipelined
// host-buffer step, the step without allocations and the device read-backs.
#include "novak_handle.h"

#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>

using namespace novak_host;

namespace {

// Everything one step needs, fixed before anything is enqueued.
struct StepCtx {
    bool adapt_in_step;      // layer adaptation and update as one persistent kernel
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
    // novak_step itself may follow the look-ahead directly: it then reads
    // theta_{t-1} from the save buffer and needs no restore pass
    if (o->extrapolated && std::strcmp(who, "step") != 0)
        return fail(o, NOVAK_ESTATE, "%s: parameters are extrapolated (Eq. 10); call novak_nesterov_restore first", who);
    if (o->half_open && std::strcmp(who, "step_begin") != 0)
        return fail(o, NOVAK_ESTATE, "%s: a step begun with novak_step_begin is still open", who);
    if (!d_params || !d_grads || !numel) return fail(o, NOVAK_EINVAL, "%s: NULL argument", who);
    if (grad_dtype != NOVAK_GRAD_F32 && grad_dtype != NOVAK_GRAD_BF16)
        return fail(o, NOVAK_EINVAL, "%s: unknown grad_dtype %d", who, grad_dtype);
    if (n != o->n || std::memcmp(numel, o->numel.data(), n * sizeof(int64_t)) != 0)
        return fail(o, NOVAK_ESTATE, "%s: tensor list differs from the attached layout", who);
    return NOVAK_OK;
}

// The plain step passes the scalars of ONE step by value: captured into a CUDA
// graph it would replay that step's scalars for ever.  Refuse instead.
int refuse_capture(novak_opt *o, const char *who, cudaStream_t stream)
{
    cudaStreamCaptureStatus st = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(stream, &st) != cudaSuccess) {
        (void)cudaGetLastError();
        return NOVAK_OK;
    }
    if (st != cudaStreamCaptureStatusNone)
        return fail(o, NOVAK_ESTATE, "%s: the stream is being captured; only a handle with "
                    "NOVAK_OPT_GRAPH_CAPTURABLE may be captured into a CUDA graph", who);
    return NOVAK_OK;
}

// What the graph-capturable step does not cover.
int check_dyn(novak_opt *o, const char *who)
{
    if (o->h.true_requested && o->h.true_steps > 0)
        return fail(o, NOVAK_ESTATE, "%s: the graph-capturable step has no true Nesterov steps (the "
                    "closure is the caller's)", who);
    return NOVAK_OK;
}

// Work table on the device, records for these pointers, the scalar plan of step t+1.
// `save`: NULL, or the save buffer of the open look-ahead (theta_{t-1} is read there).
// whole_table: the step is one launch over the whole group (novak_step), so the
// step kernel may own rows (PRE_CENTER_ROWS).
int begin_step(novak_opt *o, void *const *d_params, const void *const *d_grads, int grad_dtype,
               cudaStream_t stream, StepCtx *ctx, const void *save = nullptr,
               bool whole_table = false)
{
    int rc;
    if (!o->d_chunks && (rc = prepare_device(o, stream)) != NOVAK_OK) return rc;
    ctx->pre = step_pre_mode(o, whole_table);
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
    ctx->adapt_in_step = o->h.layer_adapt && whole_table && o->adapt_in_step && !o->dyn;
    if (ctx->adapt_in_step && (rc = prepare_adapt(o, stream)) != NOVAK_OK) return rc;
    if (o->h_adapt_error && *o->h_adapt_error)
        return fail(o, NOVAK_ECUDA, "an earlier step's layer-adaptation kernel gave up waiting for a "
                    "tensor's trust ratio and left entries un-updated; the optimizer state is not usable");
    if ((rc = refresh_records(o, d_params, d_grads, grad_dtype, save, stream)) != NOVAK_OK) return rc;
    ctx->t = o->t + 1;
    ctx->plan = make_plan(o->h, ctx->t);
    ctx->la = lookahead_action(o->h, ctx->t);
    ctx->grad_dtype = grad_dtype;
    ctx->s = make_scalars(o->h, ctx->plan);
    ctx->d_recs = o->d_recs + static_cast<size_t>(o->cur_table) * o->n;
    ctx->reverse = (o->serpentine && (ctx->t % 2 == 0)) ? 1 : 0;
    // After a statistics pass the END of the gradient is what L2 still holds:
    // the step kernel then walks the table from the end.
    if ((ctx->pre != novak::PRE_NONE && ctx->pre != novak::PRE_CENTER_ROWS) ||
        (ctx->trust && !ctx->adapt_in_step))
        ctx->reverse = 1;
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
    // the step kernel owns its rows: only tensors with longer rows need the pass
    if (ctx.pre == novak::PRE_CENTER_ROWS && o->n_long_units == 0) return cudaSuccess;
    *what = "gradient statistics kernel launch";
    const cudaError_t e = launch_stats(o, ctx, finalize, stream);
    if (e == cudaSuccess) *launches += o->h.auto_lr ? 3 : 2;
    return e;
}

cudaError_t launch_trust(novak_opt *o, const StepCtx &ctx, cudaStream_t stream, int *launches,
                         const char **what)
{
    cudaError_t e;
    if (ctx.trust && !ctx.adapt_in_step) {
        *what = "layer adaptation kernel launch";
        e = novak::launch_trust_stats(o->d_chunks, o->n_chunks, ctx.d_recs, o->n, o->tensor_first,
                                      o->prep_out, ctx.s, o->dyn ? o->d_plan : nullptr,
                                      kernel_variant(ctx.plan), ctx.grad_dtype,
                                      ctx.pre | (o->h.mom16 ? novak::PRE_MOM16 : 0),
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
    if (ctx.pre == novak::PRE_CENTER_ROWS) {
        // no norm is needed: only the means of the rows too long for the step kernel to own
        plan.plain = nullptr;
        plan.n_plain = 0;
        plan.units = o->d_long_units;
        plan.n_units = o->n_long_units;
    } else {
        plan.plain = o->d_plain ? o->d_plain : o->d_chunks;
        plan.n_plain = o->n_plain;
        plan.units = o->d_units;
        plan.n_units = o->n_units;
    }
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
    cfg.pre = ctx.pre | (o->copies.empty() ? 0 : novak::PRE_COPY16) |
              (o->h.mom16 ? novak::PRE_MOM16 : 0);
    if (ctx.adapt_in_step) {
        // statistics and update of the whole group as items of one grid
        cfg.grid = o->n_items + o->adapt_lag;
        o->last_grid = cfg.grid;
        const unsigned epoch = o->adapt_epoch == 0xffffffffu ? 1u : o->adapt_epoch + 1u;
        const cudaError_t e = novak::launch_step_adapt(
            o->d_item_code, o->d_item_chunk, o->n_items, o->adapt_lag, ctx.d_recs, o->prep_out,
            o->tensor_first, o->chunk_u2, o->chunk_p2, o->trust, o->adapt_ctl, o->adapt_arrived,
            o->adapt_ready, o->d_adapt_error, o->adapt_direction, o->adapt_slot_elems, ctx.s, epoch, kernel_variant(ctx.plan), ctx.grad_dtype,
            ctx.la, cfg, stream);
        if (e == cudaSuccess) o->adapt_epoch = epoch;
        return e;
    }
    if (ctx.pre == novak::PRE_CENTER_ROWS) {
        // always the whole group (begin_step chose the mode for a one-launch step)
        o->last_grid = o->n_rest + o->n_own;
        return novak::launch_step_rows(o->d_rest, o->n_rest, o->d_own, o->n_own, ctx.d_recs, ctx.s,
                                       kernel_variant(ctx.plan), ctx.grad_dtype, ctx.la, cfg, stream);
    }
    o->last_grid = cfg.grid;
    return novak::launch_step(o->d_chunks + c0, count, ctx.d_recs, o->prep_out, ctx.trust, ctx.s,
                              kernel_variant(ctx.plan), ctx.grad_dtype, ctx.la, cfg, stream);
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
    DeviceGuard on_device(o->device);
    int rc = check_step_args(o, "step", d_params, d_grads, numel, n, grad_dtype);
    if (rc != NOVAK_OK) return rc;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (o->dyn && (rc = check_dyn(o, "step")) != NOVAK_OK) return rc;
    if (!o->dyn && (rc = refuse_capture(o, "step", stream)) != NOVAK_OK) return rc;
    // Directly behind novak_nesterov_extrapolate (no restore in between) the step
    // reads theta_{t-1} from the save buffer and writes theta_t over Eq. 10's
    // point in the parameter tensors: the restore pass is folded into the step.
    const void *save = nullptr;
    if (o->extrapolated) {
        if (o->dyn) return fail(o, NOVAK_ESTATE, "step: parameters are extrapolated (Eq. 10)");
        if (std::memcmp(o->look_p.data(), d_params, static_cast<size_t>(n) * sizeof(void *)) != 0)
            return fail(o, NOVAK_EINVAL, "step: not the parameter tensors novak_nesterov_extrapolate was given");
        save = o->look_save;
    }
    StepCtx ctx;
    if ((rc = begin_step(o, d_params, d_grads, grad_dtype, stream, &ctx, save, true)) != NOVAK_OK) return rc;
    cudaError_t e;
    int launches = 1;
    const char *what = "";
    if (o->dyn && (rc = prepare_dyn(o, stream)) != NOVAK_OK) return rc;
    if ((e = launch_prepasses(o, ctx, stream, &launches, &what)) != cudaSuccess)
        return fail_cuda(o, e, what);
    if (o->dyn) {
        // the step counter and the scalars live on the device: a captured launch
        // replays as the next step
        novak::LaunchCfg cfg;
        cfg.grid = o->n_chunks;
        if (o->ctas_per_sm > 0) cfg.grid = std::min(o->n_chunks, o->sms * o->ctas_per_sm);
        cfg.reverse = (ctx.pre != novak::PRE_NONE || ctx.trust) ? 1 : 0;   // serpentine needs t: not here
        cfg.pdl = o->pdl;
        cfg.pre = ctx.pre | (o->copies.empty() ? 0 : novak::PRE_COPY16) |
                  (o->h.mom16 ? novak::PRE_MOM16 : 0);
        o->last_grid = cfg.grid;
        if ((e = novak::launch_step_dyn(o->d_chunks, o->n_chunks, ctx.d_recs, o->prep_out, ctx.trust, o->d_plan,
                                        o->h.nesterov, grad_dtype, cfg, stream)) != cudaSuccess)
            return fail_cuda(o, e, "step kernel launch");
        // behind it: the next step's plan, computed while this step runs
        if ((e = novak::launch_plan_next(o->d_plan, &o->h, sizeof o->h, o->pdl, stream)) != cudaSuccess)
            return fail_cuda(o, e, "plan kernel launch");
        launches += 1;
    } else if ((e = launch_range(o, ctx, 0, o->n_chunks, stream)) != cudaSuccess) {
        return fail_cuda(o, e, "step kernel launch");
    }
    if (save) {
        // the parameter tensors hold theta_t now; the save buffer is the caller's again
        o->extrapolated = false;
        o->look_save = nullptr;
    }
    commit_step(o, ctx, launches);
    return NOVAK_OK;
}

int novak_step_begin(novak_opt *o, void *const *d_params, const void *const *d_grads,
                     const int64_t *numel, int n, int grad_dtype, void *stream_)
{
    static_assert(sizeof(StepCtx) <= sizeof(o->half_ctx), "room for the open step");
    if (!o) return NOVAK_EINVAL;
    DeviceGuard on_device(o->device);
    int rc = check_step_args(o, "step_begin", d_params, d_grads, numel, n, grad_dtype);
    if (rc != NOVAK_OK) return rc;
    if (o->dyn) return fail(o, NOVAK_ESTATE, "step_begin: not available with NOVAK_OPT_GRAPH_CAPTURABLE");
    if (o->half_open) return fail(o, NOVAK_ESTATE, "step_begin: the previous step was not finished");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if ((rc = refuse_capture(o, "step_begin", stream)) != NOVAK_OK) return rc;
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
    DeviceGuard on_device(o->device);
    if (!o->half_open) return fail(o, NOVAK_ESTATE, "local_sums: no step is open");
    *d_sums = o->prep_out ? o->prep_out->local_sums : nullptr;
    return NOVAK_OK;
}

int novak_copy_local_sums(novak_opt *o, double *d_dst, void *stream_)
{
    if (!o || !d_dst) return NOVAK_EINVAL;
    DeviceGuard on_device(o->device);
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
    DeviceGuard on_device(o->device);
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
    DeviceGuard on_device(o->device);
    if (!h_params || !h_grads) return fail(o, NOVAK_EINVAL, "step_host: NULL argument");
    int rc = check_step_args(o, "step_host", d_params, const_cast<const void *const *>(d_grads),
                             numel, n, grad_dtype);
    if (rc != NOVAK_OK) return rc;
    if (o->dyn) return fail(o, NOVAK_ESTATE, "step_host: not available with NOVAK_OPT_GRAPH_CAPTURABLE");
    for (int i = 0; i < n; ++i)
        if (!h_params[i] || !h_grads[i] || !d_params[i] || !d_grads[i])
            return fail(o, NOVAK_EINVAL, "step_host: tensor %d has a NULL pointer", i);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if ((rc = refuse_capture(o, "step_host", stream)) != NOVAK_OK) return rc;
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
// Every handle of the process shares the table, so the bookkeeping and the
// sequence "compare owner -> upload -> take token -> launch" run under one
// lock: host threads with a handle each may call at the same time, and a
// launch then always finds the records its own handle uploaded last (given
// that the caller orders the GPU work, e.g. by using one stream).
std::mutex g_noalloc_mutex;
uint64_t g_noalloc_owner[64] = {};
uint64_t g_noalloc_next_token = 1;
}  // namespace

int novak_step_noalloc(novak_opt *o, void *const *d_params, const void *const *d_grads,
                       const int64_t *numel, int n, int grad_dtype, void *stream_)
{
    if (!o) return NOVAK_EINVAL;
    DeviceGuard on_device(o->device);
    if (!o->attached) return fail(o, NOVAK_ESTATE, "step_noalloc: no state attached");
    if (o->extrapolated)
        return fail(o, NOVAK_ESTATE, "step_noalloc: parameters are extrapolated (Eq. 10); call novak_nesterov_restore first");
    if (o->half_open)
        return fail(o, NOVAK_ESTATE, "step_noalloc: a step begun with novak_step_begin is still open");
    if (o->dyn) return fail(o, NOVAK_ESTATE, "step_noalloc: not available with NOVAK_OPT_GRAPH_CAPTURABLE");
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
    {
        const int rc = refuse_capture(o, "step_noalloc", stream);
        if (rc != NOVAK_OK) return rc;
    }

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
            r.p_in = r.p;
            r.g = d_grads[i];
            r.m = slice(o, 0, i);
            r.v = slice(o, 1, i);
            r.slow = la ? static_cast<float *>(slice(o, 2, i)) : nullptr;
            r.acc = traj ? static_cast<float *>(slice(o, 3, i)) : nullptr;
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
    if (dev < 0 || dev >= 64) return fail(o, NOVAK_EINVAL, "step_noalloc: device index %d out of range", dev);
    // From the owner check to the launch nothing of another handle's call may
    // come in between: the table would hold one handle's records while the
    // other handle's kernel reads it.
    std::lock_guard<std::mutex> table_lock(g_noalloc_mutex);
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
    if (o->ctas_per_sm > 0) {
        // NOVAK_OPT_CTAS_PER_SM as in novak_step; the SM count is a device
        // attribute query, not an allocation
        if (o->sms <= 0 &&
            (e = cudaDeviceGetAttribute(&o->sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess)
            return fail_cuda(o, e, "cudaDeviceGetAttribute(SM count)");
        cfg.grid = std::min(n_chunks, o->sms * o->ctas_per_sm);
    }
    cfg.reverse = (o->serpentine && (t % 2 == 0)) ? 1 : 0;
    cfg.pdl = o->pdl;
    cfg.pre = novak::PRE_NONE | (o->copies.empty() ? 0 : novak::PRE_COPY16) |
              (o->h.mom16 ? novak::PRE_MOM16 : 0);
    e = novak::launch_step(d_chunks, n_chunks, d_recs, nullptr, nullptr, s, kernel_variant(p), grad_dtype,
                           la_action, cfg, stream);
    if (e != cudaSuccess) return fail_cuda(o, e, "step kernel launch");

    o->t = t;
    o->launches += 1;
    o->last_plan = p;
    o->last_grid = cfg.grid;
    if (p.is_sync) { o->n_syncs += 1; o->last_sync = t; }
    return NOVAK_OK;
}

// ---- true Nesterov: the look-ahead around the caller's closure (Eq. 10-11) ----

size_t novak_nesterov_save_bytes(const novak_opt *o)
{
    if (!o || !o->attached) return 0;
    return static_cast<size_t>(o->region_elems) * sizeof(float);
}

namespace {

int check_look_args(novak_opt *o, const char *who, void *const *d_params, const void *d_save,
                    size_t save_bytes, const int64_t *numel, int n)
{
    if (!o->attached) return fail(o, NOVAK_ESTATE, "%s: no state attached", who);
    if (o->half_open) return fail(o, NOVAK_ESTATE, "%s: a step begun with novak_step_begin is still open", who);
    if (!o->h.true_requested)
        return fail(o, NOVAK_ESTATE, "%s: the handle was not created with NOVAK_NESTEROV_TRUE", who);
    if (!d_params || !d_save || !numel) return fail(o, NOVAK_EINVAL, "%s: NULL argument", who);
    if (n != o->n || std::memcmp(numel, o->numel.data(), n * sizeof(int64_t)) != 0)
        return fail(o, NOVAK_ESTATE, "%s: tensor list differs from the attached layout", who);
    if (save_bytes < novak_nesterov_save_bytes(o))
        return fail(o, NOVAK_EINVAL, "%s: save buffer holds %zu bytes, %zu needed", who, save_bytes,
                    novak_nesterov_save_bytes(o));
    if (reinterpret_cast<uintptr_t>(d_save) & 15u)
        return fail(o, NOVAK_EINVAL, "%s: save buffer not aligned to 16 bytes", who);
    return NOVAK_OK;
}

int look_grid(const novak_opt *o) { return std::min(o->n_chunks, o->sms * 8); }

}  // namespace

int novak_nesterov_extrapolate(novak_opt *o, void *const *d_params, void *d_save, size_t save_bytes,
                               const int64_t *numel, int n, void *stream_)
{
    if (!o) return NOVAK_EINVAL;
    DeviceGuard on_device(o->device);
    int rc = check_look_args(o, "nesterov_extrapolate", d_params, d_save, save_bytes, numel, n);
    if (rc != NOVAK_OK) return rc;
    if (o->extrapolated)
        return fail(o, NOVAK_ESTATE, "nesterov_extrapolate: parameters are extrapolated already");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (!o->d_chunks && (rc = prepare_device(o, stream)) != NOVAK_OK) return rc;
    if ((rc = prepare_look(o, d_params, stream)) != NOVAK_OK) return rc;
    const cudaError_t e = novak::launch_extrapolate(
        o->d_chunks, o->n_chunks, o->d_look, o->d_state, o->h.mom16, static_cast<float *>(d_save), static_cast<float>(o->h.beta_n), look_grid(o), o->pdl, stream);
    if (e != cudaSuccess) return fail_cuda(o, e, "look-ahead kernel launch");
    o->extrapolated = true;
    o->look_save = d_save;
    o->launches += 1;
    return NOVAK_OK;
}

int novak_nesterov_restore(novak_opt *o, void *const *d_params, const void *d_save, size_t save_bytes,
                           const int64_t *numel, int n, void *stream_)
{
    if (!o) return NOVAK_EINVAL;
    DeviceGuard on_device(o->device);
    int rc = check_look_args(o, "nesterov_restore", d_params, d_save, save_bytes, numel, n);
    if (rc != NOVAK_OK) return rc;
    if (!o->extrapolated)
        return fail(o, NOVAK_ESTATE, "nesterov_restore: nothing to restore");
    if (d_save != o->look_save ||
        std::memcmp(o->look_p.data(), d_params, static_cast<size_t>(n) * sizeof(void *)) != 0)
        return fail(o, NOVAK_EINVAL, "nesterov_restore: not the buffers novak_nesterov_extrapolate was given");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const cudaError_t e = novak::launch_restore(o->d_chunks, o->n_chunks, o->d_look,
                                                static_cast<const float *>(d_save), look_grid(o), o->pdl, stream);
    if (e != cudaSuccess) return fail_cuda(o, e, "restore kernel launch");
    o->extrapolated = false;
    o->look_save = nullptr;
    o->launches += 1;
    return NOVAK_OK;
}

int novak_get_grad_stats(novak_opt *o, double *norm, double *factor, void *stream_)
{
    if (!o) return NOVAK_EINVAL;
    DeviceGuard on_device(o->device);
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
    DeviceGuard on_device(o->device);
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
    DeviceGuard on_device(o->device);
    if (!h_out || n != o->n) return fail(o, NOVAK_EINVAL, "get_trust_ratios: NULL or wrong tensor count");
    if (!o->trust || o->t == 0) return fail(o, NOVAK_ESTATE, "get_trust_ratios: no step with layer adaptation yet");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    cudaError_t e;
    if ((e = cudaMemcpyAsync(h_out, o->trust, n * sizeof(float), cudaMemcpyDeviceToHost, stream)) != cudaSuccess ||
        (e = cudaStreamSynchronize(stream)) != cudaSuccess)
        return fail_cuda(o, e, "get_trust_ratios");
    return NOVAK_OK;
}

int novak_selftest_bounded_wait(novak_opt *o, int *gave_up, double *seconds, void *stream_)
{
    if (!o) return NOVAK_EINVAL;
    DeviceGuard on_device(o->device);
    if (!gave_up || !seconds) return fail(o, NOVAK_EINVAL, "selftest_bounded_wait: NULL output");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    // [0]: the word nobody publishes, [1]: the error word, [2..3]: the kernel's report
    unsigned long long *d = nullptr;
    cudaError_t e = cudaMalloc(reinterpret_cast<void **>(&d), 4 * sizeof(unsigned long long));
    if (e != cudaSuccess) return fail(o, NOVAK_ENOMEM, "selftest_bounded_wait: %s", cudaGetErrorString(e));
    unsigned long long h[2] = {~0ull, 0ull};
    if ((e = cudaMemsetAsync(d, 0, 4 * sizeof(unsigned long long), stream)) == cudaSuccess &&
        (e = novak::launch_adapt_wait_probe(d, 1u, reinterpret_cast<const unsigned *>(d + 1), d + 2,
                                            stream)) == cudaSuccess &&
        (e = cudaMemcpyAsync(h, d + 2, sizeof h, cudaMemcpyDeviceToHost, stream)) == cudaSuccess)
        e = cudaStreamSynchronize(stream);
    cudaFree(d);
    if (e != cudaSuccess) return fail_cuda(o, e, "selftest_bounded_wait");
    *gave_up = h[0] == 0ull ? 1 : 0;
    *seconds = static_cast<double>(h[1]) * 1e-9;
    return NOVAK_OK;
}

}  // extern "C"
