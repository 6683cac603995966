// Host side of the NOVAK step library, part 1: hyperparameter validation, the
// per-step scalar plan (double precision), the chunk and row-unit tables, the
// state layout and the entry points that touch no kernel.  Declarations and
// argument contracts are in include/novak.h.
#include "novak_handle.h"

#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>

using namespace novak_host;

namespace novak_host {

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
            // CTA's 8 warps), else up to 256 rows per unit (eight lanes per row from 32
            // elements on, a thread per row below)
            // (rows per unit a multiple of 8, so that no warp idles while others take a
            // second row)
            // (16 where two rows share a warp)
            const uint32_t step = L <= novak::kRowHalfWarpMax ? 16u : 8u;
            const uint32_t per = L >= 128u ? std::max(step, novak::kRowUnitElems / L / step * step)
                                           : novak::kRowUnitThreads;
            for (uint32_t r = 0; r < R; r += per)
                out.push_back(RowUnit{i, r, std::min(per, R - r), 0u, 0u, 1u, 0u, 0u});
        }
    }
}


void build_own_units(const int64_t *numel, const int64_t *rows, int n, std::vector<RowUnit> &out)
{
    out.clear();
    for (int i = 0; i < n; ++i) {
        if (rows[i] <= 0) continue;
        const uint32_t R = static_cast<uint32_t>(rows[i]);
        const uint32_t L = static_cast<uint32_t>(numel[i] / rows[i]);
        if (L == 0 || L > novak::kOwnRowMax) continue;
        const uint32_t per = std::max(1u, std::min(novak::kOwnUnitRows, novak::kOwnUnitElems / L));
        for (uint32_t r = 0; r < R; r += per)
            out.push_back(RowUnit{i, r, std::min(per, R - r), 0u, 0u, 1u, 0u, 0u});
    }
}

int64_t build_adapt_items(const std::vector<int> &tensor_first, int n, int64_t lead_entries, int group,
                          std::vector<int32_t> &items, std::vector<int32_t> &counts)
{
    items.clear();
    counts.clear();
    if (n <= 0) return 0;
    // A tensor's first entry (the only one besides its last that may be short) stands
    // alone; the others go in runs of `group`.
    int64_t longest = 0;                // items of the tensor that has most
    for (int i = 0; i < n; ++i) {
        const size_t before = items.size();
        int c = tensor_first[i];
        const int c1 = tensor_first[i + 1];
        while (c < c1) {
            const int cnt = (c == tensor_first[i]) ? 1 : std::min(group, c1 - c);
            items.push_back(c);
            counts.push_back(cnt);
            c += cnt;
        }
        longest = std::max<int64_t>(longest, static_cast<int64_t>(items.size() - before));
    }
    // every S part a U part waits for has a lower block index, or is the CTA's own
    return std::max<int64_t>(longest - 1, 0) + (lead_entries + group - 1) / group;
}

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

void *slice(const novak_opt *o, int array, int i)
{
    const int64_t mb = moment_bytes(o->h);
    const int64_t elem = o->slot_off[i] + o->phase[i];
    if (array < 2) return o->d_state + (array * o->region_elems + elem) * mb;
    return o->d_state + 2 * o->region_elems * mb + ((array - 2) * o->region_elems + elem) * 4;
}

size_t state_bytes_for(const Hyper &h, int64_t region_elems)
{
    return static_cast<size_t>(region_elems) *
           (2 * moment_bytes(h) + sizeof(float) * (n_state_arrays(h) - 2));
}

int pre_mode(const novak_opt *o)
{
    if (o->h.centralize && o->total_rows > 0) return novak::PRE_CENTER;
    if (o->h.clip > 0.0 || o->h.auto_lr) return novak::PRE_SCALE;
    return novak::PRE_NONE;
}

int step_pre_mode(const novak_opt *o, bool whole_table)
{
    const int pre = pre_mode(o);
    if (pre == novak::PRE_CENTER && whole_table && o->center_in_step && !o->dyn &&
        !(o->h.clip > 0.0) && !o->h.auto_lr && !o->h.layer_adapt)
        return novak::PRE_CENTER_ROWS;
    return pre;
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
    out->nesterov_variant = p.nesterov;
    out->lookahead_mode = o->h.la_mode;
    out->lookahead_k = o->h.la_k;
    out->n_tensors = o->n;
    out->n_chunks = o->n_chunks;
    out->grid = o->last_grid;
    out->block = novak::step_block_threads();
    out->warnings = o->warnings;
    out->grad_processing = pre_mode(o);
    out->layer_adaptation = o->h.layer_adapt;
    out->moment_dtype = o->h.mom16 ? NOVAK_MOMENT_BF16 : NOVAK_MOMENT_F32;
    out->beta1_t = p.beta1_t;
    out->beta2_t = p.beta2_t;
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

}  // namespace novak_host

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
    h.true_requested = 0;
    h.true_steps = 0;
    h.mom16 = 0;
    if (nesterov_variant == NOVAK_NESTEROV_TRUE) {
        // N_taylor = 0 until NOVAK_OPT_TRUE_NESTEROV_STEPS says otherwise: every
        // step runs the approximation (Section 7.3's downgrade), with a warning
        h.nesterov = NOVAK_NESTEROV_APPROX;
        h.true_requested = 1;
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
    DeviceGuard on_device(opt->device);
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
    case NOVAK_OPT_LR: h.lr = value; o->dyn_upload_rates = true; break;
    case NOVAK_OPT_WEIGHT_DECAY: h.wd = value; o->dyn_upload_rates = true; break;
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
    case NOVAK_OPT_MOMENT_DTYPE:
        if (o->attached) return fail(o, NOVAK_ESTATE, "moment dtype changes the state layout: set it before attach");
        if (value != NOVAK_MOMENT_F32 && value != NOVAK_MOMENT_BF16)
            return fail(o, NOVAK_EINVAL, "unknown moment dtype");
        h.mom16 = value == NOVAK_MOMENT_BF16 ? 1 : 0;
        break;
    case NOVAK_OPT_TRUE_NESTEROV_STEPS:
        if (!h.true_requested)
            return fail(o, NOVAK_ESTATE, "true_nesterov_steps: the handle was not created with NOVAK_NESTEROV_TRUE");
        if (o->extrapolated)
            return fail(o, NOVAK_ESTATE, "true_nesterov_steps: parameters are extrapolated; restore them first");
        if (!(value >= 0.0 && value <= 2147483647.0) || value != std::floor(value))
            return fail(o, NOVAK_EINVAL, "true_nesterov_steps must be an integer >= 0");
        h.true_steps = static_cast<int>(value);
        if (h.true_steps > 0) o->warnings &= ~static_cast<uint32_t>(NOVAK_WARN_TRUE_DOWNGRADED);
        else o->warnings |= NOVAK_WARN_TRUE_DOWNGRADED;
        break;
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
    case NOVAK_OPT_LAYER_ADAPTATION_IN_STEP:
        if (value != 0.0 && value != 1.0) return fail(o, NOVAK_EINVAL, "layer_adaptation_in_step must be 0 or 1");
        o->adapt_in_step = static_cast<int>(value);
        return NOVAK_OK;
    case NOVAK_OPT_LAYER_ADAPTATION_LEAD:
        if (o->d_adapt) return fail(o, NOVAK_ESTATE, "the lead is fixed once a step with layer adaptation was taken");
        if (!(value >= 0.0 && value <= 1073741824.0) || value != std::floor(value))
            return fail(o, NOVAK_EINVAL, "layer_adaptation_lead must be an integer in [0, 2^30]");
        o->adapt_lead_elems = static_cast<int64_t>(value);
        return NOVAK_OK;
    case NOVAK_OPT_LAYER_ADAPTATION_GROUP:
        if (o->d_adapt) return fail(o, NOVAK_ESTATE, "the group is fixed once a step with layer adaptation was taken");
        if (!(value >= 1.0 && value <= double(novak::kAdaptGroupMax)) || value != std::floor(value))
            return fail(o, NOVAK_EINVAL, "layer_adaptation_group must be an integer in [1, %d]", novak::kAdaptGroupMax);
        o->adapt_group = static_cast<int>(value);
        return NOVAK_OK;
    case NOVAK_OPT_CENTRALIZE_IN_STEP:
        if (value != 0.0 && value != 1.0) return fail(o, NOVAK_EINVAL, "centralize_in_step must be 0 or 1");
        o->center_in_step = static_cast<int>(value);
        return NOVAK_OK;
    case NOVAK_OPT_GRAPH_CAPTURABLE:
        if (o->t > 0) return fail(o, NOVAK_ESTATE, "graph_capturable is fixed once a step was taken");
        if (value != 0.0 && value != 1.0) return fail(o, NOVAK_EINVAL, "graph_capturable must be 0 or 1");
        o->dyn = static_cast<int>(value);
        return NOVAK_OK;
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
    case NOVAK_OPT_TRUE_NESTEROV_STEPS: *value = o->h.true_steps; break;
    case NOVAK_OPT_MOMENT_DTYPE: *value = o->h.mom16 ? NOVAK_MOMENT_BF16 : NOVAK_MOMENT_F32; break;
    case NOVAK_OPT_LAYER_ADAPTATION: *value = o->h.layer_adapt; break;
    case NOVAK_OPT_ADAPTIVE_BETA: *value = o->h.adaptive_beta; break;
    case NOVAK_OPT_BETA1_TAU: *value = o->h.tau1; break;
    case NOVAK_OPT_BETA2_TAU: *value = o->h.tau2; break;
    case NOVAK_OPT_CLIP_THRESHOLD: *value = o->h.clip; break;
    case NOVAK_OPT_CENTRALIZE: *value = o->h.centralize; break;
    case NOVAK_OPT_GRAPH_CAPTURABLE: *value = o->dyn; break;
    case NOVAK_OPT_CENTRALIZE_IN_STEP: *value = o->center_in_step; break;
    case NOVAK_OPT_LAYER_ADAPTATION_IN_STEP: *value = o->adapt_in_step; break;
    case NOVAK_OPT_LAYER_ADAPTATION_LEAD: *value = static_cast<double>(o->adapt_lead_elems); break;
    case NOVAK_OPT_LAYER_ADAPTATION_GROUP: *value = o->adapt_group; break;
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
    return state_bytes_for(o->h, region);
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
    // the device the buffer lives on becomes the handle's device
    int device = -1;
    cudaPointerAttributes attr;
    if (cudaPointerGetAttributes(&attr, d_state) == cudaSuccess && attr.type == cudaMemoryTypeDevice)
        device = attr.device;
    else
        (void)cudaGetLastError();       // not a device pointer the runtime knows: no guard
    {
        DeviceGuard on_device(device);
        cudaError_t e = cudaMemsetAsync(d_state, 0, need, static_cast<cudaStream_t>(stream));
        if (e != cudaSuccess) return fail_cuda(o, e, "cudaMemsetAsync(state)");
    }
    {
        DeviceGuard old_device(o->device);   // a previous attachment's tables are freed where they live
        release_device(o);
    }
    o->device = device;

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

extern "C" {

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

int novak_get_info(const novak_opt *o, novak_info *out)
{
    if (!o || !out) return NOVAK_EINVAL;
    DeviceGuard on_device(o->device);
    fill_info(o, o->last_plan, out);
    if (o->dyn && o->d_plan) {
        // replays of a captured step advance only the device's counters
        novak::DevPlan dp;
        if (read_dyn(o, &dp) != NOVAK_OK) return NOVAK_ECUDA;
        // dp.t is the step that runs next; the last one's plan is in the other slot
        out->t = dp.t - 1; out->n_syncs = dp.n_syncs; out->last_sync_step = dp.last_sync;
        if (dp.t > 1) {
            const novak::PlanSlot &s = dp.slot[(dp.t - 1) & 1];
            out->bc1 = s.bc1; out->bc2 = s.bc2; out->rho_inf = s.rho_inf; out->rho_t = s.rho_t;
            out->r_t = s.r_t; out->step_size = s.step_size; out->decay = s.decay;
            out->rect_branch = s.rect_branch; out->is_sync = s.is_sync;
            out->nesterov_variant = s.nesterov;
            out->beta1_t = s.beta1_t; out->beta2_t = s.beta2_t;
        }
    }
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
    DeviceGuard on_device(o->device);
    std::memset(out, 0, sizeof *out);
    out->magic = kMetaMagic;
    out->t = o->t; out->n_syncs = o->n_syncs; out->last_sync_step = o->last_sync;
    if (o->dyn && o->d_plan) {
        novak::DevPlan dp;
        if (read_dyn(o, &dp) != NOVAK_OK) return NOVAK_ECUDA;
        out->t = dp.t - 1; out->n_syncs = dp.n_syncs; out->last_sync_step = dp.last_sync;
    }
    out->total_numel = o->total_numel;
    out->lr = o->h.lr; out->beta1 = o->h.beta1; out->beta2 = o->h.beta2; out->eps = o->h.eps;
    out->weight_decay = o->h.wd; out->nesterov_beta = o->h.beta_n;
    out->lookahead_alpha = o->h.la_alpha;
    out->nesterov_variant = o->h.true_requested ? NOVAK_NESTEROV_TRUE : o->h.nesterov;
    out->true_nesterov_steps = o->h.true_steps;
    out->moment_dtype = o->h.mom16 ? NOVAK_MOMENT_BF16 : NOVAK_MOMENT_F32;
    out->lookahead_k = o->h.la_k;
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
    if (o->extrapolated) return fail(o, NOVAK_ESTATE, "import: parameters are extrapolated; restore them first");
    if (in->n_tensors != o->n || in->total_numel != o->total_numel ||
        in->lookahead_k != o->h.la_k || in->lookahead_mode != o->h.la_mode ||
        (in->moment_dtype == NOVAK_MOMENT_BF16) != (o->h.mom16 != 0))
        return fail(o, NOVAK_ESTATE, "import: tensor list, lookahead layout or moment dtype differs");
    if (in->t < 0 || in->n_syncs < 0) return fail(o, NOVAK_EINVAL, "import: negative counter");
    Hyper h = o->h;
    h.lr = in->lr; h.beta1 = in->beta1; h.beta2 = in->beta2; h.eps = in->eps;
    h.wd = in->weight_decay; h.beta_n = in->nesterov_beta; h.la_alpha = in->lookahead_alpha;
    h.nesterov = in->nesterov_variant; h.rectified = in->rectified;
    h.true_requested = 0;
    h.true_steps = 0;
    if (in->nesterov_variant == NOVAK_NESTEROV_TRUE) {
        if (in->true_nesterov_steps < 0) return fail(o, NOVAK_EINVAL, "import: negative true_nesterov_steps");
        h.nesterov = NOVAK_NESTEROV_APPROX;
        h.true_requested = 1;
        h.true_steps = in->true_nesterov_steps;
    }
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
    o->dyn_upload_counters = o->dyn_upload_rates = true;
    o->warnings |= in->warnings;
    if (h.true_requested) {
        if (h.true_steps > 0) o->warnings &= ~static_cast<uint32_t>(NOVAK_WARN_TRUE_DOWNGRADED);
        else o->warnings |= NOVAK_WARN_TRUE_DOWNGRADED;
    }
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

int64_t novak_build_own_units(const int64_t *numel, const int64_t *rows, int n, int32_t *tensor,
                              int64_t *row0, int64_t *n_rows, int64_t cap)
{
    if (!numel || !rows || n <= 0 || cap < 0) return -1;
    for (int i = 0; i < n; ++i)
        if (numel[i] <= 0 || rows[i] < 0 || (rows[i] > 0 && (numel[i] % rows[i] != 0 ||
                                                             numel[i] >= (int64_t(1) << 31))))
            return -1;
    std::vector<RowUnit> units;
    build_own_units(numel, rows, n, units);
    const int64_t count = static_cast<int64_t>(units.size());
    for (int64_t i = 0; i < count && i < cap; ++i) {
        if (tensor) tensor[i] = units[i].tensor;
        if (row0) row0[i] = units[i].row0;
        if (n_rows) n_rows[i] = units[i].n_rows;
    }
    return count;
}

int64_t novak_build_adapt_order(const int32_t *tensor_first, int n, int64_t lead_entries, int group,
                                int32_t *out, int32_t *count, int64_t cap, int64_t *lag)
{
    if (!tensor_first || n <= 0 || lead_entries < 0 || cap < 0 || tensor_first[0] != 0 ||
        group < 1 || group > novak::kAdaptGroupMax)
        return -1;
    for (int i = 0; i < n; ++i)
        if (tensor_first[i + 1] < tensor_first[i]) return -1;
    std::vector<int> first(tensor_first, tensor_first + n + 1);
    std::vector<int32_t> items, counts;
    const int64_t l = build_adapt_items(first, n, lead_entries, group, items, counts);
    if (lag) *lag = l;
    const int64_t total = static_cast<int64_t>(items.size());
    for (int64_t i = 0; i < total && i < cap; ++i) {
        if (out) out[i] = items[i];
        if (count) count[i] = counts[i];
    }
    return total;
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
