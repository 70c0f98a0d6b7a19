// C ABI of libams: argument checks, workspace layout and kernel sequencing.  No
// device memory is allocated here; nothing crosses to the host between kernels.
#include <new>
#include <string.h>

#include "ams_common.cuh"

namespace ams {

struct Layout {
    size_t status, eff_lens, seq_bad, scores, usage, logits, ex_logits, cbuf, n_seg, raw_cuts, seg_bounds, quotas, keep_idx, part, fin, total;
    int units, T_cap, seg_cap, n_slices, slice_len, rows_pad_cap;
};

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

static bool config_ok(const ams_config *c, int *why)
{
    *why = AMS_ERR_INVALID_ARG;
    if (!c) return false;
    if (c->n_layers < 1 || c->n_q_heads < 1 || c->n_kv_heads < 1 || c->max_batch < 1) return false;
    if (c->max_seq_len < kPage || c->max_seq_len > 131072 || c->max_seq_len % kPage) return false;
    if (c->max_window < 0 || c->max_budget < 1 || c->max_budget >= c->max_seq_len) return false;
    if (c->max_segments < 1 || c->max_segments > 1024) return false;
    if (c->l_min < 1 || c->l_max < 0 || c->q_min < 0 || c->n_sink < 0 || c->n_last < 0) return false;
    if (!(c->ema_lambda >= 0.0f && c->ema_lambda < 1.0f)) return false;
    if (!(c->ema_beta >= 0.0f && c->ema_beta <= 1.0f)) return false;
    if (!(c->eps > 0.0f) || !(c->eps < 1e30f)) return false;
    if (c->pool_kernel < 1 || c->pool_kernel > 63 || !(c->pool_kernel & 1)) return false;
    if (c->decoupled != 0 && c->decoupled != 1) return false;
    if ((c->fixed_segments != 0 && c->fixed_segments != 1) || (c->uniform_quotas != 0 && c->uniform_quotas != 1)) return false;
    if (c->expected_scorer != 0 && c->expected_scorer != 1) return false;
    *why = AMS_ERR_UNSUPPORTED;
    if (c->head_dim != kHeadDim || c->page_size != kPage) return false;
    if (c->n_q_heads % c->n_kv_heads) return false;
    const long long sc = (long long)c->max_segments + (c->l_max > 0 ? 2LL * (c->max_seq_len / c->l_max) : 0) + 4;
    if (sc > 4096) return false;
    *why = AMS_OK;
    return true;
}

static int segment_capacity(const ams_config *c)
{
    return c->max_segments + (c->l_max > 0 ? 2 * (c->max_seq_len / c->l_max) : 0) + 4;
}

// Token slices of the scorer kernels: at most 32 per sequence, at least 512 tokens.
static void slicing(int T_cap, int *slice_len, int *n_slices)
{
    int sl = 512;
    const int need = (T_cap + 31) / 32;
    if (need > sl) sl = (need + 63) / 64 * 64;
    *slice_len = sl;
    *n_slices = (T_cap + sl - 1) / sl;
}

static int rows_padded(int rows)
{
    if (rows >= 64) return (rows + 127) / 128 * 128; // tensor-core scorer: 128-row query blocks
    const int rb = tova_rows_block(rows < 1 ? 1 : rows);
    return (rows + rb - 1) / rb * rb;
}

// Tensor-core scorer: a block takes at least this many 128-token tiles, so that a unit is
// shared by at most 31 blocks.
static int tc_tiles_per_block_min(int T_cap)
{
    const int tiles = (T_cap + 127) / 128;
    const int need = (tiles + 29) / 30;
    return need > 8 ? need : 8;
}

static Layout make_layout(const ams_config *c)
{
    Layout y;
    y.units = c->n_layers * c->max_batch * c->n_kv_heads;
    y.T_cap = c->max_seq_len;
    y.seg_cap = segment_capacity(c);
    slicing(y.T_cap, &y.slice_len, &y.n_slices);
    const int tc_parts = ((y.T_cap + 127) / 128 + tc_tiles_per_block_min(y.T_cap) - 1) / tc_tiles_per_block_min(y.T_cap) + 1;
    if (tc_parts > y.n_slices) y.n_slices = tc_parts;
    const int rows_cap = (c->n_q_heads / c->n_kv_heads) * (c->max_window > 0 ? c->max_window : 1);
    y.rows_pad_cap = rows_padded(rows_cap);
    const size_t U = (size_t)y.units, T = (size_t)y.T_cap;
    size_t off = 0;
    y.status = off;     off = align_up(off + 64, 256);
    y.eff_lens = off;   off = align_up(off + (size_t)c->max_batch * 4, 256);
    y.seq_bad = off;    off = align_up(off + (size_t)c->max_batch * 4, 256);
    y.scores = off;     off = align_up(off + U * T * 4, 256);
    // second per-token array: the usage when it is smoothed or comes from another scorer than the base scores
    y.usage = off;      off = align_up(off + ((c->pool_kernel > 1 || c->decoupled) ? U * T * 4 : 0), 256);
    y.cbuf = off;       off = align_up(off + U * T * 8, 256);
    y.n_seg = off;      off = align_up(off + U * 4, 256);
    y.raw_cuts = off;   off = align_up(off + U * (size_t)(c->max_segments + 1) * 4, 256);
    y.seg_bounds = off; off = align_up(off + U * (size_t)(y.seg_cap + 1) * 4, 256);
    y.quotas = off;     off = align_up(off + U * (size_t)y.seg_cap * 4, 256);
    y.keep_idx = off;   off = align_up(off + U * (size_t)c->max_budget * 4, 256);
    const size_t part_per = (size_t)y.n_slices * (size_t)(y.rows_pad_cap * 2 > kHeadDim ? y.rows_pad_cap * 2 : kHeadDim) * 4;
    y.part = off;       off = align_up(off + U * part_per, 256);
    const size_t fin_per = (size_t)((y.rows_pad_cap > kHeadDim ? y.rows_pad_cap : kHeadDim) + 8) * 4;
    y.fin = off;        off = align_up(off + U * fin_per, 256);
    // narrow query blocks keep their logits (rows_pad floats per token, at most 1/4 of the K bytes) so that
    // the usage pass need not read K again
    y.logits = off;     off = align_up(off + (y.rows_pad_cap <= 16 && c->max_window > 0 ? U * T * (size_t)y.rows_pad_cap * 4 : 0), 256);
    // expected-attention scorer: one logit per (query head, token), so that K is read once
    y.ex_logits = off;  off = align_up(off + (c->expected_scorer ? U * T * (size_t)(c->n_q_heads / c->n_kv_heads) * 4 : 0), 256);
    y.total = off;
    return y;
}

} // namespace ams

using namespace ams;

struct ams_state {
    ams_config cfg;
    Layout lay;
    unsigned char *ws;
    void *ema;
    int32_t last_launches;
    cudaEvent_t ev[32];
    const float *q_mean; // query statistics of the expected-attention scorer (ams_set_query_stats)
    const void *q_cov;
    float score_eps;
    bool profiling;
    int n_ev;
    int ev_ids[32];
};

extern "C" {

void ams_config_default(ams_config *cfg)
{
    if (!cfg) return;
    memset(cfg, 0, sizeof *cfg);
    cfg->head_dim = kHeadDim;
    cfg->page_size = kPage;
    cfg->max_segments = 32;
    cfg->l_min = 16;
    cfg->l_max = 256;
    cfg->q_min = 1;
    cfg->n_sink = 4;
    cfg->n_last = 16;
    cfg->ema_lambda = 0.9f;
    cfg->ema_beta = 0.9f;
    cfg->eps = 1e-8f;
    cfg->causal_window = 1;
    cfg->pool_kernel = 1;
    cfg->decoupled = 0;
    cfg->fixed_segments = 0;
    cfg->uniform_quotas = 0;
    cfg->expected_scorer = 0;
}

size_t ams_ema_state_bytes(const ams_config *cfg)
{
    int why;
    if (!config_ok(cfg, &why)) return 0;
    return (size_t)cfg->n_layers * cfg->max_batch * cfg->n_kv_heads * (size_t)cfg->max_seq_len * 4;
}

size_t ams_workspace_bytes(const ams_config *cfg)
{
    int why;
    if (!config_ok(cfg, &why)) return 0;
    return make_layout(cfg).total;
}

int32_t ams_segment_capacity(const ams_config *cfg)
{
    int why;
    if (!config_ok(cfg, &why)) return 0;
    return segment_capacity(cfg);
}

int ams_init_state(const ams_config *cfg, void *ema_state, void *workspace, size_t workspace_bytes,
                   void *stream, ams_state **out)
{
    int why;
    if (!out) return AMS_ERR_INVALID_ARG;
    *out = nullptr;
    if (!config_ok(cfg, &why)) return why;
    if (!ema_state || !workspace || ((uintptr_t)workspace & 255) || ((uintptr_t)ema_state & 15)) return AMS_ERR_INVALID_ARG;
    const Layout lay = make_layout(cfg);
    if (workspace_bytes < lay.total) return AMS_ERR_CAPACITY;
    cudaStream_t s = (cudaStream_t)stream;
    if (cudaMemsetAsync(ema_state, 0, ams_ema_state_bytes(cfg), s) != cudaSuccess) return AMS_ERR_CUDA;
    // status word, effective lengths and error flags; kept positions and segment counts start from zero so that
    // nothing downstream ever indexes with an uninitialised value
    if (cudaMemsetAsync(workspace, 0, lay.scores, s) != cudaSuccess) return AMS_ERR_CUDA;
    if (cudaMemsetAsync((unsigned char *)workspace + lay.n_seg, 0, lay.raw_cuts - lay.n_seg, s) != cudaSuccess) return AMS_ERR_CUDA;
    if (cudaMemsetAsync((unsigned char *)workspace + lay.keep_idx, 0, lay.part - lay.keep_idx, s) != cudaSuccess) return AMS_ERR_CUDA;
    ams_state *st = new (std::nothrow) ams_state;
    if (!st) return AMS_ERR_INTERNAL;
    st->cfg = *cfg;
    st->lay = lay;
    st->ws = (unsigned char *)workspace;
    st->ema = ema_state;
    st->last_launches = 0;
    st->q_mean = nullptr;
    st->q_cov = nullptr;
    st->score_eps = 0.0f;
    st->profiling = false;
    st->n_ev = 0;
    *out = st;
    return AMS_OK;
}

int ams_compress(ams_state *st, void *k_pages, void *v_pages, int64_t num_pages, int32_t *block_table,
                 int32_t block_table_stride, int32_t *seq_lens, int32_t batch, const void *obs_queries,
                 int32_t window, void *ema_state, int32_t budget, int32_t n_segments, int32_t scorer_id,
                 const int32_t *dst_pages, const float *ext_scores, const float *ext_usage, const ams_debug_views *dbg,
                 void *stream)
{
    if (!st || !k_pages || !v_pages || !block_table || !seq_lens || !ema_state || !dst_pages) return AMS_ERR_INVALID_ARG;
    const ams_config &c = st->cfg;
    if (batch < 1 || batch > c.max_batch || num_pages < 1) return AMS_ERR_INVALID_ARG;
    if (budget < 1 || budget > c.max_budget) return AMS_ERR_INVALID_ARG;
    if (n_segments < 1 || n_segments > c.max_segments) return AMS_ERR_INVALID_ARG;
    if (block_table_stride < (budget + kPage - 1) / kPage) return AMS_ERR_INVALID_ARG;
    if (scorer_id == AMS_SCORER_TOVA) {
        if (!obs_queries || window < 1 || window > c.max_window) return AMS_ERR_INVALID_ARG;
    } else if (scorer_id == AMS_SCORER_EXTERNAL) {
        if (!ext_scores) return AMS_ERR_INVALID_ARG;
    } else if (scorer_id == AMS_SCORER_EXPECTED) {
        if (!c.expected_scorer) return AMS_ERR_CAPACITY; // no room was reserved for the logits
        if (!st->q_mean || !st->q_cov) return AMS_ERR_INVALID_ARG;
    } else if (scorer_id != AMS_SCORER_KEYDIFF) {
        return AMS_ERR_INVALID_ARG;
    }
    if (ext_usage && scorer_id != AMS_SCORER_EXTERNAL) return AMS_ERR_INVALID_ARG;
    // key-only base scores with the window attention as mass signal
    const bool split = (scorer_id == AMS_SCORER_KEYDIFF || scorer_id == AMS_SCORER_EXPECTED) && c.decoupled && obs_queries && window >= 1;
    if (split && window > c.max_window) return AMS_ERR_INVALID_ARG;
    if (((uintptr_t)k_pages | (uintptr_t)v_pages | (uintptr_t)obs_queries | (uintptr_t)ema_state | (uintptr_t)ext_scores |
         (uintptr_t)ext_usage) & 15) return AMS_ERR_INVALID_ARG;

    const Layout &y = st->lay;
    cudaStream_t s = (cudaStream_t)stream;
    DevParams p;
    memset(&p, 0, sizeof p);
    p.L = c.n_layers; p.B = batch; p.Bmax = c.max_batch; p.H = c.n_kv_heads; p.G = c.n_q_heads / c.n_kv_heads;
    p.W = scorer_id == AMS_SCORER_TOVA ? window : 0;
    p.rows = p.G * (p.W > 0 ? p.W : 1);
    p.T_cap = y.T_cap; p.seg_cap = y.seg_cap; p.Tk = budget; p.S = n_segments; p.n_dst = (budget + kPage - 1) / kPage;
    p.l_min = c.l_min; p.l_max = c.l_max; p.q_min = c.q_min; p.n_sink = c.n_sink; p.n_last = c.n_last;
    p.causal = c.causal_window ? 1 : 0;
    p.fixed_seg = c.fixed_segments; p.uniform_q = c.uniform_quotas;
    p.lambda = c.ema_lambda; p.beta = c.ema_beta; p.eps = c.eps;
    p.k_pages = (__nv_bfloat16 *)k_pages; p.v_pages = (__nv_bfloat16 *)v_pages; p.num_pages = num_pages;
    p.block_table = block_table; p.bt_stride = block_table_stride;
    p.seq_lens = (const int *)(st->ws + y.eff_lens); p.seq_lens_out = seq_lens;
    p.seq_bad = (int *)(st->ws + y.seq_bad);
    p.q = (const __nv_bfloat16 *)obs_queries; p.ema = (float *)ema_state; p.dst_pages = dst_pages;
    p.scores = (float *)(st->ws + y.scores);
    p.usage = p.scores;
    if (scorer_id == AMS_SCORER_EXTERNAL) {
        p.scores = const_cast<float *>(ext_scores);
        p.usage = ext_usage ? ext_usage : ext_scores;
    }
    float *usage_buf = (float *)(st->ws + y.usage);
    p.cbuf = (u64 *)(st->ws + y.cbuf);
    p.n_seg = (int *)(st->ws + y.n_seg); p.seg_bounds = (int *)(st->ws + y.seg_bounds);
    p.quotas = (int *)(st->ws + y.quotas); p.keep_idx = (int *)(st->ws + y.keep_idx);
    p.raw_cuts = (int *)(st->ws + y.raw_cuts);
    p.mass_dbg = dbg ? dbg->mass : nullptr;
    p.part = (float *)(st->ws + y.part); p.fin = (float *)(st->ws + y.fin);
    p.slice_len = y.slice_len; p.n_slices = y.n_slices;
    p.rows_pad = scorer_id == AMS_SCORER_TOVA ? rows_padded(p.rows) : kHeadDim;
    p.tc_tpc_min = tc_tiles_per_block_min(y.T_cap);
    p.tc_stages = p.rows_pad <= 256 ? 4 : 2; // even: each stage then belongs to one of the two MMA issuers
    p.status = (int *)(st->ws + y.status);
    p.logits = (y.rows_pad_cap <= 16 && c.max_window > 0) ? (float *)(st->ws + y.logits) : nullptr;
    p.q_mean = st->q_mean; p.q_cov = (const __nv_bfloat16 *)st->q_cov; p.score_eps = st->score_eps;
    p.ex_logits = c.expected_scorer ? (float *)(st->ws + y.ex_logits) : nullptr;

    int rc = AMS_OK;
    LaunchCtx ctx;
    ctx.s = s;
    ctx.ev = st->profiling ? st->ev : nullptr;
    ctx.max_ev = 32;
    ctx.begin();
    // lengths and page ids are checked once, on the device, before anything forms an address from them
    p.W = (scorer_id == AMS_SCORER_TOVA || split) ? window : 0;
    rc = launch_prepare(p, seq_lens, (int *)(st->ws + y.eff_lens), ctx);
    p.W = scorer_id == AMS_SCORER_TOVA ? window : 0;
    if (rc == AMS_OK && scorer_id == AMS_SCORER_TOVA) {
        rc = launch_score_tova(p, ctx);
    } else if (rc == AMS_OK && (scorer_id == AMS_SCORER_KEYDIFF || scorer_id == AMS_SCORER_EXPECTED)) {
        if (split) {
            // the window attention goes through the score array into the usage array (smoothed on the way
            // if asked for); the key-only score then takes the score array
            DevParams pt = p;
            pt.W = window;
            pt.rows = pt.G * window;
            pt.rows_pad = rows_padded(pt.rows);
            pt.tc_stages = pt.rows_pad <= 256 ? 4 : 2;
            rc = launch_score_tova(pt, ctx);
            if (rc == AMS_OK) rc = launch_smooth_usage(p, p.scores, usage_buf, c.pool_kernel, ctx);
            p.usage = usage_buf;
        }
        if (rc == AMS_OK) rc = scorer_id == AMS_SCORER_KEYDIFF ? launch_score_keydiff(p, ctx) : launch_score_expected(p, ctx);
    }
    if (rc == AMS_OK && c.pool_kernel > 1 && !split) {
        rc = launch_smooth_usage(p, p.usage, usage_buf, c.pool_kernel, ctx);
        p.usage = usage_buf;
    }
    if (rc == AMS_OK) rc = segsel_supported(p) ? launch_segsel(p, ctx) : AMS_ERR_UNSUPPORTED;
    if (rc == AMS_OK && dbg) {
        // inspection copies are taken before the table is rewritten
        const size_t U = (size_t)p.L * p.B * p.H;
        cudaError_t e = cudaSuccess;
        if (dbg->scores && e == cudaSuccess) e = cudaMemcpyAsync(dbg->scores, p.scores, U * p.T_cap * 4, cudaMemcpyDeviceToDevice, s);
        if (dbg->usage && e == cudaSuccess) e = cudaMemcpyAsync(dbg->usage, p.usage, U * p.T_cap * 4, cudaMemcpyDeviceToDevice, s);
        if (dbg->n_segments && e == cudaSuccess) e = cudaMemcpyAsync(dbg->n_segments, p.n_seg, U * 4, cudaMemcpyDeviceToDevice, s);
        if (dbg->seg_bounds && e == cudaSuccess) e = cudaMemcpyAsync(dbg->seg_bounds, p.seg_bounds, U * (size_t)(p.seg_cap + 1) * 4, cudaMemcpyDeviceToDevice, s);
        if (dbg->quotas && e == cudaSuccess) e = cudaMemcpyAsync(dbg->quotas, p.quotas, U * (size_t)p.seg_cap * 4, cudaMemcpyDeviceToDevice, s);
        if (dbg->keep_idx && e == cudaSuccess) e = cudaMemcpyAsync(dbg->keep_idx, p.keep_idx, U * (size_t)p.Tk * 4, cudaMemcpyDeviceToDevice, s);
        if (e != cudaSuccess) rc = AMS_ERR_CUDA;
        if (rc == AMS_OK && dbg->prev_kept && dbg->retained_iou) rc = launch_retained_iou(p, dbg->prev_kept, dbg->retained_iou, ctx);
    }
    if (rc == AMS_OK) rc = launch_gather(p, ctx);
    st->last_launches = ctx.launches;
    st->n_ev = ctx.n_ev;
    memcpy(st->ev_ids, ctx.ids, sizeof ctx.ids);
    return rc;
}

int ams_set_query_stats(ams_state *st, const float *q_mean, const void *q_cov, float score_eps)
{
    if (!st || !q_mean || !q_cov || !(score_eps >= 0.0f) || !(score_eps < 1e30f)) return AMS_ERR_INVALID_ARG;
    if (((uintptr_t)q_mean | (uintptr_t)q_cov) & 15) return AMS_ERR_INVALID_ARG;
    st->q_mean = q_mean;
    st->q_cov = q_cov;
    st->score_eps = score_eps;
    return AMS_OK;
}

int ams_get_status(ams_state *st, void *stream, int32_t *detail)
{
    if (!st) return AMS_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    int32_t host[4] = {0, 0, 0, 0};
    if (cudaMemcpyAsync(host, st->ws + st->lay.status, sizeof host, cudaMemcpyDeviceToHost, s) != cudaSuccess) return AMS_ERR_CUDA;
    if (cudaMemsetAsync(st->ws + st->lay.status, 0, sizeof host, s) != cudaSuccess) return AMS_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return AMS_ERR_CUDA;
    if (detail) memcpy(detail, host, sizeof host);
    return host[0];
}

int ams_debug_expire_wait(ams_state *st, uint32_t polls, void *stream)
{
    if (!st || polls < 1 || polls > (1u << 20)) return AMS_ERR_INVALID_ARG;
    return launch_expire_wait((int *)(st->ws + st->lay.status), polls, (cudaStream_t)stream);
}

int32_t ams_last_launch_count(const ams_state *st) { return st ? st->last_launches : 0; }

int ams_set_profiling(ams_state *st, int enable)
{
    if (!st) return AMS_ERR_INVALID_ARG;
    if (enable && !st->profiling) {
        for (int i = 0; i < 32; ++i)
            if (cudaEventCreate(&st->ev[i]) != cudaSuccess) return AMS_ERR_CUDA;
        st->profiling = true;
    } else if (!enable && st->profiling) {
        for (int i = 0; i < 32; ++i) cudaEventDestroy(st->ev[i]);
        st->profiling = false;
    }
    st->n_ev = 0;
    return AMS_OK;
}

int ams_get_kernel_times(ams_state *st, float *ms)
{
    if (!st || !ms) return AMS_ERR_INVALID_ARG;
    for (int i = 0; i < kKernCount; ++i) ms[i] = 0.0f;
    if (!st->profiling || st->n_ev < 2) return AMS_ERR_INVALID_ARG;
    if (cudaEventSynchronize(st->ev[st->n_ev - 1]) != cudaSuccess) return AMS_ERR_CUDA;
    for (int i = 1; i < st->n_ev; ++i) {
        float t = 0.0f;
        if (cudaEventElapsedTime(&t, st->ev[i - 1], st->ev[i]) != cudaSuccess) return AMS_ERR_CUDA;
        const int id = st->ev_ids[i];
        if (id >= 0 && id < kKernCount) ms[id] += t;
    }
    return AMS_OK;
}

const char *ams_kernel_name(int32_t idx)
{
    static const char *names[kKernCount] = {"score_phase1", "score_combine", "score_phase2", "segment_select",
                                            "gather", "table_update", "usage_signal", "prepare", "segments_quotas", "select_compact"};
    return idx >= 0 && idx < kKernCount ? names[idx] : nullptr;
}

int ams_free(ams_state *st)
{
    if (!st) return AMS_ERR_INVALID_ARG;
    if (st->profiling) ams_set_profiling(st, 0);
    delete st;
    return AMS_OK;
}

const char *ams_strerror(int code)
{
    switch (code) {
    case AMS_OK: return "ok";
    case AMS_ERR_INVALID_ARG: return "invalid argument";
    case AMS_ERR_UNSUPPORTED: return "unsupported configuration";
    case AMS_ERR_CAPACITY: return "capacity exceeded";
    case AMS_ERR_CUDA: return "CUDA runtime error";
    case AMS_ERR_TIMEOUT: return "bounded device wait expired";
    case AMS_ERR_INTERNAL: return "internal consistency check failed";
    default: return "unknown error";
    }
}

} // extern "C"
