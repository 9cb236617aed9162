// C-ABI entry points (see include/acache.h): argument validation, workspace layout and the
// kernel sequences of the affix-cache refresh path.  Everything is enqueued on the caller's
// stream; nothing here allocates device memory or synchronises (except acache_poll_status).
#include <array>
#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <functional>
#include <new>
#include <string>

#include "../../include/acache.h"
#include "kernels.h"

using namespace acache;

struct acache_ctx {
    acache_model_desc d;
    size_t ws_need = 0;
    unsigned char* ws = nullptr;
    size_t ws_have = 0;
    // workspace offsets (bytes)
    size_t o_status, o_row_pos, o_row_pos2, o_row_src, o_xn, o_q, o_o, o_h1, o_xn2, o_act, o_knew, o_vnew;
    size_t o_mrow_pos, o_mrow_src, o_xn_mask, o_qmask, o_stats, o_partial, o_slot;
    size_t o_rowmask, partial_bytes;
    size_t o_xstage, o_ystage, o_sstage, o_astage, o_gemm, o_attn, o_gridbar, o_mcidx, o_lstats, o_lxn, o_keymask;
    std::string err;
    uint64_t launches = 0;
    void* stash_rows = nullptr;   // set for the duration of a host-buffer call: device copy of the gathered rows of x
    int debug_expire_once = 0;      // acache_debug_expire_next_wait: consumed by the next Q/K/V projection
    // optional per-stage timing (acache_stage_timing)
    bool timing = false;
    cudaEvent_t ev[ACACHE_N_STAGES + 1] = {};
    bool ev_hit[ACACHE_N_STAGES + 1] = {};
};

namespace {

acache_status fail(acache_ctx* c, acache_status s, const char* fmt, ...) {
    if (c) {
        char buf[512];
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(buf, sizeof buf, fmt, ap);
        va_end(ap);
        c->err = buf;
    }
    return s;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

size_t take(size_t& cur, size_t bytes) {
    size_t at = cur;
    cur += (bytes + 255) & ~size_t(255);
    return at;
}

template <class T>
T* wsp(acache_ctx* c, size_t off) { return reinterpret_cast<T*>(c->ws + off); }

// Marks the start of stage `i` (and the end of the stages before it) on the stream.
void mark(acache_ctx* c, int i, cudaStream_t st) {
    if (!c->timing) return;
    cudaEventRecord(c->ev[i], st);
    c->ev_hit[i] = true;
}

acache_status check_cuda(acache_ctx* c, const char* what) {
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(c, ACACHE_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
    return ACACHE_OK;
}

// shared_ok: the call only reads the cache, so one copy may serve the whole batch (batch_stride 0)
acache_status check_request(acache_ctx* c, const acache_request* r, const acache_kv* kv, int k, bool need_rope,
                            bool shared_ok = false) {
    const acache_model_desc& d = c->d;
    if (!c->ws) return fail(c, ACACHE_ERR_WORKSPACE, "workspace not set");
    if (!r) return fail(c, ACACHE_ERR_INVALID_ARG, "request is NULL");
    if (r->batch < 0 || r->batch > d.max_batch) return fail(c, ACACHE_ERR_INVALID_ARG, "batch %d outside [0, %d]", r->batch, d.max_batch);
    if (r->ctx_len <= 0 || r->ctx_len > d.max_ctx) return fail(c, ACACHE_ERR_INVALID_ARG, "ctx_len %d outside (0, %d]", r->ctx_len, d.max_ctx);
    if (r->affix_len < 0 || r->affix_len > d.max_affix || r->affix_start < 0 ||
        (int64_t)r->affix_start + r->affix_len > r->ctx_len)
        return fail(c, ACACHE_ERR_INVALID_ARG, "affix span [%d, +%d) outside the context / max_affix", r->affix_start, r->affix_len);
    if (r->n_masked < 0 || r->n_masked > d.max_masked) return fail(c, ACACHE_ERR_INVALID_ARG, "n_masked %d outside [0, %d]", r->n_masked, d.max_masked);
    if (r->n_extra < 0 || k < 0 || k > r->affix_len) return fail(c, ACACHE_ERR_INVALID_ARG, "k %d / n_extra %d out of range", k, r->n_extra);
    if ((int64_t)k + r->n_extra > d.max_rows) return fail(c, ACACHE_ERR_INVALID_ARG, "k + n_extra = %d exceeds max_rows %d", k + r->n_extra, d.max_rows);
    if (r->n_masked > 0 && !r->masked_pos) return fail(c, ACACHE_ERR_INVALID_ARG, "masked_pos is NULL");
    if (r->n_extra > 0 && !r->extra_rows) return fail(c, ACACHE_ERR_INVALID_ARG, "extra_rows is NULL");
    if (need_rope && (!r->rope_cos || !r->rope_sin || !aligned16(r->rope_cos) || !aligned16(r->rope_sin)))
        return fail(c, ACACHE_ERR_INVALID_ARG, "rope table NULL or misaligned");
    if (kv) {
        if (!kv->k || !kv->v || !aligned16(kv->k) || !aligned16(kv->v)) return fail(c, ACACHE_ERR_INVALID_ARG, "cache pointer NULL or misaligned");
        if (kv->ctx_capacity < r->ctx_len) return fail(c, ACACHE_ERR_INVALID_ARG, "ctx_capacity %d < ctx_len %d", kv->ctx_capacity, r->ctx_len);
        const bool shared = kv->batch_stride == 0;
        if (shared && !shared_ok)
            return fail(c, ACACHE_ERR_INVALID_ARG, "batch_stride 0 (one cache shared by the batch) is only valid for calls that do not write the cache");
        if (!shared && (kv->batch_stride < (int64_t)kv->ctx_capacity * d.n_kv_heads * d.head_dim || (kv->batch_stride & 7)))
            return fail(c, ACACHE_ERR_INVALID_ARG, "batch_stride smaller than one request's cache or not a multiple of 8");
    }
    return ACACHE_OK;
}

acache_status check_weights(acache_ctx* c, const acache_layer_weights* w, bool q_only) {
    if (!w) return fail(c, ACACHE_ERR_INVALID_ARG, "weights is NULL");
    const void* need[] = {w->attn_norm_g, w->wq, w->wk, w->wv, w->wo, w->mlp_norm_g, w->w_gate, w->w_up, w->w_down};
    const int n = q_only ? 2 : 9;
    for (int i = 0; i < n; ++i)
        if (!need[i] || !aligned16(need[i])) return fail(c, ACACHE_ERR_INVALID_ARG, "weight pointer %d NULL or misaligned", i);
    if (c->d.qkv_bias && (!w->bq || (!q_only && (!w->bk || !w->bv))))
        return fail(c, ACACHE_ERR_INVALID_ARG, "qkv_bias set but a bias pointer is NULL");
    return ACACHE_OK;
}

// Q for the masked rows, then Eq. 4-5.
acache_status run_score(acache_ctx* c, const acache_request* r, const void* q_mask, const acache_kv* kv,
                        float* scores, int accumulate, int norm_full, int defer_head_sum, cudaStream_t st, int early_k = 0) {
    ScoreArgs a{};
    a.early_k = early_k;
    a.q_mask = q_mask;
    a.cache_k = kv->k;
    a.kv_batch_stride = kv->batch_stride;
    a.batch = r->batch; a.m = r->n_masked;
    a.n_heads = c->d.n_heads; a.n_kv_heads = c->d.n_kv_heads; a.head_dim = c->d.head_dim;
    a.affix_start = r->affix_start; a.affix_len = r->affix_len;
    a.norm_lo = norm_full ? 0 : r->affix_start;
    a.norm_len = norm_full ? r->ctx_len : r->affix_len;
    a.row_stats = wsp<float>(c, c->o_stats);
    a.head_partial = wsp<float>(c, c->o_partial);
    a.scores = scores;
    a.accumulate = accumulate;
    a.defer_head_sum = defer_head_sum;
    a.status = wsp<uint32_t>(c, c->o_status);
    int n = launch_score(a, st);
    if (n < 0) return fail(c, ACACHE_ERR_UNSUPPORTED_SHAPE, "n_masked %d too large for the scoring kernel", r->n_masked);
    c->launches += n;
    return check_cuda(c, "score");
}

// The recompute of rows R.  fused_cache != null: K/V go straight into the cache and
// attention reads it; otherwise K/V go to k_new/v_new and attention reads through a slot map.
// The private slot array a decode pass over shared storage works against: k anchors and e extra rows per
// request as an earlier refresh pass over the same storage wrote them; out_rows[b, i] = the slot row that
// holds row i of the rows recomputed now.
// K blocks past the shared-memory ring that each projection asks into L2 before its dependency wait (masked-row
// queries, q/k/v, output, gate/up, down).  Worth it only behind kernels that leave memory idle for a while: the
// previous step's last finish, and scoring + selection (measured at 103 rows: 168.8 us per layer-step with none,
// 167.9 with 8 blocks for the first two, 170.7 with 8 for the down projection).  ACACHE_GEMM_PREFETCH_BY="a,b,c,d,e"
// overrides.
static int prefetch_by(int which) {
    static const std::array<int, 5> v = [] {
        std::array<int, 5> r{8, 8, 0, 0, 0};
        if (const char* e = getenv("ACACHE_GEMM_PREFETCH_BY")) sscanf(e, "%d,%d,%d,%d,%d", &r[0], &r[1], &r[2], &r[3], &r[4]);
        return r;
    }();
    return v[which];
}
// Eq. 4-5 taken from the attention of the rows being recomputed (the probe of Section 3.2: the masked rows are among them)
struct FusedScore {
    const uint32_t* rowmask;
    int rm_words;
    float* scores;
    int accumulate;
    int norm_full;          // Eq. 4's softmax over every key (the attention's own denominator) instead of the affix keys
};
struct PrivateRows {
    const int32_t* anchor_idx;
    int k;
    const int32_t* extra_rows;
    int e;
    const int32_t* out_rows;
};
// Slot map and key masks of the fresh rows are the same for every layer of a pass: the first layer of a
// multi-layer call builds them in the workspace, the later ones reuse them.
struct MapReuse { bool reuse; };

acache_status run_recompute(acache_ctx* c, const acache_layer_weights* w, const acache_request* r,
                            const acache_kv* kv, bool fuse_scatter, const void* x, int x_is_compact,
                            const int32_t* anchor_idx, int k, void* k_new, void* v_new, void* y, cudaStream_t st,
                            const PrivateRows* priv = nullptr, MapReuse maps = MapReuse{false}, bool drop_non_anchor = false,
                            const FusedScore* fs = nullptr,
                            const std::function<acache_status()>& after_qkv = std::function<acache_status()>()) {
    const acache_model_desc& d = c->d;
    const int rows = k + r->n_extra, n = r->batch * rows;
    if (n == 0) {
        mark(c, ACACHE_N_STAGES, st);
        return ACACHE_OK;
    }
    const int qd = d.n_heads * d.head_dim, kvd = d.n_kv_heads * d.head_dim;
    int32_t* row_pos = wsp<int32_t>(c, c->o_row_pos);
    int64_t* row_src = wsp<int64_t>(c, c->o_row_src);
    void* xn = wsp<void>(c, c->o_xn);
    void* q = wsp<void>(c, c->o_q);
    void* o = wsp<void>(c, c->o_o);
    void* h1 = wsp<void>(c, c->o_h1);
    void* xn2 = wsp<void>(c, c->o_xn2);
    void* act = wsp<void>(c, c->o_act);
    uint32_t* status = wsp<uint32_t>(c, c->o_status);

    mark(c, ACACHE_STAGE_QKV, st);
    unsigned int* grid_bar = wsp<unsigned int>(c, c->o_gridbar);
    float* partial = wsp<float>(c, c->o_gemm);

    GemmArgs g{};
    g.a = xn; g.M = n; g.K = d.hidden;
    g.prep.enabled = 1; g.prep.x = x; g.prep.x_is_compact = x_is_compact;
    g.prep.x_batch_stride = (int64_t)r->ctx_len * d.hidden;
    g.prep.anchor_idx = anchor_idx; g.prep.k = k; g.prep.extra_rows = r->extra_rows; g.prep.e = r->n_extra;
    g.prep.affix_start = r->affix_start; g.prep.affix_len = r->affix_len; g.prep.ctx_len = r->ctx_len;
    g.prep.gain = w->attn_norm_g; g.prep.eps = d.rms_eps; g.prep.row_pos = row_pos; g.prep.row_src = row_src;
    if (!x_is_compact && r->token_ids) { g.prep.token_ids = r->token_ids; g.prep.table_rows = r->n_embed; }
    // x in page-locked host memory: the gathered rows are kept on the device for the residual of the output projection
    void* x_rows = (c->stash_rows && !r->token_ids) ? c->stash_rows : nullptr;
    g.prep.raw_out = x_rows;
    g.b[0] = w->wq; g.b[1] = w->wk; g.b[2] = w->wv;
    g.n[0] = qd; g.n[1] = kvd; g.n[2] = kvd;
    g.epilogue = kEpiQKV;
    g.bias[0] = d.qkv_bias ? w->bq : nullptr;
    g.bias[1] = d.qkv_bias ? w->bk : nullptr;
    g.bias[2] = d.qkv_bias ? w->bv : nullptr;
    g.row_pos = row_pos; g.rope_cos = r->rope_cos; g.rope_sin = r->rope_sin;
    g.head_dim = d.head_dim; g.rope_segments = 2;
    g.out[0] = q; g.out[1] = k_new; g.out[2] = v_new;
    if (fuse_scatter) { g.cache_k = kv->k; g.cache_v = kv->v; }
    g.kv_batch_stride = kv->batch_stride; g.rows_per_req = rows;
    if (priv) { g.kv_out_rows = priv->out_rows; g.kv_out_stride = priv->k + priv->e; }
    g.partial = partial; g.status = status; g.grid_bar = grid_bar;
    g.prefetch_blocks = prefetch_by(1);
    g.debug_expire = c->debug_expire_once;
    c->debug_expire_once = 0;
    { int nl = launch_gemm(g, st); if (nl < 0) return check_cuda(c, "qkv projection") == ACACHE_OK ? fail(c, ACACHE_ERR_CUDA, "qkv projection launch failed") : ACACHE_ERR_CUDA;
    c->launches += nl; }

    if (after_qkv) {            // work of the caller that wants the fresh K/V in place but precedes the attention
        const acache_status sq = after_qkv();
        if (sq != ACACHE_OK) return sq;
    }
    mark(c, ACACHE_STAGE_ATTENTION, st);
    AttnArgs at{};
    at.q = q; at.cache_k = kv->k; at.cache_v = kv->v; at.kv_batch_stride = kv->batch_stride;
    if (!fuse_scatter) {
        // the rows that serve their positions from k_new / v_new: the rows recomputed now, or the whole private
        // slot array of which they refreshed a part
        const int fresh = priv ? priv->k + priv->e : rows;
        const int32_t* fresh_pos = row_pos;
        if (priv) {
            int32_t* rp2 = wsp<int32_t>(c, c->o_row_pos2);
            if (!maps.reuse) {
                launch_row_positions(priv->anchor_idx, priv->k, priv->extra_rows, priv->e, r->affix_start, r->affix_len,
                                     r->ctx_len, r->batch, rp2, status, st);
                c->launches += 1;
            }
            fresh_pos = rp2;
            at.n_fresh = fresh;
        }
        int32_t* slot = wsp<int32_t>(c, c->o_slot);
        at.k_new = k_new; at.v_new = v_new; at.slot = slot;
        // key masks of the same map, for the kernel that reads cache and fresh rows as two sources
        at.excl_words = (r->ctx_len + 31) / 32; at.keep_words = (fresh + 31) / 32;
        uint32_t* km = wsp<uint32_t>(c, c->o_keymask);
        at.pos_excl = km; at.row_keep = km + (size_t)r->batch * at.excl_words;
        if (!maps.reuse) {
            launch_build_slot_map(slot, r->ctx_len, fresh_pos, fresh, r->batch, st);
            launch_key_masks(slot, r->ctx_len, fresh_pos, fresh, r->batch, km, at.excl_words,
                             km + (size_t)r->batch * at.excl_words, at.keep_words, st);
            c->launches += 2;
        }
    }
    if (drop_non_anchor) {
        // DropNA layout (Section 5.3): the affix positions that are not anchors do not exist as keys.  The bits
        // live behind the two masks of the two-source attention; with fresh rows as a second source they are also
        // OR-ed into the cache-exclusion mask (the anchors then come from the fresh rows).
        const int words = (r->ctx_len + 31) / 32;
        uint32_t* km = wsp<uint32_t>(c, c->o_keymask);
        uint32_t* kd = km + (size_t)r->batch * (words + (d.max_rows + 31) / 32 + 2);
        launch_drop_mask(anchor_idx, k, r->affix_start, r->affix_len, r->ctx_len, r->batch, kd, fuse_scatter ? nullptr : km, words, st);
        c->launches += 1;
        at.key_drop = kd; at.excl_words = words;
    }
    at.batch = r->batch; at.n = rows; at.ctx_len = r->ctx_len;
    at.n_heads = d.n_heads; at.n_kv_heads = d.n_kv_heads; at.head_dim = d.head_dim;
    at.o = o;
    at.status = status;
    at.part_o = wsp<float>(c, c->o_attn);
    at.part_ml = at.part_o + (size_t)2 * 296 * 64 * d.head_dim;
    if (fs) {
        at.score_rowmask = fs->rowmask; at.rm_words = fs->rm_words; at.score_partial = wsp<float>(c, c->o_partial);
        at.affix_start = r->affix_start; at.affix_len = r->affix_len; at.score_norm_full = fs->norm_full;
    }
    c->launches += launch_attention(at, st);
    if (fs) {
        launch_score_reduce_tiles(wsp<float>(c, c->o_partial), fs->rowmask, fs->rm_words, fs->scores, r->batch, d.n_heads,
                                  (rows + 127) / 128, r->affix_len, fs->accumulate, st);
        c->launches += 1;
    }

    mark(c, ACACHE_STAGE_OPROJ, st);
    GemmArgs go{};
    go.a = o; go.M = n; go.K = qd; go.b[0] = w->wo; go.n[0] = d.hidden;
    go.epilogue = kEpiResidual; go.resid = x_rows ? x_rows : x; go.resid_off = x_rows ? nullptr : row_src; go.c = h1;
    go.partial = partial; go.status = status; go.grid_bar = grid_bar;
    go.prefetch_blocks = prefetch_by(2);
    { int nl = launch_gemm(go, st); if (nl < 0) return check_cuda(c, "output projection") == ACACHE_OK ? fail(c, ACACHE_ERR_CUDA, "output projection launch failed") : ACACHE_ERR_CUDA;
    c->launches += nl; }
    mark(c, ACACHE_STAGE_GATE_UP, st);

    GemmArgs gu{};
    gu.prep.enabled = 2; gu.prep.x = h1; gu.prep.gain = w->mlp_norm_g; gu.prep.eps = d.rms_eps;   // xn2 = RMSNorm(h1)
    gu.a = xn2; gu.M = n; gu.K = d.hidden; gu.b[0] = w->w_gate; gu.b[1] = w->w_up; gu.n[0] = d.ffn; gu.n[1] = d.ffn;
    gu.epilogue = kEpiSwiGLU; gu.c = act;
    gu.partial = partial; gu.status = status; gu.grid_bar = grid_bar;
    gu.prefetch_blocks = prefetch_by(3);
    { int nl = launch_gemm(gu, st); if (nl < 0) return check_cuda(c, "gate/up projection") == ACACHE_OK ? fail(c, ACACHE_ERR_CUDA, "gate/up projection launch failed") : ACACHE_ERR_CUDA;
    c->launches += nl; }

    mark(c, ACACHE_STAGE_DOWN, st);
    GemmArgs gd{};
    gd.a = act; gd.M = n; gd.K = d.ffn; gd.b[0] = w->w_down; gd.n[0] = d.hidden;
    gd.epilogue = kEpiResidual; gd.resid = h1; gd.resid_off = nullptr; gd.c = y;
    gd.partial = partial; gd.status = status; gd.grid_bar = grid_bar;
    gd.prefetch_blocks = prefetch_by(4);
    { int nl = launch_gemm(gd, st); if (nl < 0) return check_cuda(c, "down projection") == ACACHE_OK ? fail(c, ACACHE_ERR_CUDA, "down projection launch failed") : ACACHE_ERR_CUDA;
    c->launches += nl; }
    mark(c, ACACHE_N_STAGES, st);
    return check_cuda(c, "recompute");
}

}  // namespace

// Set by the multi-layer entry points around their layers after the first (same rows, same maps); the
// single-layer entry points read it.  Thread-local: a context is used from one thread at a time.
static thread_local bool g_reuse_maps = false;

namespace {
// Device-side address of page-locked host memory (nullptr for pageable or unknown memory).
const void* mapped_device_pointer(const void* host) {
    cudaPointerAttributes at{};
    if (!host || cudaPointerGetAttributes(&at, host) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    return at.type == cudaMemoryTypeHost ? at.devicePointer : nullptr;
}
}  // namespace

extern "C" {

acache_status acache_create(const acache_model_desc* desc, acache_ctx** out) {
    if (!desc || !out) return ACACHE_ERR_INVALID_ARG;
    *out = nullptr;
    const acache_model_desc& d = *desc;
    if (d.hidden <= 0 || d.n_heads <= 0 || d.n_kv_heads <= 0 || d.ffn <= 0 || d.max_batch <= 0 || d.max_ctx <= 0 ||
        d.max_affix < 0 || d.max_rows < 0 || d.max_masked < 0 || d.max_vocab < 0 || d.max_block < 0 ||
        !(d.rms_eps >= 0.f))
        return ACACHE_ERR_INVALID_ARG;
    if (d.head_dim != 64 && d.head_dim != 128) return ACACHE_ERR_UNSUPPORTED_SHAPE;
    if (d.n_heads % d.n_kv_heads) return ACACHE_ERR_UNSUPPORTED_SHAPE;
    const int qd = d.n_heads * d.head_dim, kvd = d.n_kv_heads * d.head_dim;
    if (qd % 128 || kvd % 128 || d.ffn % 128 || d.hidden % 128) return ACACHE_ERR_UNSUPPORTED_SHAPE;
    acache_ctx* c = new (std::nothrow) acache_ctx();
    if (!c) return ACACHE_ERR_INVALID_ARG;
    c->d = d;
    const size_t nr = (size_t)d.max_batch * d.max_rows, nm = (size_t)d.max_batch * d.max_masked;
    size_t cur = 0;
    c->o_status = take(cur, 256);
    c->o_gridbar = take(cur, 256);
    c->o_row_pos = take(cur, nr * 4);
    c->o_row_pos2 = take(cur, nr * 4);
    c->o_row_src = take(cur, nr * 8);
    c->o_xn = take(cur, nr * d.hidden * 2);
    c->o_q = take(cur, nr * qd * 2);
    c->o_o = take(cur, nr * qd * 2);
    c->o_h1 = take(cur, nr * d.hidden * 2);
    c->o_xn2 = take(cur, nr * d.hidden * 2);
    c->o_act = take(cur, nr * d.ffn * 2);
    c->o_knew = take(cur, nr * kvd * 2);
    c->o_vnew = take(cur, nr * kvd * 2);
    c->o_mrow_pos = take(cur, nm * 4);
    c->o_mrow_src = take(cur, nm * 8);
    c->o_mcidx = take(cur, nm * 4);
    c->o_xn_mask = take(cur, nm * d.hidden * 2);
    c->o_qmask = take(cur, nm * qd * 2);
    c->o_stats = take(cur, (size_t)d.max_batch * d.n_heads * score_num_splits(d.max_ctx) * d.max_masked * 8);
    {
        // per-head column sums [B, H, L]; when the scores come out of the probe's attention, per (head, query tile):
        // [B, H, ceil(rows / 128), L], as far as that stays within 256 MB (else the separate scoring kernels run)
        const size_t per_head = (size_t)d.max_batch * d.n_heads * d.max_affix * 4;
        const size_t tiles = (size_t)(d.max_rows + 127) / 128;
        c->partial_bytes = d.head_dim == 128 && per_head * tiles <= ((size_t)256 << 20) ? per_head * std::max<size_t>(tiles, 1) : per_head;
        c->o_partial = take(cur, c->partial_bytes);
    }
    c->o_rowmask = take(cur, (size_t)d.max_batch * ((d.max_rows + 31) / 32 + 8) * 4);
    c->o_slot = take(cur, (size_t)d.max_batch * d.max_ctx * 4);
    c->o_keymask = take(cur, (size_t)d.max_batch * (2 * ((d.max_ctx + 31) / 32) + (d.max_rows + 31) / 32 + 4) * 4);
    c->o_xstage = take(cur, (size_t)d.max_batch * d.max_ctx * d.hidden * 2);
    c->o_ystage = take(cur, nr * d.hidden * 2);
    c->o_sstage = take(cur, (size_t)d.max_batch * d.max_affix * 4);
    c->o_astage = take(cur, (size_t)d.max_batch * d.max_affix * 4);
    {
        const int nri = (int)nr, nmi = (int)nm;
        size_t pb = gemm_partial_bytes(nri, d.hidden, qd + 2 * kvd, false);
        pb = std::max(pb, gemm_partial_bytes(nri, qd, d.hidden, false));
        pb = std::max(pb, gemm_partial_bytes(nri, d.hidden, d.ffn, true));
        pb = std::max(pb, gemm_partial_bytes(nri, d.ffn, d.hidden, false));
        pb = std::max(pb, gemm_partial_bytes(nmi, d.hidden, qd, false));
        c->o_gemm = take(cur, pb);
    }
    c->o_attn = take(cur, attention_scratch_bytes(d.head_dim));
    {
        const size_t lrows = (size_t)d.max_batch * (d.max_block > 0 ? d.max_block : 0);
        const size_t ltiles = d.max_vocab > 0 ? (size_t)(d.max_vocab + 255) / 256 : 0;
        c->o_lstats = take(cur, lrows * ltiles * 16 * 16);
        c->o_lxn = take(cur, lrows * d.hidden * 2);
    }
    c->ws_need = cur;
    *out = c;
    return ACACHE_OK;
}

size_t acache_workspace_bytes(const acache_ctx* ctx) { return ctx ? ctx->ws_need : 0; }

acache_status acache_set_workspace(acache_ctx* ctx, void* dev_ptr, size_t bytes, acache_stream_t stream) {
    if (!ctx) return ACACHE_ERR_INVALID_ARG;
    if (!dev_ptr || (reinterpret_cast<uintptr_t>(dev_ptr) & 255u)) return fail(ctx, ACACHE_ERR_INVALID_ARG, "workspace NULL or not 256-byte aligned");
    if (bytes < ctx->ws_need) return fail(ctx, ACACHE_ERR_WORKSPACE, "workspace %zu < %zu bytes", bytes, ctx->ws_need);
    ctx->ws = static_cast<unsigned char*>(dev_ptr);
    ctx->ws_have = bytes;
    // status word and grid-barrier words are adjacent: clear both
    if (cudaMemsetAsync(ctx->ws + ctx->o_status, 0, 512, stream) != cudaSuccess) return check_cuda(ctx, "memset");
    return ACACHE_OK;
}

void acache_destroy(acache_ctx* ctx) {
    if (!ctx) return;
    for (cudaEvent_t e : ctx->ev)
        if (e) cudaEventDestroy(e);
    delete ctx;
}

acache_status acache_stage_timing(acache_ctx* ctx, int enable) {
    if (!ctx) return ACACHE_ERR_INVALID_ARG;
    if (enable && !ctx->ev[0]) {
        for (cudaEvent_t& e : ctx->ev)
            if (cudaEventCreate(&e) != cudaSuccess) return check_cuda(ctx, "cudaEventCreate");
    }
    ctx->timing = enable != 0;
    for (bool& h : ctx->ev_hit) h = false;
    return ACACHE_OK;
}

acache_status acache_read_stage_times(acache_ctx* ctx, float* ms) {
    if (!ctx || !ms) return ACACHE_ERR_INVALID_ARG;
    if (!ctx->timing || !ctx->ev_hit[ACACHE_N_STAGES]) return fail(ctx, ACACHE_ERR_INVALID_ARG, "no timed layer-step to read");
    if (cudaEventSynchronize(ctx->ev[ACACHE_N_STAGES]) != cudaSuccess) return check_cuda(ctx, "cudaEventSynchronize");
    for (int i = 0; i < ACACHE_N_STAGES; ++i) {
        ms[i] = 0.f;
        if (!ctx->ev_hit[i]) continue;
        int j = i + 1;
        while (!ctx->ev_hit[j]) ++j;          // the next stage that ran (the end mark always did)
        if (cudaEventElapsedTime(&ms[i], ctx->ev[i], ctx->ev[j]) != cudaSuccess) return check_cuda(ctx, "cudaEventElapsedTime");
    }
    return ACACHE_OK;
}

const char* acache_last_error(const acache_ctx* ctx) { return ctx ? ctx->err.c_str() : "context is NULL"; }

uint64_t acache_launch_count(const acache_ctx* ctx) { return ctx ? ctx->launches : 0; }

acache_status acache_poll_status(acache_ctx* ctx, acache_stream_t stream, uint32_t* host_flags) {
    if (!ctx || !host_flags) return ACACHE_ERR_INVALID_ARG;
    if (!ctx->ws) return fail(ctx, ACACHE_ERR_WORKSPACE, "workspace not set");
    uint32_t v = 0;
    if (cudaMemcpyAsync(&v, ctx->ws + ctx->o_status, 4, cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
        cudaMemsetAsync(ctx->ws + ctx->o_status, 0, 4, stream) != cudaSuccess ||
        cudaStreamSynchronize(stream) != cudaSuccess)
        return check_cuda(ctx, "poll_status") == ACACHE_OK ? fail(ctx, ACACHE_ERR_CUDA, "poll_status failed") : ACACHE_ERR_CUDA;
    *host_flags = v;
    if (v & ACACHE_FLAG_WAIT_EXPIRED) {
        // a kernel gave up half way: its grid-barrier words are stale, re-arm them
        cudaMemsetAsync(ctx->ws + ctx->o_gridbar, 0, 256, stream);
        cudaStreamSynchronize(stream);
        return fail(ctx, ACACHE_ERR_TIMEOUT, "a bounded device-side wait expired");
    }
    return ACACHE_OK;
}

acache_status acache_debug_expire_next_wait(acache_ctx* ctx) {
    if (!ctx) return ACACHE_ERR_INVALID_ARG;
    ctx->debug_expire_once = 1;
    return ACACHE_OK;
}

int32_t acache_k_from_ratio(int32_t affix_len, double ratio) {
    if (affix_len <= 0 || !(ratio > 0.0)) return 0;
    double k = std::ceil(ratio * (double)affix_len - 1e-9);
    if (k < 0) k = 0;
    if (k > affix_len) k = affix_len;
    return (int32_t)k;
}

acache_status acache_score_anchors(acache_ctx* ctx, const acache_request* req, const void* q_mask,
                                   const acache_kv* kv, float* scores, int accumulate, int norm_full,
                                   acache_stream_t stream) {
    if (!ctx) return ACACHE_ERR_INVALID_ARG;
    if (!kv) return fail(ctx, ACACHE_ERR_INVALID_ARG, "kv is NULL");
    acache_status s = check_request(ctx, req, kv, 0, false, true);
    if (s != ACACHE_OK) return s;
    if (!scores || (req->n_masked > 0 && (!q_mask || !aligned16(q_mask)))) return fail(ctx, ACACHE_ERR_INVALID_ARG, "q_mask / scores NULL or misaligned");
    return run_score(ctx, req, q_mask, kv, scores, accumulate, norm_full, 0, stream);
}

acache_status acache_select_topk(acache_ctx* ctx, const float* scores, int32_t batch, int32_t affix_len, int32_t k,
                                 int32_t* anchor_idx, acache_stream_t stream) {
    if (!ctx) return ACACHE_ERR_INVALID_ARG;
    if (batch < 0 || affix_len < 0 || k < 0 || k > affix_len) return fail(ctx, ACACHE_ERR_INVALID_ARG, "batch %d, affix_len %d, k %d out of range", batch, affix_len, k);
    if (batch == 0 || k == 0) return ACACHE_OK;
    if (!scores || !anchor_idx) return fail(ctx, ACACHE_ERR_INVALID_ARG, "scores / anchor_idx is NULL");
    launch_topk(const_cast<float*>(scores), batch, affix_len, k, anchor_idx, nullptr, 0, 0, stream);
    ctx->launches += 1;
    return check_cuda(ctx, "topk");
}

acache_status acache_score_kv_deviation(acache_ctx* ctx, const acache_request* req, const acache_kv* kv_ref,
                                        const acache_kv* kv_full, float* scores, int accumulate, acache_stream_t stream) {
    if (!ctx) return ACACHE_ERR_INVALID_ARG;
    if (!kv_ref || !kv_full) return fail(ctx, ACACHE_ERR_INVALID_ARG, "kv_ref / kv_full is NULL");
    acache_status s = check_request(ctx, req, kv_ref, 0, false, true);
    if (s != ACACHE_OK) return s;
    if ((s = check_request(ctx, req, kv_full, 0, false, true)) != ACACHE_OK) return s;
    if (!scores) return fail(ctx, ACACHE_ERR_INVALID_ARG, "scores is NULL");
    if (req->batch == 0 || req->affix_len == 0) return ACACHE_OK;
    launch_kv_deviation(kv_ref->k, kv_ref->v, kv_ref->batch_stride, kv_full->k, kv_full->v, kv_full->batch_stride,
                        req->affix_start, req->affix_len, ctx->d.n_kv_heads * ctx->d.head_dim, req->batch, scores, accumulate,
                        stream);
    ctx->launches += 1;
    return check_cuda(ctx, "kv deviation");
}

acache_status acache_recompute_anchors(acache_ctx* ctx, const acache_layer_weights* w, const acache_request* req,
                                       const acache_kv* kv, const void* x, int x_is_compact,
                                       const int32_t* anchor_idx, int32_t k, void* k_new, void* v_new, void* y,
                                       acache_stream_t stream) {
    if (!ctx) return ACACHE_ERR_INVALID_ARG;
    if (!kv) return fail(ctx, ACACHE_ERR_INVALID_ARG, "kv is NULL");
    acache_status s = check_request(ctx, req, kv, k, true, true);
    if (s != ACACHE_OK) return s;
    if ((s = check_weights(ctx, w, false)) != ACACHE_OK) return s;
    if (req->batch * (k + req->n_extra) == 0) return ACACHE_OK;
    if (!x || !k_new || !v_new || !y || !aligned16(x) || !aligned16(k_new) || !aligned16(v_new) || !aligned16(y))
        return fail(ctx, ACACHE_ERR_INVALID_ARG, "x / k_new / v_new / y NULL or misaligned");
    if (k > 0 && !anchor_idx) return fail(ctx, ACACHE_ERR_INVALID_ARG, "anchor_idx is NULL");
    return run_recompute(ctx, w, req, kv, false, x, x_is_compact, anchor_idx, k, k_new, v_new, y, stream, nullptr,
                         MapReuse{g_reuse_maps});
}

acache_status acache_scatter_kv(acache_ctx* ctx, const acache_request* req, acache_kv* kv, const int32_t* anchor_idx,
                                int32_t k, const void* k_new, const void* v_new, acache_stream_t stream) {
    if (!ctx) return ACACHE_ERR_INVALID_ARG;
    if (!kv) return fail(ctx, ACACHE_ERR_INVALID_ARG, "kv is NULL");
    acache_status s = check_request(ctx, req, kv, k, false);
    if (s != ACACHE_OK) return s;
    if (req->batch * (k + req->n_extra) == 0) return ACACHE_OK;
    if (!k_new || !v_new || !aligned16(k_new) || !aligned16(v_new)) return fail(ctx, ACACHE_ERR_INVALID_ARG, "k_new / v_new NULL or misaligned");
    if (k > 0 && !anchor_idx) return fail(ctx, ACACHE_ERR_INVALID_ARG, "anchor_idx is NULL");
    launch_scatter_kv(kv->k, kv->v, kv->batch_stride, req->ctx_len, anchor_idx, k, req->extra_rows, req->n_extra,
                      req->batch, req->affix_start, req->affix_len, ctx->d.n_kv_heads * ctx->d.head_dim, k_new, v_new,
                      wsp<uint32_t>(ctx, ctx->o_status), stream);
    ctx->launches += 1;
    return check_cuda(ctx, "scatter");
}

}  // extern "C"

namespace {
// The layer-step on one working cache per request (k_new = v_new = NULL: fresh K/V go straight into the cache) or
// on storage that is not written (fresh K/V to k_new / v_new [B, K + e, Hkv, d]; the cache may be shared).
acache_status layer_step_impl(acache_ctx* ctx, const acache_layer_weights* w, const acache_request* req,
                              const acache_kv* kv, const void* x, int x_is_compact, double ratio, uint32_t flags,
                              float* scores, int32_t* anchor_idx, void* k_new, void* v_new, void* y,
                              acache_stream_t stream) {
    if (!ctx) return ACACHE_ERR_INVALID_ARG;
    if (!kv) return fail(ctx, ACACHE_ERR_INVALID_ARG, "kv is NULL");
    if (!req) return fail(ctx, ACACHE_ERR_INVALID_ARG, "request is NULL");
    const acache_model_desc& d = ctx->d;
    const int k = acache_k_from_ratio(req->affix_len, ratio);
    const bool to_slots = k_new != nullptr;
    acache_status s = check_request(ctx, req, kv, k, true, to_slots);
    if (s != ACACHE_OK) return s;
    const bool do_score = flags & ACACHE_F_SCORE, do_select = flags & ACACHE_F_SELECT;
    const bool do_recompute = !(flags & ACACHE_F_NO_RECOMPUTE);
    if ((s = check_weights(ctx, w, !do_recompute)) != ACACHE_OK) return s;
    if (!x || !aligned16(x)) return fail(ctx, ACACHE_ERR_INVALID_ARG, "x NULL or misaligned");
    if ((do_score || do_select) && !scores) return fail(ctx, ACACHE_ERR_INVALID_ARG, "scores is NULL");
    if (k > 0 && !anchor_idx) return fail(ctx, ACACHE_ERR_INVALID_ARG, "anchor_idx is NULL");
    if (do_recompute && req->batch * (k + req->n_extra) > 0 && (!y || !aligned16(y))) return fail(ctx, ACACHE_ERR_INVALID_ARG, "y NULL or misaligned");

    if (ctx->timing) for (bool& h : ctx->ev_hit) h = false;
    bool fused_head_sum = false;
    // The probe (Section 3.2): no anchors, no selection in this call, the masked rows among the rows being recomputed, the
    // softmax of Eq. 4 over the affix keys.  Its scores are the masked-to-affix part of its own attention: no query
    // projection of the masked rows and no pass over the affix keys of their own.
    static const bool fuse_on = [] { const char* e = getenv("ACACHE_SCORE_FUSED"); return !e || atoi(e) != 0; }();
    FusedScore fs{};
    bool score_in_attention = false;
    static const bool attn_tc_on = [] { const char* e = getenv("ACACHE_ATTN_TC"); return !(e && e[0] == '0'); }();
    if (fuse_on && attn_tc_on && !to_slots && do_score && !do_select && do_recompute && k == 0 && d.head_dim == 128 &&
        req->batch > 0 && req->affix_len > 0 && req->n_masked > 0 && req->n_extra > 0 && (kv->batch_stride & 7) == 0 &&
        (size_t)req->batch * d.n_heads * ((req->n_extra + 127) / 128) * req->affix_len * 4 <= ctx->partial_bytes) {
        fs.rm_words = (req->n_extra + 31) / 32;
        uint32_t* rm = wsp<uint32_t>(ctx, ctx->o_rowmask);
        launch_row_mask(req->masked_pos, req->n_masked, req->extra_rows, req->n_extra, 0, req->batch, rm, fs.rm_words,
                        wsp<uint32_t>(ctx, ctx->o_status), stream);
        ctx->launches += 1;
        fs.rowmask = rm; fs.scores = scores; fs.accumulate = (flags & ACACHE_F_ACCUMULATE) ? 1 : 0;
        fs.norm_full = (flags & ACACHE_F_SCORE_NORM_FULL) ? 1 : 0;
        score_in_attention = true;
    }
    // Scoring with the separate kernels (the masked rows' query projection, then Eq. 4-5 over the cached keys).  With the
    // softmax of Eq. 4 over every key of the context, a probe call (no anchors, no selection here, rows written into the
    // cache) scores after its rows' fresh K are in the cache, as the probe's own attention sees them (Section 3.2);
    // every other call scores the cache as given, before anything is recomputed.
    auto score_now = [&]() -> acache_status {
        if (do_score && !score_in_attention && req->batch > 0 && req->affix_len > 0) {
            void* qmask = wsp<void>(ctx, ctx->o_qmask);
            mark(ctx, ACACHE_STAGE_MASK_Q, stream);
            if (req->n_masked > 0) {
                int32_t* mpos = wsp<int32_t>(ctx, ctx->o_mrow_pos);
                void* xnm = wsp<void>(ctx, ctx->o_xn_mask);
                GemmArgs g{};
                g.a = xnm; g.M = req->batch * req->n_masked; g.K = d.hidden;
                g.prep.enabled = 1; g.prep.x = x; g.prep.x_is_compact = x_is_compact;
                if (x_is_compact) {
                    // the masked rows are among the extra rows of the compact input: find where
                    int32_t* cidx = wsp<int32_t>(ctx, ctx->o_mcidx);
                    launch_match_rows(req->masked_pos, req->n_masked, req->extra_rows, req->n_extra, k, req->batch, cidx,
                                      wsp<uint32_t>(ctx, ctx->o_status), stream);
                    ctx->launches += 1;
                    g.prep.compact_idx = cidx;
                    g.prep.compact_rows = k + req->n_extra;
                }
                g.prep.x_batch_stride = (int64_t)req->ctx_len * d.hidden;
                g.prep.anchor_idx = nullptr; g.prep.k = 0; g.prep.extra_rows = req->masked_pos; g.prep.e = req->n_masked;
                g.prep.affix_start = req->affix_start; g.prep.affix_len = req->affix_len; g.prep.ctx_len = req->ctx_len;
                g.prep.gain = w->attn_norm_g; g.prep.eps = d.rms_eps; g.prep.row_pos = mpos;
                g.prep.row_src = wsp<int64_t>(ctx, ctx->o_mrow_src);
                if (!x_is_compact && req->token_ids) { g.prep.token_ids = req->token_ids; g.prep.table_rows = req->n_embed; }
                g.b[0] = w->wq; g.n[0] = d.n_heads * d.head_dim;
                // W_q is read again by the Q/K/V projection a few kernels later: leave it in L2 (measured: that
                // projection 43.7 -> 40.8 us at 103 rows)
                static const int keep_wq = [] { const char* e = getenv("ACACHE_KEEP_WQ"); return e ? atoi(e) : 1; }();
                g.keep_weights = keep_wq && do_recompute;      // a scoring-only pass (the probe) never reads W_q again
                g.epilogue = kEpiQKV;
                g.bias[0] = d.qkv_bias ? w->bq : nullptr;
                g.row_pos = mpos; g.rope_cos = req->rope_cos; g.rope_sin = req->rope_sin;
                g.head_dim = d.head_dim; g.rope_segments = 1; g.out[0] = qmask; g.rows_per_req = req->n_masked;
                g.partial = wsp<float>(ctx, ctx->o_gemm); g.status = wsp<uint32_t>(ctx, ctx->o_status);
                g.grid_bar = wsp<unsigned int>(ctx, ctx->o_gridbar);
                g.prefetch_blocks = prefetch_by(0);
                { int nl = launch_gemm(g, stream); if (nl < 0) return check_cuda(ctx, "masked-row query projection") == ACACHE_OK ? fail(ctx, ACACHE_ERR_CUDA, "masked-row query projection launch failed") : ACACHE_ERR_CUDA;
                ctx->launches += nl; }
            }
            mark(ctx, ACACHE_STAGE_SCORE, stream);
            // with a selection to follow, the ordered sum over heads is folded into the selection kernel
            // (only while one CTA per request can read all heads' partial sums quickly: at L = 8192 the separate,
            // grid-wide head sum takes 4 us where the folded one took 28)
            fused_head_sum = do_select && k > 0 && req->n_masked > 0 && (int64_t)req->affix_len * d.n_heads <= 65536;
            // the masked rows' projection was launched just above: nothing that writes the cache is the scoring kernels'
            // direct predecessor, so they may request their first key tiles early
            s = run_score(ctx, req, qmask, kv, scores, (flags & ACACHE_F_ACCUMULATE) ? 1 : 0,
                          (flags & ACACHE_F_SCORE_NORM_FULL) ? 1 : 0, fused_head_sum ? 1 : 0, stream, req->n_masked > 0 ? 1 : 0);
            if (s != ACACHE_OK) return s;
        }
        return ACACHE_OK;
    };
    const bool score_late = do_score && !score_in_attention && !do_select && do_recompute && k == 0 && !to_slots &&
                            (flags & ACACHE_F_SCORE_NORM_FULL) && req->n_extra > 0;
    if (!score_late && (s = score_now()) != ACACHE_OK) return s;
    if (do_select && k > 0 && req->batch > 0) {
        mark(ctx, ACACHE_STAGE_TOPK, stream);
        launch_topk(scores, req->batch, req->affix_len, k, anchor_idx,
                    fused_head_sum ? wsp<float>(ctx, ctx->o_partial) : nullptr, d.n_heads,
                    (flags & ACACHE_F_ACCUMULATE) ? 1 : 0, stream);
        ctx->launches += 1;
    }
    if (do_recompute)
        return run_recompute(ctx, w, req, kv, !to_slots, x, x_is_compact, anchor_idx, k, k_new, v_new, y, stream, nullptr,
                             MapReuse{false}, (flags & ACACHE_F_DROP_NON_ANCHOR) != 0, score_in_attention ? &fs : nullptr,
                             score_late ? std::function<acache_status()>(score_now) : std::function<acache_status()>());
    mark(ctx, ACACHE_N_STAGES, stream);
    return check_cuda(ctx, "layer_step");
}
}  // namespace

extern "C" {

acache_status acache_layer_step(acache_ctx* ctx, const acache_layer_weights* w, const acache_request* req,
                                acache_kv* kv, const void* x, int x_is_compact, double ratio, uint32_t flags,
                                float* scores, int32_t* anchor_idx, void* y, acache_stream_t stream) {
    return layer_step_impl(ctx, w, req, kv, x, x_is_compact, ratio, flags, scores, anchor_idx, nullptr, nullptr, y, stream);
}

acache_status acache_layer_step_shared(acache_ctx* ctx, const acache_layer_weights* w, const acache_request* req,
                                       const acache_kv* kv, const void* x, int x_is_compact, double ratio,
                                       uint32_t flags, float* scores, int32_t* anchor_idx, void* k_new, void* v_new,
                                       void* y, acache_stream_t stream) {
    if (!ctx) return ACACHE_ERR_INVALID_ARG;
    if (!(flags & ACACHE_F_NO_RECOMPUTE) && (!k_new || !v_new || !aligned16(k_new) || !aligned16(v_new)))
        return fail(ctx, ACACHE_ERR_INVALID_ARG, "k_new / v_new NULL or misaligned");
    static char dummy;        // a scoring-only call stores no K/V: any non-NULL value selects the read-only path
    return layer_step_impl(ctx, w, req, kv, x, x_is_compact, ratio, flags, scores, anchor_idx, k_new ? k_new : &dummy,
                           v_new ? v_new : &dummy, y, stream);
}

acache_status acache_predict_commit(acache_ctx* ctx, const void* h, int32_t h_rows, const int32_t* block_rows,
                                    int32_t batch, int32_t n_blk, const void* final_norm_g, const void* w_lm,
                                    int32_t vocab, float threshold, int32_t* token, float* confidence,
                                    int32_t* commit, acache_stream_t stream) {
    if (!ctx) return ACACHE_ERR_INVALID_ARG;
    if (!ctx->ws) return fail(ctx, ACACHE_ERR_WORKSPACE, "workspace not set");
    const acache_model_desc& d = ctx->d;
    if (batch < 0 || n_blk < 0 || h_rows <= 0 || vocab <= 0) return fail(ctx, ACACHE_ERR_INVALID_ARG, "negative size");
    if ((int64_t)batch * n_blk > (int64_t)d.max_batch * d.max_block || vocab > d.max_vocab)
        return fail(ctx, ACACHE_ERR_INVALID_ARG, "batch * n_blk = %lld / vocab = %d exceed the context's limits (%lld, %d)",
                    (long long)batch * n_blk, vocab, (long long)d.max_batch * d.max_block, d.max_vocab);
    if (vocab % 128) return fail(ctx, ACACHE_ERR_UNSUPPORTED_SHAPE, "vocab %d is not a multiple of 128", vocab);
    if (batch * n_blk == 0) return ACACHE_OK;
    if (!h || !block_rows || !final_norm_g || !w_lm || !token || !confidence || !commit || !aligned16(h) ||
        !aligned16(final_norm_g) || !aligned16(w_lm))
        return fail(ctx, ACACHE_ERR_INVALID_ARG, "NULL or misaligned pointer");
    GemmArgs g{};
    g.a = wsp<void>(ctx, ctx->o_lxn); g.M = batch * n_blk; g.K = d.hidden;
    g.b[0] = w_lm; g.n[0] = vocab;
    g.epilogue = kEpiLogits;
    g.prep.enabled = 3; g.prep.x = h; g.prep.x_is_compact = 1; g.prep.compact_idx = block_rows; g.prep.compact_rows = h_rows;
    g.prep.k = 0; g.prep.e = n_blk; g.prep.gain = final_norm_g; g.prep.eps = d.rms_eps;
    g.logit_stats = wsp<float4>(ctx, ctx->o_lstats);
    g.partial = wsp<float>(ctx, ctx->o_gemm); g.status = wsp<uint32_t>(ctx, ctx->o_status);
    g.grid_bar = wsp<unsigned int>(ctx, ctx->o_gridbar);
    int nl = launch_gemm(g, stream);
    if (nl < 0) return check_cuda(ctx, "LM head") == ACACHE_OK ? fail(ctx, ACACHE_ERR_CUDA, "LM head launch failed") : ACACHE_ERR_CUDA;
    ctx->launches += nl;
    nl = launch_predict_commit(g, batch, n_blk, threshold, token, confidence, commit, stream);
    if (nl < 0) return check_cuda(ctx, "predict/commit") == ACACHE_OK ? fail(ctx, ACACHE_ERR_CUDA, "predict/commit launch failed") : ACACHE_ERR_CUDA;
    ctx->launches += nl;
    return check_cuda(ctx, "predict_commit");
}

acache_status acache_denoise_step(acache_ctx* ctx, int32_t n_layers, const acache_layer_weights* layers,
                                  acache_kv* kvs, const acache_request* req, const void* x0,
                                  const int32_t* anchor_idx, int32_t k, void* y_a, void* y_b, void** y_last,
                                  const int32_t* block_rows, int32_t n_blk, const void* final_norm_g,
                                  const void* w_lm, int32_t vocab, float threshold, int32_t* token,
                                  float* confidence, int32_t* commit, acache_stream_t stream) {
    if (!ctx) return ACACHE_ERR_INVALID_ARG;
    if (n_layers <= 0 || !layers || !kvs || !req || !x0 || !y_a || !y_b)
        return fail(ctx, ACACHE_ERR_INVALID_ARG, "NULL argument or n_layers <= 0");
    if (k < 0 || k > req->affix_len) return fail(ctx, ACACHE_ERR_INVALID_ARG, "k %d outside [0, affix_len]", k);
    // the ratio that maps back to exactly k anchors
    const double ratio = req->affix_len > 0 ? ((double)k - 0.5) / (double)req->affix_len : 0.0;
    if (acache_k_from_ratio(req->affix_len, k > 0 ? ratio : 0.0) != k) return fail(ctx, ACACHE_ERR_INVALID_ARG, "k not representable");
    const void* x = x0;
    void* y = y_a;
    for (int n = 0; n < n_layers; ++n) {
        y = (n & 1) ? y_b : y_a;
        acache_status s = acache_layer_step(ctx, &layers[n], req, &kvs[n], x, n > 0, k > 0 ? ratio : 0.0, 0u, nullptr,
                                            const_cast<int32_t*>(anchor_idx), y, stream);
        if (s != ACACHE_OK) return s;
        x = y;
    }
    if (y_last) *y_last = y;
    const int rows = k + req->n_extra;
    if (n_blk == 0 || req->batch == 0) return ACACHE_OK;
    if (rows == 0) return fail(ctx, ACACHE_ERR_INVALID_ARG, "no rows were recomputed: nothing to predict from");
    return acache_predict_commit(ctx, y, rows, block_rows, req->batch, n_blk, final_norm_g, w_lm, vocab, threshold, token,
                                 confidence, commit, stream);
}

acache_status acache_denoise_step_shared(acache_ctx* ctx, int32_t n_layers, const acache_layer_weights* layers,
                                         const acache_kv* kvs, const acache_request* req, const void* x0,
                                         const int32_t* anchor_idx, int32_t k, void* const* k_new, void* const* v_new,
                                         void* y_a, void* y_b, void** y_last, const int32_t* block_rows, int32_t n_blk,
                                         const void* final_norm_g, const void* w_lm, int32_t vocab, float threshold,
                                         int32_t* token, float* confidence, int32_t* commit, acache_stream_t stream) {
    if (!ctx) return ACACHE_ERR_INVALID_ARG;
    if (n_layers <= 0 || !layers || !kvs || !req || !x0 || !y_a || !y_b || !k_new || !v_new)
        return fail(ctx, ACACHE_ERR_INVALID_ARG, "NULL argument or n_layers <= 0");
    const void* x = x0;
    void* y = y_a;
    for (int n = 0; n < n_layers; ++n) {
        y = (n & 1) ? y_b : y_a;
        g_reuse_maps = n > 0;
        acache_status s = acache_recompute_anchors(ctx, &layers[n], req, &kvs[n], x, n > 0, anchor_idx, k, k_new[n], v_new[n], y,
                                                   stream);
        g_reuse_maps = false;
        if (s != ACACHE_OK) return s;
        x = y;
    }
    if (y_last) *y_last = y;
    const int rows = k + req->n_extra;
    if (n_blk == 0 || req->batch == 0) return ACACHE_OK;
    if (rows == 0) return fail(ctx, ACACHE_ERR_INVALID_ARG, "no rows were recomputed: nothing to predict from");
    return acache_predict_commit(ctx, y, rows, block_rows, req->batch, n_blk, final_norm_g, w_lm, vocab, threshold, token,
                                 confidence, commit, stream);
}

acache_status acache_recompute_rows_shared(acache_ctx* ctx, const acache_layer_weights* w, const acache_request* req_rows,
                                           const acache_request* req_slots, const acache_kv* kv, const void* x,
                                           int x_is_compact, const int32_t* anchor_idx, int32_t k, const int32_t* slot_rows,
                                           void* k_slots, void* v_slots, void* y, acache_stream_t stream) {
    if (!ctx) return ACACHE_ERR_INVALID_ARG;
    if (!kv || !req_slots) return fail(ctx, ACACHE_ERR_INVALID_ARG, "kv / req_slots is NULL");
    acache_status s = check_request(ctx, req_rows, kv, 0, true, true);
    if (s != ACACHE_OK) return s;
    if ((s = check_request(ctx, req_slots, kv, k, true, true)) != ACACHE_OK) return s;
    if ((s = check_weights(ctx, w, false)) != ACACHE_OK) return s;
    if (req_rows->batch != req_slots->batch || req_rows->ctx_len != req_slots->ctx_len ||
        req_rows->affix_start != req_slots->affix_start || req_rows->affix_len != req_slots->affix_len)
        return fail(ctx, ACACHE_ERR_INVALID_ARG, "req_rows and req_slots describe different contexts");
    if (req_rows->batch * req_rows->n_extra == 0) return ACACHE_OK;
    if (k + req_slots->n_extra == 0) return fail(ctx, ACACHE_ERR_INVALID_ARG, "the private slot array is empty");
    if (!x || !k_slots || !v_slots || !y || !slot_rows || !aligned16(x) || !aligned16(k_slots) || !aligned16(v_slots) ||
        !aligned16(y))
        return fail(ctx, ACACHE_ERR_INVALID_ARG, "x / k_slots / v_slots / y / slot_rows NULL or misaligned");
    if (k > 0 && !anchor_idx) return fail(ctx, ACACHE_ERR_INVALID_ARG, "anchor_idx is NULL");
    const PrivateRows priv{anchor_idx, k, req_slots->extra_rows, req_slots->n_extra, slot_rows};
    return run_recompute(ctx, w, req_rows, kv, false, x, x_is_compact, nullptr, 0, k_slots, v_slots, y, stream, &priv,
                         MapReuse{g_reuse_maps});
}

acache_status acache_decode_step_shared(acache_ctx* ctx, int32_t n_layers, const acache_layer_weights* layers,
                                        const acache_kv* kvs, const acache_request* req_rows,
                                        const acache_request* req_slots, const void* x0, const int32_t* anchor_idx,
                                        int32_t k, const int32_t* slot_rows, void* const* k_slots, void* const* v_slots,
                                        void* y_a, void* y_b, void** y_last, const int32_t* block_rows, int32_t n_blk,
                                        const void* final_norm_g, const void* w_lm, int32_t vocab, float threshold,
                                        int32_t* token, float* confidence, int32_t* commit, acache_stream_t stream) {
    if (!ctx) return ACACHE_ERR_INVALID_ARG;
    if (n_layers <= 0 || !layers || !kvs || !req_rows || !req_slots || !x0 || !y_a || !y_b || !k_slots || !v_slots)
        return fail(ctx, ACACHE_ERR_INVALID_ARG, "NULL argument or n_layers <= 0");
    const void* x = x0;
    void* y = y_a;
    for (int n = 0; n < n_layers; ++n) {
        y = (n & 1) ? y_b : y_a;
        g_reuse_maps = n > 0;
        acache_status s = acache_recompute_rows_shared(ctx, &layers[n], req_rows, req_slots, &kvs[n], x, n > 0, anchor_idx, k,
                                                       slot_rows, k_slots[n], v_slots[n], y, stream);
        g_reuse_maps = false;
        if (s != ACACHE_OK) return s;
        x = y;
    }
    if (y_last) *y_last = y;
    if (n_blk == 0 || req_rows->batch == 0) return ACACHE_OK;
    if (req_rows->n_extra == 0) return fail(ctx, ACACHE_ERR_INVALID_ARG, "no rows were recomputed: nothing to predict from");
    return acache_predict_commit(ctx, y, req_rows->n_extra, block_rows, req_rows->batch, n_blk, final_norm_g, w_lm, vocab,
                                 threshold, token, confidence, commit, stream);
}

acache_status acache_generate_block_shared(acache_ctx* ctx, int32_t n_layers, const acache_layer_weights* layers,
                                           const acache_kv* kvs, const acache_request* req_refresh,
                                           const acache_request* req_decode, const void* embed, const int32_t* anchor_idx,
                                           int32_t k, void* const* k_slots, void* const* v_slots, void* y_a, void* y_b,
                                           const int32_t* block_rows_refresh, const int32_t* block_rows_decode,
                                           int32_t n_blk, const void* final_norm_g, const void* w_lm, int32_t vocab,
                                           float threshold, int32_t mask_id, int32_t max_steps, int32_t* token,
                                           float* confidence, int32_t* commit, int32_t* remaining, int32_t* steps_done,
                                           acache_stream_t stream) {
    if (!ctx) return ACACHE_ERR_INVALID_ARG;
    if (!req_refresh || !req_decode || !steps_done || !remaining)
        return fail(ctx, ACACHE_ERR_INVALID_ARG, "NULL argument");
    if (!req_refresh->token_ids || req_refresh->token_ids != req_decode->token_ids)
        return fail(ctx, ACACHE_ERR_INVALID_ARG, "both requests must name the same token_ids array");
    if (req_decode->n_extra != n_blk || req_decode->batch != req_refresh->batch || req_decode->ctx_len != req_refresh->ctx_len)
        return fail(ctx, ACACHE_ERR_INVALID_ARG, "req_decode must recompute exactly the block's n_blk rows of the same batch");
    if (req_refresh->batch > 4096) return fail(ctx, ACACHE_ERR_INVALID_ARG, "batch too large for the step loop");
    *steps_done = 0;
    if (req_refresh->batch == 0 || n_blk == 0 || max_steps <= 0) return ACACHE_OK;
    int32_t* ids = const_cast<int32_t*>(req_refresh->token_ids);
    int32_t left[4096];
    for (int step = 0; step < max_steps; ++step) {
        // step 0 fills the private slots with the anchors and every request-specific row; later steps refresh
        // the block's rows inside those slots
        acache_status s;
        if (step == 0)
            s = acache_denoise_step_shared(ctx, n_layers, layers, kvs, req_refresh, embed, anchor_idx, k, k_slots, v_slots, y_a, y_b,
                                           nullptr, block_rows_refresh, n_blk, final_norm_g, w_lm, vocab, threshold, token,
                                           confidence, commit, stream);
        else
            s = acache_decode_step_shared(ctx, n_layers, layers, kvs, req_decode, req_refresh, embed, anchor_idx, k,
                                          block_rows_refresh, k_slots, v_slots, y_a, y_b, nullptr, block_rows_decode, n_blk,
                                          final_norm_g, w_lm, vocab, threshold, token, confidence, commit, stream);
        if (s != ACACHE_OK) return s;
        s = acache_commit_update(ctx, ids, req_refresh->ctx_len, req_decode->extra_rows, req_refresh->batch, n_blk, token,
                                 confidence, mask_id, threshold, remaining, stream);
        if (s != ACACHE_OK) return s;
        *steps_done = step + 1;
        if (cudaMemcpyAsync(left, remaining, sizeof(int32_t) * req_refresh->batch, cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
            cudaStreamSynchronize(stream) != cudaSuccess)
            return check_cuda(ctx, "generate_block_shared read-back") == ACACHE_OK ? fail(ctx, ACACHE_ERR_CUDA, "read-back failed")
                                                                                   : ACACHE_ERR_CUDA;
        int total = 0;
        for (int b = 0; b < req_refresh->batch; ++b) total += left[b];
        if (total == 0) break;
    }
    return ACACHE_OK;
}

acache_status acache_probe_select(acache_ctx* ctx, int32_t n_layers, const acache_layer_weights* layers, acache_kv* kvs,
                                  const acache_request* req, const void* x0, double ratio, uint32_t flags, void* y_a,
                                  void* y_b, float* scores, int32_t* anchor_idx, acache_stream_t stream) {
    if (!ctx) return ACACHE_ERR_INVALID_ARG;
    if (n_layers <= 0 || !layers || !kvs || !req || !x0 || !y_a || !y_b || !scores)
        return fail(ctx, ACACHE_ERR_INVALID_ARG, "NULL argument or n_layers <= 0");
    if (flags & ~(uint32_t)ACACHE_F_SCORE_NORM_FULL) return fail(ctx, ACACHE_ERR_INVALID_ARG, "only ACACHE_F_SCORE_NORM_FULL is accepted here");
    const int k = acache_k_from_ratio(req->affix_len, ratio);
    if (k > 0 && !anchor_idx) return fail(ctx, ACACHE_ERR_INVALID_ARG, "anchor_idx is NULL");
    const void* x = x0;
    for (int n = 0; n < n_layers; ++n) {
        void* y = (n & 1) ? y_b : y_a;
        // K = 0 anchors: the rows are the request-specific ones; the affix keys stay as cached (stale)
        acache_status s = acache_layer_step(ctx, &layers[n], req, &kvs[n], x, n > 0, 0.0,
                                            flags | ACACHE_F_SCORE | (n > 0 ? ACACHE_F_ACCUMULATE : 0u), scores, nullptr, y, stream);
        if (s != ACACHE_OK) return s;
        x = y;
    }
    return acache_select_topk(ctx, scores, req->batch, req->affix_len, k, anchor_idx, stream);
}

acache_status acache_commit_update(acache_ctx* ctx, int32_t* token_ids, int32_t ctx_len, const int32_t* block_pos,
                                   int32_t batch, int32_t n_blk, const int32_t* token, const float* confidence,
                                   int32_t mask_id, float threshold, int32_t* remaining, acache_stream_t stream) {
    if (!ctx) return ACACHE_ERR_INVALID_ARG;
    if (!ctx->ws) return fail(ctx, ACACHE_ERR_WORKSPACE, "workspace not set");
    if (batch < 0 || n_blk < 0 || ctx_len <= 0) return fail(ctx, ACACHE_ERR_INVALID_ARG, "negative size");
    if (batch == 0) return ACACHE_OK;
    if (!token_ids || !remaining || (n_blk > 0 && (!block_pos || !token || !confidence)))
        return fail(ctx, ACACHE_ERR_INVALID_ARG, "NULL pointer");
    launch_commit_update(token_ids, ctx_len, block_pos, batch, n_blk, token, confidence, mask_id, threshold, remaining,
                         wsp<uint32_t>(ctx, ctx->o_status), stream);
    ctx->launches += 1;
    return check_cuda(ctx, "commit_update");
}

acache_status acache_generate_block(acache_ctx* ctx, int32_t n_layers, const acache_layer_weights* layers, acache_kv* kvs,
                                    const acache_request* req_refresh, const acache_request* req_decode,
                                    const void* embed, const int32_t* anchor_idx, int32_t k, void* y_a, void* y_b,
                                    const int32_t* block_rows_refresh, const int32_t* block_rows_decode, int32_t n_blk,
                                    const void* final_norm_g, const void* w_lm, int32_t vocab, float threshold,
                                    int32_t mask_id, int32_t max_steps, int32_t* token, float* confidence,
                                    int32_t* commit, int32_t* remaining, int32_t* steps_done, acache_stream_t stream) {
    if (!ctx) return ACACHE_ERR_INVALID_ARG;
    if (!req_refresh || !req_decode || !steps_done || !remaining)
        return fail(ctx, ACACHE_ERR_INVALID_ARG, "NULL argument");
    if (!req_refresh->token_ids || req_refresh->token_ids != req_decode->token_ids)
        return fail(ctx, ACACHE_ERR_INVALID_ARG, "both requests must name the same token_ids array");
    if (req_decode->n_extra != n_blk || req_decode->batch != req_refresh->batch || req_decode->ctx_len != req_refresh->ctx_len)
        return fail(ctx, ACACHE_ERR_INVALID_ARG, "req_decode must recompute exactly the block's n_blk rows of the same batch");
    if (req_refresh->batch > 4096) return fail(ctx, ACACHE_ERR_INVALID_ARG, "batch too large for the step loop");
    *steps_done = 0;
    if (req_refresh->batch == 0 || n_blk == 0 || max_steps <= 0) return ACACHE_OK;
    int32_t* ids = const_cast<int32_t*>(req_refresh->token_ids);
    int32_t left[4096];
    for (int step = 0; step < max_steps; ++step) {
        // step 0 refreshes the anchors and every request-specific row; later steps only the block's rows
        const bool refresh = step == 0;
        const acache_request* r = refresh ? req_refresh : req_decode;
        acache_status s = acache_denoise_step(ctx, n_layers, layers, kvs, r, embed, refresh ? anchor_idx : nullptr,
                                              refresh ? k : 0, y_a, y_b, nullptr,
                                              refresh ? block_rows_refresh : block_rows_decode, n_blk, final_norm_g, w_lm,
                                              vocab, threshold, token, confidence, commit, stream);
        if (s != ACACHE_OK) return s;
        s = acache_commit_update(ctx, ids, r->ctx_len, req_decode->extra_rows, r->batch, n_blk, token, confidence, mask_id,
                                 threshold, remaining, stream);
        if (s != ACACHE_OK) return s;
        *steps_done = step + 1;
        // the schedule ends when no request has a masked position left in the block: one small read-back per step
        if (cudaMemcpyAsync(left, remaining, sizeof(int32_t) * r->batch, cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
            cudaStreamSynchronize(stream) != cudaSuccess)
            return check_cuda(ctx, "generate_block read-back") == ACACHE_OK ? fail(ctx, ACACHE_ERR_CUDA, "read-back failed") : ACACHE_ERR_CUDA;
        int total = 0;
        for (int b = 0; b < r->batch; ++b) total += left[b];
        if (total == 0) break;
    }
    return ACACHE_OK;
}

int32_t acache_host_x_in_place(const void* x_host) {
    static const bool on = [] { const char* e = getenv("ACACHE_HOST_X_IN_PLACE"); return !e || atoi(e) != 0; }();
    return on && mapped_device_pointer(x_host) != nullptr;
}

acache_status acache_layer_step_host(acache_ctx* ctx, const acache_layer_weights* w, const acache_request* req,
                                     acache_kv* kv, const void* x_host, double ratio, uint32_t flags,
                                     float* scores_host, int32_t* anchor_idx_host, void* y_host,
                                     acache_stream_t stream) {
    if (!ctx) return ACACHE_ERR_INVALID_ARG;
    if (!req || !x_host || !scores_host || !y_host) return fail(ctx, ACACHE_ERR_INVALID_ARG, "NULL argument");
    if (!ctx->ws) return fail(ctx, ACACHE_ERR_WORKSPACE, "workspace not set");
    const acache_model_desc& d = ctx->d;
    if (req->batch < 0 || req->batch > d.max_batch || req->ctx_len <= 0 || req->ctx_len > d.max_ctx ||
        req->affix_len < 0 || req->affix_len > d.max_affix)
        return fail(ctx, ACACHE_ERR_INVALID_ARG, "batch / ctx_len / affix_len outside the context's limits");
    const int k = acache_k_from_ratio(req->affix_len, ratio);
    if (k > 0 && !anchor_idx_host) return fail(ctx, ACACHE_ERR_INVALID_ARG, "anchor_idx_host is NULL");
    void* xs = wsp<void>(ctx, ctx->o_xstage);
    void* ys = wsp<void>(ctx, ctx->o_ystage);
    float* ss = wsp<float>(ctx, ctx->o_sstage);
    int32_t* as = wsp<int32_t>(ctx, ctx->o_astage);
    const size_t xb = (size_t)req->batch * req->ctx_len * d.hidden * 2;
    // The step reads x row by row (the masked rows and the rows it recomputes), a small part of the whole:
    // page-locked x is read in place over the bus by the kernels, anything else is staged whole (in place only
    // while those rows are at most a quarter of x: reads over the bus from a kernel are slower, byte for byte,
    // than the copy engine's transfer).  The recomputed rows are needed twice (projection input, residual of the
    // output projection): the row preparation leaves a copy in the staging buffer, which is free then, and the
    // residual is read from there (measured: 290 -> 219 us per step at 103 rows).
    const int64_t pulled = (int64_t)req->n_masked + (int64_t)k + req->n_extra;
    const void* x_dev = pulled * 4 <= req->ctx_len && acache_host_x_in_place(x_host) ? mapped_device_pointer(x_host) : nullptr;
    if (!x_dev) {
        if (cudaMemcpyAsync(xs, x_host, xb, cudaMemcpyHostToDevice, stream) != cudaSuccess) return check_cuda(ctx, "H2D x");
        x_dev = xs;
    }
    ctx->stash_rows = x_dev != xs ? xs : nullptr;
    acache_status s = acache_layer_step(ctx, w, req, kv, x_dev, 0, ratio, flags | ACACHE_F_SCORE | ACACHE_F_SELECT, ss, as,
                                        ys, stream);
    ctx->stash_rows = nullptr;
    if (s != ACACHE_OK) return s;
    // Results: y through the copy engine (written over the bus by the projection's epilogue it cost 40 us more); scores
    // and anchors, when page-locked, by one small copy kernel instead of two more transfers.
    void* s_map = const_cast<void*>(mapped_device_pointer(scores_host));
    void* a_map = k ? const_cast<void*>(mapped_device_pointer(anchor_idx_host)) : nullptr;
    const size_t rows = (size_t)req->batch * (k + req->n_extra);
    const size_t n_s = (size_t)req->batch * req->affix_len, n_a = (size_t)req->batch * k;
    bool ok = true;
    if (!(flags & ACACHE_F_NO_RECOMPUTE) && rows)
        ok &= cudaMemcpyAsync(y_host, ys, rows * d.hidden * 2, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
    if (s_map && (a_map || !k) && n_s + n_a < (1u << 30)) {
        launch_copy_out_words(ss, s_map, (int)n_s, as, a_map, (int)n_a, stream);
        ++ctx->launches;
    } else {
        if (k) ok &= cudaMemcpyAsync(anchor_idx_host, as, n_a * 4, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
        ok &= cudaMemcpyAsync(scores_host, ss, n_s * 4, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
    }
    if (!ok) return check_cuda(ctx, "D2H") == ACACHE_OK ? fail(ctx, ACACHE_ERR_CUDA, "D2H copy failed") : ACACHE_ERR_CUDA;
    return ACACHE_OK;
}

}  // extern "C"
