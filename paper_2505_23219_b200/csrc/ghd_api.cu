// C-ABI entry points of libghd: argument validation, workspace layout, and the
// order in which the kernels of a layer / a step are enqueued.
#include <cstdio>
#include <cstring>
#include <new>

#include "internal.h"

namespace ghd {

struct StepGraph {
    std::vector<uint64_t> key;
    cudaGraphExec_t exec;
    int64_t kernels;
};

static size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

size_t carve_workspace(ghd_ctx* c, char* base) {
    const ghd_model_cfg& m = c->cfg;
    const size_t N = m.max_nodes, d = m.d_model, f = m.d_ffn, es = (m.dtype == GHD_F32) ? 4 : 2;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t at = off; off = align_up(off + bytes, 256); return base ? base + at : nullptr; };
    const size_t raw_cols = (3 * d > 2 * f) ? 3 * d : 2 * f;
    c->status = (int*)take(256);
    c->kv_len_word = c->status ? c->status + 16 : nullptr;       // same 256-byte block, its own 64-byte line
    c->counters = (int*)take(sizeof(int) * 4096);
    for (int b = 0; b < 2; ++b) c->ssq[b] = (float*)take(sizeof(float) * SSQ_MAX_TILES * SSQ_PITCH);
    c->xres = (float*)take(N * d * 4);
    c->hbuf = take(N * d * es);
    c->qbuf = take(N * d * es);
    c->attnbuf = take(N * d * es);
    c->ubuf = take(N * f * es);
    c->raw = (float*)take(N * raw_cols * 4);
    c->att_o = (float*)take((size_t)c->max_splits * N * d * 4);
    c->att_ml = (float*)take((size_t)c->max_splits * N * m.n_heads * 2 * 4);
    c->gemm_part = (float*)take((size_t)c->sm_count * 2 * 256 * 128 * 4);
    c->logits = (float*)take(N * (size_t)m.vocab * 4);
    c->mlogits = (float*)take((size_t)GHD_MAX_DRAFT_HEADS * m.vocab * 4);
    return off;
}

static ghd_status fail(ghd_ctx* c, ghd_status s, const char* what) {
    if (c) snprintf(c->err, sizeof(c->err), "%s", what);
    return s;
}

static ghd_status check_cuda(ghd_ctx* c, const char* where) {
    const cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) return GHD_OK;
    snprintf(c->err, sizeof(c->err), "%s: %s", where, cudaGetErrorString(e));
    return GHD_ECUDA;
}

static ghd_status check_tree(ghd_ctx* c, const ghd_tree* t) {
    if (!t || !t->mask || !t->depth || !t->pos || !t->rope) return fail(c, GHD_EINVAL, "tree: null pointer");
    if (t->n < 1 || t->n > c->cfg.max_nodes || t->n_words != (t->n + 63) / 64) return fail(c, GHD_ETREE, "tree: not built");
    if (t->kv_len == GHD_KV_LEN_DEVICE) return GHD_OK;       // checked on the device when the tree was built
    if (t->kv_len < 0 || t->kv_len + t->n > c->cfg.max_kv_len) return fail(c, GHD_ENOSPACE, "tree: kv_len + n > max_kv_len");
    return GHD_OK;
}

// One projection: tcgen05 kernel with the fused epilogue when it applies, else the
// CUDA-core GEMM into the raw buffer followed by the matching element-wise kernel.
static ghd_status project(ghd_ctx* c, const void* x, const void* w, int n, int k, int m, const EpiArgs& epi,
                          const ghd_tree* t, const ghd_kv_layer* kv) {
    const bool tc_ok = c->cfg.dtype == GHD_F16 && gemm_tc_supported(c, n, k, m, epi.mode);
    if (c->opt_gemm_path == 2 && !tc_ok) return fail(c, GHD_EUNSUPPORTED, "tcgen05 GEMM does not take this shape/type");
    if (tc_ok && c->opt_gemm_path != 1) {
        c->path_count[GHD_PATH_GEMM_TILE]++;
        return launch_gemm_tc(c, x, w, n, k, m, epi);
    }
    c->path_count[GHD_PATH_GEMM_SIMT]++;
    float* dst = (epi.mode == EPI_RAW) ? epi.out_f32 : c->raw;
    launch_gemm_simt(c, x, w, n, k, m, dst);
    switch (epi.mode) {
        case EPI_ROPE_KV: launch_rope_append(c, dst, t, kv); break;
        case EPI_RESID: launch_residual(c, dst, n); break;
        case EPI_SWIGLU: launch_swiglu(c, dst, n); break;
        default: break;
    }
    return GHD_OK;
}

// RMSNorm of the residual stream into hbuf, first folding in a projection whose reduction was deferred.
static void norm_into_h(ghd_ctx* c, const void* gain, int n) {
    if (c->pending.active) launch_fold_pending(c, n, gain, c->hbuf, nullptr);
    else launch_rmsnorm(c, c->xres, gain, n, c->hbuf);
}

// Projection whose result is added to the residual stream.  On the tcgen05 path the k-split partial
// tiles are left in the workspace and the next norm kernel sums them (no CTA waits, no fix-up pass).
static ghd_status project_residual(ghd_ctx* c, const void* x, const void* w, int n, int k, int m, EpiArgs e,
                                   const ghd_tree* t, const ghd_kv_layer* kv) {
    if (c->cfg.dtype == GHD_F16 && c->opt_gemm_path != 1 && gemm_tc_supported(c, n, k, m, EPI_DEFER)) {
        e.mode = EPI_DEFER;
        c->path_count[GHD_PATH_GEMM_TILE]++;
        return launch_gemm_tc(c, x, w, n, k, m, e);
    }
    e.mode = EPI_RESID; e.out_f32 = c->xres;
    return project(c, x, w, n, k, m, e, t, kv);
}

static ghd_status attention(ghd_ctx* c, const void* q, const ghd_kv_layer* kv, const ghd_tree* t, void* out) {
    const bool tc_ok = attn_tc_supported(c, t);
    const bool coo = c->opt_attn_sparse == 1;
    if (coo && (!t->coo_ptr || !t->coo_col)) return fail(c, GHD_EINVAL, "attention: the tree carries no coordinate index");
    if (c->opt_attn_path == 2 && !tc_ok) return fail(c, GHD_EUNSUPPORTED, "tcgen05 attention does not take this type/shape");
    if (coo) c->path_count[GHD_PATH_ATTN_COO]++;
    if (tc_ok && c->opt_attn_path != 1) { c->path_count[GHD_PATH_ATTN_TC]++; return launch_attn_tc(c, q, kv, t, out, coo); }
    c->path_count[GHD_PATH_ATTN_SIMT]++;
    launch_attn_simt(c, q, kv, t, out, coo);
    return GHD_OK;
}

static EpiArgs epi_base(ghd_ctx* c, const ghd_tree* t) {
    EpiArgs e{};
    e.rope = t->rope; e.kv_len = t->kv_len; e.kv_len_dev = kv_len_dev_of(c, t); e.max_kv_len = c->cfg.max_kv_len; e.d_head = c->cfg.d_head; e.d_model = c->cfg.d_model;
    return e;
}

static ghd_status layer_body(ghd_ctx* c, const ghd_layer_weights* w, const ghd_kv_layer* kv, const ghd_tree* t) {
    const ghd_model_cfg& m = c->cfg;
    const int n = t->n, d = m.d_model, f = m.d_ffn;
    ghd_status s;
    EpiArgs e = epi_base(c, t);
    norm_into_h(c, w->rms1, n);
    e.mode = EPI_ROPE_KV; e.out_t = c->qbuf; e.k_cache = kv->k; e.v_cache = kv->v;
    if ((s = project(c, c->hbuf, w->wqkv, n, d, 3 * d, e, t, kv)) != GHD_OK) return s;
    if ((s = attention(c, c->qbuf, kv, t, c->attnbuf)) != GHD_OK) return s;
    if ((s = project_residual(c, c->attnbuf, w->wo, n, d, d, e, t, kv)) != GHD_OK) return s;
    norm_into_h(c, w->rms2, n);
    e.mode = EPI_SWIGLU; e.out_t = c->ubuf;
    if ((s = project(c, c->hbuf, w->w_gate_up, n, d, 2 * f, e, t, kv)) != GHD_OK) return s;
    if ((s = project_residual(c, c->ubuf, w->w_down, n, f, d, e, t, kv)) != GHD_OK) return s;
    return GHD_OK;
}

// True when the four projections of a layer can run on the tcgen05 path with the norms folded into their
// epilogues: the projection into the residual stream adds, writes the gain-weighted rows of the next
// norm and per-tile sums of squares; the projection that reads those rows multiplies by 1 / rms.
static bool fused_norm_ok(const ghd_ctx* c, int n) {
    const ghd_model_cfg& m = c->cfg;
    if (c->opt_fused_norm != 1 || m.dtype != GHD_F16 || c->opt_gemm_path == 1) return false;
    return gemm_tc_supported(c, n, m.d_model, 3 * m.d_model, EPI_ROPE_KV) && gemm_tc_supported(c, n, m.d_model, m.d_model, EPI_RESID_NORM) &&
           gemm_tc_supported(c, n, m.d_model, 2 * m.d_ffn, EPI_SWIGLU) && gemm_tc_supported(c, n, m.d_ffn, m.d_model, EPI_RESID_NORM);
}

static void with_row_scale(ghd_ctx* c, EpiArgs& e) {
    e.ssq_in = c->ssq[c->h_ssq];
    e.ssq_in_tiles = c->ssq_tiles[c->h_ssq];
    e.rms_eps = c->cfg.rms_eps;
}

// First norm of a call on the fused-norm path.
static void prenorm_into_h(ghd_ctx* c, const void* gain, int n) {
    launch_prenorm(c, gain, n, c->hbuf, c->ssq[0]);
    c->ssq_tiles[0] = 1;
    c->h_ssq = 0;
}

// One layer on the fused-norm path.  On entry hbuf holds xres * rms1 gain with its sums of squares in
// ssq[h_ssq]; on exit hbuf holds xres * next_gain likewise (next_gain = nullptr: residual stream only).
static ghd_status layer_body_fused(ghd_ctx* c, const ghd_layer_weights* w, const ghd_kv_layer* kv, const ghd_tree* t, const void* next_gain) {
    const ghd_model_cfg& m = c->cfg;
    const int n = t->n, d = m.d_model, f = m.d_ffn;
    ghd_status s;
    const EpiArgs base = epi_base(c, t);
    EpiArgs e = base;
    e.mode = EPI_ROPE_KV; e.out_t = c->qbuf; e.k_cache = kv->k; e.v_cache = kv->v;
    with_row_scale(c, e);
    if ((s = project(c, c->hbuf, w->wqkv, n, d, 3 * d, e, t, kv)) != GHD_OK) return s;
    if ((s = attention(c, c->qbuf, kv, t, c->attnbuf)) != GHD_OK) return s;
    int nxt = c->h_ssq ^ 1;
    e = base;
    e.mode = EPI_RESID_NORM; e.out_f32 = c->xres; e.gain = w->rms2; e.xg_out = c->hbuf; e.ssq_out = c->ssq[nxt];
    if ((s = project(c, c->attnbuf, w->wo, n, d, d, e, t, kv)) != GHD_OK) return s;
    c->ssq_tiles[nxt] = d / 128;
    c->h_ssq = nxt;
    e = base;
    e.mode = EPI_SWIGLU; e.out_t = c->ubuf;
    with_row_scale(c, e);
    if ((s = project(c, c->hbuf, w->w_gate_up, n, d, 2 * f, e, t, kv)) != GHD_OK) return s;
    nxt = c->h_ssq ^ 1;
    e = base;
    if (next_gain) { e.mode = EPI_RESID_NORM; e.gain = next_gain; e.xg_out = c->hbuf; e.ssq_out = c->ssq[nxt]; }
    else e.mode = EPI_RESID;
    e.out_f32 = c->xres;
    if ((s = project(c, c->ubuf, w->w_down, n, f, d, e, t, kv)) != GHD_OK) return s;
    if (next_gain) { c->ssq_tiles[nxt] = d / 128; c->h_ssq = nxt; }
    else c->h_ssq = -1;
    return GHD_OK;
}

static ghd_status step_body(ghd_ctx* c, const ghd_model_weights* w, ghd_kv_layer* kv, const ghd_tree* t,
                            const int32_t* tokens, float* logits, int32_t* amax) {
    const ghd_model_cfg& m = c->cfg;
    ghd_status s;
    launch_embed(c, w->embed, tokens, t->n);
    EpiArgs e{};
    e.mode = EPI_RAW; e.out_f32 = logits;
    c->h_ssq = -1;
    if (fused_norm_ok(c, t->n) && gemm_tc_supported(c, t->n, m.d_model, m.vocab, EPI_RAW)) {
        prenorm_into_h(c, m.n_layers > 0 ? w->layers[0].rms1 : w->rms_final, t->n);
        for (int l = 0; l < m.n_layers; ++l)
            if ((s = layer_body_fused(c, &w->layers[l], &kv[l], t, l + 1 < m.n_layers ? w->layers[l + 1].rms1 : w->rms_final)) != GHD_OK) return s;
        with_row_scale(c, e);       // hbuf stays gain-weighted: the drafting heads divide by the rms themselves
        if ((s = project(c, c->hbuf, w->lm_head, t->n, m.d_model, m.vocab, e, t, nullptr)) != GHD_OK) return s;
        launch_argmax(c, logits, t->n, m.vocab, amax);
        return GHD_OK;
    }
    for (int l = 0; l < m.n_layers; ++l)
        if ((s = layer_body(c, &w->layers[l], &kv[l], t)) != GHD_OK) return s;
    norm_into_h(c, w->rms_final, t->n);
    if ((s = project(c, c->hbuf, w->lm_head, t->n, m.d_model, m.vocab, e, t, nullptr)) != GHD_OK) return s;
    launch_argmax(c, logits, t->n, m.vocab, amax);
    return GHD_OK;
}

}  // namespace ghd

using namespace ghd;

extern "C" {

ghd_status ghd_create(const ghd_model_cfg* cfg, void* cuda_stream, ghd_ctx** out) {
    if (!cfg || !out) return GHD_EINVAL;
    *out = nullptr;
    if (cfg->d_model <= 0 || cfg->n_heads <= 0 || cfg->d_ffn <= 0 || cfg->vocab <= 0 || cfg->n_layers < 0 ||
        cfg->max_kv_len <= 0 || cfg->max_nodes < 1 || cfg->max_nodes > GHD_MAX_NODES ||
        (cfg->dtype != GHD_F32 && cfg->dtype != GHD_F16) || !(cfg->rms_eps >= 0.f) || !(cfg->rope_theta > 0.f))
        return GHD_EINVAL;
    if (cfg->d_model != cfg->n_heads * cfg->d_head || cfg->n_kv_heads != cfg->n_heads ||
        (cfg->d_head != 64 && cfg->d_head != 128) || cfg->d_model % 8 || cfg->d_ffn % 8)
        return GHD_ESHAPE;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return GHD_ECUDA;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return GHD_ECUDA;
    ghd_ctx* c = new (std::nothrow) ghd_ctx();
    if (!c) return GHD_EINVAL;
    memset(c->err, 0, sizeof(c->err));
    c->cfg = *cfg;
    c->stream = (cudaStream_t)cuda_stream;
    c->cur = c->stream;
    c->cap_stream = nullptr;
    c->device = dev;
    c->sm_count = sms;
    c->opt_gemm_path = c->opt_attn_splits = c->opt_attn_path = c->opt_graph = c->opt_gemm_ctas = c->opt_gemm_burst = c->opt_no_pdl = c->opt_gemm_stages = c->opt_gemm_epi = c->opt_attn_sparse = c->opt_chain_calls = c->opt_fused_norm = c->opt_gemm_pair = c->opt_attn_rows = c->opt_gemm_skew = c->opt_attn_small = 0;
    c->ws = nullptr;
    c->ws_bytes = 0;
    c->max_splits = 16;
    c->pending.active = 0;
    c->h_ssq = -1;
    c->kv_len_hint = 0;
    c->entry_fresh = c->opt_chain_calls ? 0 : 1;
    c->attr_gemm = c->attr_attn = c->attr_attn_small = false;
    c->launches = 0;
    memset(c->path_count, 0, sizeof(c->path_count));
    c->tmaps = new std::map<TmapKey, std::vector<uint64_t>>();
    c->graphs = new std::vector<StepGraph*>();
    carve_workspace(c, nullptr);
    *out = c;
    return GHD_OK;
}

void ghd_destroy(ghd_ctx* c) {
    if (!c) return;
    for (StepGraph* g : *c->graphs) { cudaGraphExecDestroy(g->exec); delete g; }
    if (c->cap_stream) cudaStreamDestroy(c->cap_stream);
    delete c->graphs;
    delete c->tmaps;
    delete c;
}

size_t ghd_workspace_bytes(const ghd_ctx* c) {
    if (!c) return 0;
    ghd_ctx tmp = *c;
    return carve_workspace(&tmp, nullptr);
}

ghd_status ghd_set_workspace(ghd_ctx* c, void* dev_ptr, size_t bytes) {
    if (!c || !dev_ptr) return GHD_EINVAL;
    if (((uintptr_t)dev_ptr & 255) != 0) return fail(c, GHD_EINVAL, "workspace must be 256-byte aligned");
    if (bytes < ghd_workspace_bytes(c)) return fail(c, GHD_ENOSPACE, "workspace too small");
    c->ws = (char*)dev_ptr;
    c->ws_bytes = bytes;
    carve_workspace(c, c->ws);
    // status word and tile arrival counters must start at zero
    if (cudaMemsetAsync(c->status, 0, 256 + sizeof(int) * 4096, c->stream) != cudaSuccess) return check_cuda(c, "workspace clear");
    return GHD_OK;
}

ghd_status ghd_set_option(ghd_ctx* c, int32_t option, int32_t value) {
    if (!c || value < 0) return GHD_EINVAL;
    switch (option) {
        case GHD_OPT_GEMM_PATH: if (value > 2) return GHD_EINVAL; c->opt_gemm_path = value; break;
        case GHD_OPT_ATTN_SPLITS: if (value > c->max_splits) return GHD_EINVAL; c->opt_attn_splits = value; break;
        case GHD_OPT_ATTN_PATH: if (value > 2) return GHD_EINVAL; c->opt_attn_path = value; break;
        case GHD_OPT_GRAPH: if (value > 2) return GHD_EINVAL; c->opt_graph = value; break;
        case GHD_OPT_GEMM_CTAS: c->opt_gemm_ctas = value; break;
        case GHD_OPT_NO_PDL: c->opt_no_pdl = value ? 1 : 0; break;
        case GHD_OPT_GEMM_STAGES: if (value == 1 || value > 10) return GHD_EINVAL; c->opt_gemm_stages = value; break;
        case GHD_OPT_CHAIN_CALLS: c->opt_chain_calls = value ? 1 : 0; break;
        case GHD_OPT_FUSED_NORM: if (value > 1) return GHD_EINVAL; c->opt_fused_norm = value; break;
        case GHD_OPT_GEMM_PAIR: if (value > 2) return GHD_EINVAL; c->opt_gemm_pair = value; break;
        case GHD_OPT_ATTN_ROWS: if (value > 1) return GHD_EINVAL; c->opt_attn_rows = value; break;
        case GHD_OPT_GEMM_SKEW: if (value > 64) return GHD_EINVAL; c->opt_gemm_skew = value; break;
        case GHD_OPT_ATTN_SMALL: if (value > 2) return GHD_EINVAL; c->opt_attn_small = value; break;
        case GHD_OPT_ATTN_SPARSE: if (value > 1) return GHD_EINVAL; c->opt_attn_sparse = value; break;
        case GHD_OPT_GEMM_EPI: if (value > 2) return GHD_EINVAL; c->opt_gemm_epi = value; break;
        case GHD_OPT_GEMM_BURST: if (value > 8) return GHD_EINVAL; c->opt_gemm_burst = value; break;
        default: return GHD_EINVAL;
    }
    return GHD_OK;
}

static ghd_status tree_common(ghd_ctx* c, int32_t n, int32_t kv_len, ghd_tree* tree) {
    if (!c || !tree) return GHD_EINVAL;
    if (!tree->mask || !tree->parent || !tree->depth || !tree->pos || !tree->rope) return fail(c, GHD_EINVAL, "tree: null buffer");
    if ((tree->coo_ptr == nullptr) != (tree->coo_col == nullptr)) return fail(c, GHD_EINVAL, "tree: give both index buffers or neither");
    if (n < 1 || n > c->cfg.max_nodes) return fail(c, GHD_ETREE, "tree: n outside [1, max_nodes]");
    if (kv_len == GHD_KV_LEN_DEVICE) {
        if (n > c->cfg.max_kv_len) return fail(c, GHD_ENOSPACE, "tree: n > max_kv_len");
        return GHD_OK;
    }
    if (kv_len < 0) return fail(c, GHD_EINVAL, "tree: negative kv_len");
    if ((int64_t)kv_len + n > c->cfg.max_kv_len) return fail(c, GHD_ENOSPACE, "tree: kv_len + n > max_kv_len");
    return GHD_OK;
}

ghd_status ghd_tree_build(ghd_ctx* c, const int32_t* parent_host, int32_t n, int32_t kv_len, ghd_tree* tree) {
    ghd_status s = tree_common(c, n, kv_len, tree);
    if (s != GHD_OK) return s;
    if (!parent_host) return fail(c, GHD_EINVAL, "tree: null parent array");
    if (parent_host[0] != -1) return fail(c, GHD_ETREE, "tree: parent[0] must be -1");
    for (int i = 1; i < n; ++i)
        if (parent_host[i] < 0 || parent_host[i] >= i) return fail(c, GHD_ETREE, "tree: need 0 <= parent[i] < i");
    tree->n = n; tree->kv_len = kv_len; tree->n_words = (n + 63) / 64; tree->has_parent = 1;
    launch_tree_build(c, parent_host, tree);
    return check_cuda(c, "tree_build");
}

ghd_status ghd_tree_from_mask(ghd_ctx* c, const uint64_t* mask_host, const int32_t* depth_host,
                              const int32_t* parent_host, int32_t n, int32_t kv_len, ghd_tree* tree) {
    ghd_status s = tree_common(c, n, kv_len, tree);
    if (s != GHD_OK) return s;
    if (!mask_host) return fail(c, GHD_EINVAL, "tree: null mask");
    const int W = (n + 63) / 64;
    for (int i = 0; i < n; ++i) {
        if (!((mask_host[(size_t)i * W + (i >> 6)] >> (i & 63)) & 1ull)) return fail(c, GHD_ETREE, "mask: row lacks its own bit");
        for (int j = i + 1; j < W * 64; ++j)
            if ((mask_host[(size_t)i * W + (j >> 6)] >> (j & 63)) & 1ull) return fail(c, GHD_ETREE, "mask: bit above the diagonal");
        if (depth_host && (depth_host[i] < 0 || depth_host[i] >= n)) return fail(c, GHD_ETREE, "mask: bad depth");
    }
    if (parent_host) {
        if (parent_host[0] != -1) return fail(c, GHD_ETREE, "tree: parent[0] must be -1");
        for (int i = 1; i < n; ++i)
            if (parent_host[i] < 0 || parent_host[i] >= i) return fail(c, GHD_ETREE, "tree: need 0 <= parent[i] < i");
    }
    tree->n = n; tree->kv_len = kv_len; tree->n_words = W; tree->has_parent = parent_host ? 1 : 0;
    // pageable host memory: the copies are staged before the call returns
    cudaMemcpyAsync(tree->mask, mask_host, sizeof(uint64_t) * n * W, cudaMemcpyHostToDevice, c->stream);
    if (depth_host) cudaMemcpyAsync(tree->depth, depth_host, sizeof(int32_t) * n, cudaMemcpyHostToDevice, c->stream);
    if (parent_host) cudaMemcpyAsync(tree->parent, parent_host, sizeof(int32_t) * n, cudaMemcpyHostToDevice, c->stream);
    launch_tree_from_mask(c, tree, depth_host != nullptr, mask_host);
    return check_cuda(c, "tree_from_mask");
}

ghd_status ghd_verify_layer(ghd_ctx* c, const ghd_layer_weights* w, ghd_kv_layer* kv, const ghd_tree* tree,
                            const void* x_in, void* x_out) {
    if (!c || !w || !kv || !x_in || !x_out) return GHD_EINVAL;
    if (!c->ws) return fail(c, GHD_ENOSPACE, "no workspace set");
    if (!w->wqkv || !w->wo || !w->w_gate_up || !w->w_down || !w->rms1 || !w->rms2 || !kv->k || !kv->v)
        return fail(c, GHD_EINVAL, "layer: null weight or cache pointer");
    ghd_status s = check_tree(c, tree);
    if (s != GHD_OK) return s;
    if (kv->len != tree->kv_len) return fail(c, GHD_EINVAL, "layer: kv.len differs from tree.kv_len");
    c->pending.active = 0;
    c->entry_fresh = c->opt_chain_calls ? 0 : 1;
    launch_load_x(c, x_in, tree->n);
    c->h_ssq = -1;
    if (fused_norm_ok(c, tree->n)) {
        prenorm_into_h(c, w->rms1, tree->n);
        if ((s = layer_body_fused(c, w, kv, tree, nullptr)) != GHD_OK) return s;
        launch_store_x(c, x_out, tree->n);
        return check_cuda(c, "verify_layer");
    }
    if ((s = layer_body(c, w, kv, tree)) != GHD_OK) return s;
    if (c->pending.active) launch_fold_pending(c, tree->n, nullptr, nullptr, x_out);
    else launch_store_x(c, x_out, tree->n);
    return check_cuda(c, "verify_layer");
}

ghd_status ghd_verify_step(ghd_ctx* c, const ghd_model_weights* w, ghd_kv_layer* kv, const ghd_tree* tree,
                           const int32_t* tokens_dev, float* logits_dev, int32_t* argmax_dev) {
    if (!c || !w || !kv || !tokens_dev || !argmax_dev) return GHD_EINVAL;
    if (!c->ws) return fail(c, GHD_ENOSPACE, "no workspace set");
    if (!w->embed || !w->rms_final || !w->lm_head || (c->cfg.n_layers > 0 && !w->layers))
        return fail(c, GHD_EINVAL, "step: null weight pointer");
    ghd_status s = check_tree(c, tree);
    if (s != GHD_OK) return s;
    for (int l = 0; l < c->cfg.n_layers; ++l) {
        const ghd_layer_weights& lw = w->layers[l];
        if (!lw.wqkv || !lw.wo || !lw.w_gate_up || !lw.w_down || !lw.rms1 || !lw.rms2 || !kv[l].k || !kv[l].v)
            return fail(c, GHD_EINVAL, "step: null layer weight or cache pointer");
        if (kv[l].len != tree->kv_len) return fail(c, GHD_EINVAL, "step: kv.len differs from tree.kv_len");
    }
    float* logits = logits_dev ? logits_dev : c->logits;
    c->pending.active = 0;
    c->entry_fresh = c->opt_chain_calls ? 0 : 1;
    if (c->opt_graph != 2) {
        if ((s = step_body(c, w, kv, tree, tokens_dev, logits, argmax_dev)) != GHD_OK) return s;
        return check_cuda(c, "verify_step");
    }
    // Graph replay: the key is every value the enqueued kernels depend on.
    std::vector<uint64_t> key;
    auto push = [&](const void* p) { key.push_back((uint64_t)(uintptr_t)p); };
    push(w->embed); push(w->rms_final); push(w->lm_head); push(tokens_dev); push(logits); push(argmax_dev);
    push(tree->mask); push(tree->depth); push(tree->pos); push(tree->rope); push(tree->coo_ptr); push(tree->coo_col);
    key.push_back(((uint64_t)(uint32_t)tree->n << 32) | (uint32_t)tree->kv_len);
    for (int o : {c->opt_gemm_path, c->opt_attn_splits, c->opt_attn_path, c->opt_gemm_ctas, c->opt_gemm_burst, c->opt_no_pdl, c->opt_gemm_stages, c->opt_gemm_epi, c->opt_attn_sparse, c->opt_chain_calls, c->opt_fused_norm, c->opt_gemm_pair, c->opt_attn_rows, c->opt_gemm_skew, c->opt_attn_small})
        key.push_back((uint64_t)(uint32_t)o);       // every option that changes what is enqueued
    for (int l = 0; l < c->cfg.n_layers; ++l) {
        const ghd_layer_weights& lw = w->layers[l];
        push(lw.wqkv); push(lw.wo); push(lw.w_gate_up); push(lw.w_down); push(lw.rms1); push(lw.rms2);
        push(kv[l].k); push(kv[l].v);
    }
    for (StepGraph* g : *c->graphs)
        if (g->key == key) {
            if (cudaGraphLaunch(g->exec, c->stream) != cudaSuccess) return check_cuda(c, "graph launch");
            c->launches += g->kernels;
            return GHD_OK;
        }
    // The caller's stream may be the legacy default stream, which cannot be captured:
    // record the kernels on a stream of our own (nothing executes there) and replay
    // the instantiated graph on the caller's stream.
    const int64_t before = c->launches;
    if (!c->cap_stream && cudaStreamCreateWithFlags(&c->cap_stream, cudaStreamNonBlocking) != cudaSuccess)
        return check_cuda(c, "capture stream");
    if (cudaStreamBeginCapture(c->cap_stream, cudaStreamCaptureModeThreadLocal) != cudaSuccess) return check_cuda(c, "begin capture");
    c->cur = c->cap_stream;
    s = step_body(c, w, kv, tree, tokens_dev, logits, argmax_dev);
    c->cur = c->stream;
    cudaGraph_t graph = nullptr;
    const cudaError_t ce = cudaStreamEndCapture(c->cap_stream, &graph);
    if (s != GHD_OK) { if (graph) cudaGraphDestroy(graph); c->launches = before; return s; }
    if (ce != cudaSuccess || !graph) { c->launches = before; cudaGetLastError(); return fail(c, GHD_ECUDA, "stream capture failed"); }
    cudaGraphExec_t exec = nullptr;
    if (cudaGraphInstantiate(&exec, graph, 0) != cudaSuccess) { cudaGraphDestroy(graph); c->launches = before; return check_cuda(c, "graph instantiate"); }
    cudaGraphDestroy(graph);
    StepGraph* g = new StepGraph{key, exec, c->launches - before};
    if (c->graphs->size() >= 8) { cudaGraphExecDestroy(c->graphs->front()->exec); delete c->graphs->front(); c->graphs->erase(c->graphs->begin()); }
    c->graphs->push_back(g);
    if (cudaGraphLaunch(exec, c->stream) != cudaSuccess) return check_cuda(c, "graph launch");
    return GHD_OK;
}

ghd_status ghd_copy_hidden(ghd_ctx* c, int32_t n, float* dst_dev) {
    if (!c || !dst_dev || n < 1 || n > c->cfg.max_nodes) return GHD_EINVAL;
    if (!c->ws) return fail(c, GHD_ENOSPACE, "no workspace set");
    if (cudaMemcpyAsync(dst_dev, c->xres, sizeof(float) * (size_t)n * c->cfg.d_model, cudaMemcpyDeviceToDevice, c->stream) != cudaSuccess)
        return check_cuda(c, "copy_hidden");
    return GHD_OK;
}

ghd_status ghd_accept(ghd_ctx* c, const ghd_tree* tree, const int32_t* tokens_dev, const int32_t* argmax_dev,
                      ghd_accept_result* out_dev) {
    if (!c || !tokens_dev || !argmax_dev || !out_dev) return GHD_EINVAL;
    ghd_status s = check_tree(c, tree);
    if (s != GHD_OK) return s;
    if (!tree->has_parent || !tree->parent) return fail(c, GHD_EINVAL, "accept: tree has no parent array");
    launch_accept(c, tree, tokens_dev, argmax_dev, out_dev);
    return check_cuda(c, "accept");
}

ghd_status ghd_kv_len_set(ghd_ctx* c, int32_t kv_len) {
    if (!c) return GHD_EINVAL;
    if (!c->ws) return fail(c, GHD_ENOSPACE, "no workspace set");
    if (kv_len < 0 || kv_len >= c->cfg.max_kv_len) return fail(c, GHD_ENOSPACE, "kv_len_set: kv_len outside the cache");
    launch_kv_len_set(c, kv_len);
    return check_cuda(c, "kv_len_set");
}

ghd_status ghd_kv_len_get(ghd_ctx* c, int32_t* kv_len_host) {
    if (!c || !kv_len_host) return GHD_EINVAL;
    if (!c->ws) return fail(c, GHD_ENOSPACE, "no workspace set");
    if (cudaStreamSynchronize(c->stream) != cudaSuccess) return check_cuda(c, "stream synchronize");
    if (cudaMemcpy(kv_len_host, c->kv_len_word, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return check_cuda(c, "kv_len read");
    return GHD_OK;
}

ghd_status ghd_kv_commit(ghd_ctx* c, const ghd_kv_layer* kv, int32_t n_layers, int32_t kv_len, const ghd_accept_result* result_dev) {
    if (!c || !kv || !result_dev || n_layers < 1) return GHD_EINVAL;
    if (kv_len == GHD_KV_LEN_DEVICE && !c->ws) return fail(c, GHD_ENOSPACE, "no workspace set");
    if (kv_len != GHD_KV_LEN_DEVICE && (kv_len < 0 || kv_len + 1 > c->cfg.max_kv_len)) return fail(c, GHD_ENOSPACE, "kv_commit: kv_len outside the cache");
    for (int l = 0; l < n_layers; ++l)
        if (!kv[l].k || !kv[l].v) return fail(c, GHD_EINVAL, "kv_commit: null cache pointer");
    launch_kv_commit(c, kv, n_layers, kv_len, result_dev);
    return check_cuda(c, "kv_commit");
}

ghd_status ghd_medusa_draft(ghd_ctx* c, const ghd_medusa_weights* w, const ghd_accept_result* result_dev, const int32_t* topk_host,
                            int32_t* cand_dev, float* logits_dev) {
    if (!c || !w || !w->w1 || !w->w2 || !result_dev || !topk_host || !cand_dev) return GHD_EINVAL;
    if (!c->ws) return fail(c, GHD_ENOSPACE, "no workspace set");
    if (w->n_heads < 1 || w->n_heads > GHD_MAX_DRAFT_HEADS) return fail(c, GHD_EINVAL, "medusa: n_heads outside [1, 8]");
    for (int k = 0; k < w->n_heads; ++k)
        if (topk_host[k] < 1 || topk_host[k] > GHD_MAX_TOPK || topk_host[k] > c->cfg.vocab) return fail(c, GHD_EINVAL, "medusa: top-k outside [1, 16]");
    const ghd_model_cfg& m = c->cfg;
    const int d = m.d_model, K = w->n_heads;
    const size_t es = m.dtype == GHD_F32 ? 4 : 2;
    if ((size_t)K * d > (size_t)m.max_nodes * ((3 * d > 2 * m.d_ffn) ? 3 * d : 2 * m.d_ffn) || (size_t)K * d > (size_t)m.max_nodes * m.d_ffn)
        return fail(c, GHD_ENOSPACE, "medusa: workspace too small for the heads' activations");
    float* logits = logits_dev ? logits_dev : c->mlogits;
    c->pending.active = 0;
    c->entry_fresh = c->opt_chain_calls ? 0 : 1;
    launch_medusa_gather(c, result_dev, c->attnbuf, c->h_ssq >= 0 ? c->ssq[c->h_ssq] : nullptr, c->h_ssq >= 0 ? c->ssq_tiles[c->h_ssq] : 0);
    EpiArgs e{};
    e.mode = EPI_RAW; e.out_f32 = c->raw;
    ghd_status s = project(c, c->attnbuf, w->w1, 1, d, K * d, e, nullptr, nullptr);      // all heads' W1 rows in one projection
    if (s != GHD_OK) return s;
    launch_medusa_res(c, c->attnbuf, c->raw, K, c->ubuf);
    for (int k = 0; k < K; ++k) {
        e.out_f32 = logits + (size_t)k * m.vocab;
        s = project(c, (const char*)c->ubuf + (size_t)k * d * es, (const char*)w->w2 + (size_t)k * m.vocab * d * es, 1, d, m.vocab, e, nullptr, nullptr);
        if (s != GHD_OK) return s;
    }
    launch_medusa_topk(c, logits, K, m.vocab, topk_host, cand_dev);
    return check_cuda(c, "medusa_draft");
}

ghd_status ghd_tree_fill_tokens(ghd_ctx* c, const int32_t* cand_dev, const ghd_accept_result* result_dev, const int32_t* level_dev,
                                const int32_t* rank_dev, int32_t n, int32_t* tokens_dev) {
    if (!c || !cand_dev || !result_dev || !level_dev || !rank_dev || !tokens_dev) return GHD_EINVAL;
    if (n < 1 || n > c->cfg.max_nodes) return fail(c, GHD_ETREE, "tree_fill: n outside [1, max_nodes]");
    launch_tree_fill(c, cand_dev, result_dev, level_dev, rank_dev, n, tokens_dev);
    return check_cuda(c, "tree_fill_tokens");
}

ghd_status ghd_linear(ghd_ctx* c, const void* x, const void* w, int32_t n, int32_t k, int32_t m, float* y) {
    if (!c || !x || !w || !y || n < 1 || k < 1 || m < 1) return GHD_EINVAL;
    if (n > c->cfg.max_nodes) return fail(c, GHD_ENOSPACE, "linear: n > max_nodes");
    if (k % 8) return fail(c, GHD_ESHAPE, "linear: k must be a multiple of 8");
    if (!c->ws) return fail(c, GHD_ENOSPACE, "no workspace set");
    EpiArgs e{};
    e.mode = EPI_RAW; e.out_f32 = y;
    c->entry_fresh = c->opt_chain_calls ? 0 : 1;
    ghd_status s = project(c, x, w, n, k, m, e, nullptr, nullptr);
    return s != GHD_OK ? s : check_cuda(c, "linear");
}

ghd_status ghd_gate_up(ghd_ctx* c, const void* h, const void* w_gate_up, int32_t n, void* u) {
    if (!c || !h || !w_gate_up || !u || n < 1) return GHD_EINVAL;
    if (n > c->cfg.max_nodes) return fail(c, GHD_ENOSPACE, "gate_up: n > max_nodes");
    if (!c->ws) return fail(c, GHD_ENOSPACE, "no workspace set");
    EpiArgs e{};
    e.mode = EPI_SWIGLU; e.out_t = u;
    c->entry_fresh = c->opt_chain_calls ? 0 : 1;
    void* keep = c->ubuf;
    c->ubuf = u;                     // the CUDA-core path writes its SwiGLU output through the context's buffer pointer
    const ghd_status s = project(c, h, w_gate_up, n, c->cfg.d_model, 2 * c->cfg.d_ffn, e, nullptr, nullptr);
    c->ubuf = keep;
    return s != GHD_OK ? s : check_cuda(c, "gate_up");
}

ghd_status ghd_rmsnorm(ghd_ctx* c, const float* x, const void* g, int32_t n, void* out) {
    if (!c || !x || !g || !out || n < 1) return GHD_EINVAL;
    c->entry_fresh = c->opt_chain_calls ? 0 : 1;
    launch_rmsnorm(c, x, g, n, out);
    return check_cuda(c, "rmsnorm");
}

ghd_status ghd_tree_attention(ghd_ctx* c, const void* q, const ghd_kv_layer* kv, const ghd_tree* tree, void* out) {
    if (!c || !q || !kv || !kv->k || !kv->v || !out) return GHD_EINVAL;
    if (!c->ws) return fail(c, GHD_ENOSPACE, "no workspace set");
    ghd_status s = check_tree(c, tree);
    if (s != GHD_OK) return s;
    c->entry_fresh = c->opt_chain_calls ? 0 : 1;
    if ((s = attention(c, q, kv, tree, out)) != GHD_OK) return s;
    return check_cuda(c, "tree_attention");
}

ghd_status ghd_argmax(ghd_ctx* c, const float* logits, int32_t n, int32_t v, int32_t* out) {
    if (!c || !logits || !out || n < 1 || v < 1) return GHD_EINVAL;
    c->entry_fresh = c->opt_chain_calls ? 0 : 1;
    launch_argmax(c, logits, n, v, out);
    return check_cuda(c, "argmax");
}

ghd_status ghd_sync_status(ghd_ctx* c) {
    if (!c) return GHD_EINVAL;
    if (cudaStreamSynchronize(c->stream) != cudaSuccess) return check_cuda(c, "stream synchronize");
    if (!c->ws) return GHD_OK;
    int st = 0;
    if (cudaMemcpy(&st, c->status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return check_cuda(c, "status read");
    if (st == DEV_KV_RANGE) {
        snprintf(c->err, sizeof(c->err), "the cache length on the device left [0, max_kv_len - n]");
        cudaMemset(c->status, 0, sizeof(int));
        return GHD_ENOSPACE;
    }
    if (st != DEV_OK) {
        snprintf(c->err, sizeof(c->err), "device wait expired (code %d)", st);
        int keep = 0;                                          // the cache length survives the clean-up
        cudaMemcpy(&keep, c->kv_len_word, sizeof(int), cudaMemcpyDeviceToHost);
        cudaMemset(c->status, 0, 256 + sizeof(int) * 4096);   // status word and tile arrival counters
        cudaMemcpy(c->kv_len_word, &keep, sizeof(int), cudaMemcpyHostToDevice);
        return GHD_ETIMEOUT;
    }
    return GHD_OK;
}

const char* ghd_status_str(ghd_status s) {
    switch (s) {
        case GHD_OK: return "ok";
        case GHD_EINVAL: return "invalid argument";
        case GHD_ESHAPE: return "unsupported model shape";
        case GHD_ETREE: return "invalid tree";
        case GHD_ENOSPACE: return "not enough space";
        case GHD_ECUDA: return "CUDA error";
        case GHD_ETIMEOUT: return "device wait timed out";
        case GHD_EUNSUPPORTED: return "unsupported";
    }
    return "unknown";
}

const char* ghd_last_error(const ghd_ctx* c) { return c ? c->err : ""; }
int64_t ghd_launch_count(const ghd_ctx* c) { return c ? c->launches : 0; }
int64_t ghd_path_count(const ghd_ctx* c, int32_t path) { return (c && path >= 0 && path < 8) ? c->path_count[path] : 0; }

}  // extern "C"
