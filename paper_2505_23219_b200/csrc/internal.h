// Internal declarations shared by the translation units of libghd.
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <map>
#include <tuple>
#include <utility>
#include <vector>

#include "ghd.h"

namespace ghd {

// Device status word values (first failure wins).
enum : int { DEV_OK = 0, DEV_TIMEOUT_TMA = 1, DEV_TIMEOUT_MMA = 2, DEV_TIMEOUT_EPI = 3, DEV_TIMEOUT_TMEM = 4, DEV_TIMEOUT_GRID = 5, DEV_KV_RANGE = 6 };

// Epilogues of the projection GEMMs.
enum Epilogue : int {
    EPI_RAW = 0,      // out float [n][m] = acc
    EPI_ROPE_KV = 1,  // q rotated -> q buffer; k rotated, v -> cache rows kv_len + i
    EPI_RESID = 2,    // xres[n][m] += acc (float residual stream)
    EPI_SWIGLU = 3,   // u T [n][m/2] = SiLU(gate) * up, weight rows [gate | up]
    EPI_DEFER = 4,    // partial tiles only; the next kernel adds them to the residual stream
    EPI_RESID_NORM = 5,   // xres += acc; xg T [n][m] = xres * gain (not yet divided by the rms); per-tile sums of squares
};

constexpr int SSQ_PITCH = GHD_MAX_NODES;   // floats per 128-feature tile in a sum-of-squares buffer
constexpr int SSQ_MAX_TILES = 64;

struct EpiArgs {
    int mode;
    float* out_f32;       // EPI_RAW target / EPI_RESID residual stream (in place)
    void* out_t;          // EPI_ROPE_KV: q buffer T [n][d]; EPI_SWIGLU: u T [n][f]
    void* k_cache;        // EPI_ROPE_KV
    void* v_cache;
    const float* rope;    // [n][d_head] cos/sin pairs
    int kv_len, max_kv_len, d_head, d_model;
    const int* kv_len_dev;    // non-null: the cache length comes from this device word instead of kv_len
    // Column scale: the input rows are gain-weighted but not yet normalised; node i's result is multiplied by
    // 1 / sqrt(sum_t ssq_in[t][i] / k + eps) before the epilogue proper (nullptr: no scale).
    const float* ssq_in;
    int ssq_in_tiles;
    float rms_eps;
    // EPI_RESID_NORM (out_f32 = residual stream): gain T [m] of the NEXT norm, xg_out T [n][m], ssq_out [m/128][SSQ_PITCH]
    const void* gain;
    void* xg_out;
    float* ssq_out;
};

struct TmapKey {
    const void* ptr; uint64_t rows, cols, planes, plane_stride; uint32_t box_rows, box_cols;
    bool operator<(const TmapKey& o) const {
        return std::tie(ptr, rows, cols, planes, plane_stride, box_rows, box_cols) <
               std::tie(o.ptr, o.rows, o.cols, o.planes, o.plane_stride, o.box_rows, o.box_cols);
    }
};

struct StepGraph;

// Partial tiles left behind by a projection in EPI_DEFER mode: CTA c holds k-steps
// [total*c/ctas, total*(c+1)/ctas) of the flattened (tile, k-step) space; its first unit is in
// slot 0, its second (if any) in slot 1, each slot [columns][128 rows] float.
struct PendingPartials {
    int active, kiters, ctas, m;
    int stride;       // CTA distance between two contributors of a tile (2 when CTA pairs ran the projection)
    long long total;
    size_t slot_elems;
    // per 128-row tile, worked out on the host (integer divisions are expensive on the device):
    // first contributing CTA, number of contributors, and the slot of the first one (later ones use slot 0)
    unsigned short first_cta[128];
    unsigned char n_contrib[128], first_slot[128];
};

}  // namespace ghd

struct ghd_ctx {
    ghd_model_cfg cfg;
    cudaStream_t stream;      // the caller's stream
    cudaStream_t cur;         // where launches go: `stream`, or `cap_stream` while a graph is being captured
    cudaStream_t cap_stream;  // library-owned stream used only for graph capture (nothing ever runs on it)
    int device, sm_count;
    // options
    int opt_gemm_path, opt_attn_splits, opt_attn_path, opt_graph, opt_gemm_ctas, opt_gemm_burst, opt_no_pdl, opt_gemm_stages, opt_gemm_epi, opt_attn_sparse, opt_chain_calls, opt_fused_norm, opt_gemm_pair, opt_attn_rows, opt_gemm_skew, opt_attn_small;
    // workspace carve (all device pointers into the caller's buffer)
    char* ws;
    size_t ws_bytes;
    float* xres;      // [max_nodes][d_model] residual stream
    void* hbuf;       // T [max_nodes][d_model] normalised activations
    void* qbuf;       // T [max_nodes][d_model] rotated queries
    void* attnbuf;    // T [max_nodes][d_model] attention output
    void* ubuf;       // T [max_nodes][d_ffn]
    float* raw;       // float [max_nodes][max(3 d_model, 2 d_ffn)] un-fused GEMM output
    float* att_o;     // float [splits][max_nodes][d_model] attention partial numerators
    float* att_ml;    // float [splits][max_nodes][n_heads][2] running max / sum
    float* gemm_part; // float [ctas][2][256][128] split tile partial sums
    int* counters;    // int [tiles] arrival counters (zero between launches)
    float* ssq[2];    // float [SSQ_MAX_TILES][SSQ_PITCH] per-tile sums of squares of the residual stream (two, used in turn)
    int ssq_tiles[2]; // tiles that hold data in each
    int h_ssq;        // which of them describes hbuf (-1: hbuf is already normalised)
    float* logits;    // float [max_nodes][vocab]
    float* mlogits;   // float [8][vocab] logits of the drafting heads
    int* status;      // device status word
    int* kv_len_word; // device word with the cache length (calls given GHD_KV_LEN_DEVICE read it)
    int kv_len_hint;  // what the host last wrote there: sizes launches whose grid depends on the length
    int max_splits;
    ghd::PendingPartials pending;   // projection output not yet folded into xres
    // bookkeeping
    int entry_fresh;          // 1 until the first launch of a public call: that launch is fully serialised (see launch_k)
    bool attr_gemm, attr_attn, attr_attn_small;  // dynamic shared memory limits raised on this context's device
    int64_t launches;
    int64_t path_count[8];   // launches per kernel family (ghd_path)
    char err[256];
    std::map<ghd::TmapKey, std::vector<uint64_t>>* tmaps;   // cached tensor maps (128-byte blobs)
    std::vector<ghd::StepGraph*>* graphs;
};

namespace ghd {

// Programmatic dependent launch.  A kernel launched with `pdl` may start while its predecessor in
// the stream is still running; it must call pdl_wait() before it touches anything another kernel
// writes or reads-then-overwrites (only constant weights and its own on-chip set-up may come
// earlier), and calls pdl_trigger() once its blocks hold the resources later kernels could compete for.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
// Cache length of a call: the host's value, or (dev != nullptr) the context's device word, clamped so that the
// rows kv_len .. kv_len + n - 1 stay inside the cache whatever the word holds.
__device__ __forceinline__ int resolve_kv_len(int host, const int* dev, int max_kv_len, int n) {
    if (!dev) return host;
    int v = __ldcg(dev);
    if (v > max_kv_len - n) v = max_kv_len - n;
    return v < 0 ? 0 : v;
}
#endif

// cluster_x > 1: the CTAs of a grid row (gridDim.x a multiple of cluster_x) are launched as thread-block clusters.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kc(ghd_ctx* c, bool pdl, int cluster_x, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = c->cur;
    cudaLaunchAttribute attr[2];
    int na = 0;
    if (cluster_x > 1) {
        attr[na].id = cudaLaunchAttributeClusterDimension;
        attr[na].val.clusterDim.x = (unsigned)cluster_x;
        attr[na].val.clusterDim.y = 1;
        attr[na].val.clusterDim.z = 1;
        ++na;
    }
    // The first kernel of a public call is never launched programmatically: what ran before it on the
    // stream belongs to the caller and may still be writing weights or cache rows that our kernels read
    // ahead of their dependency wait.
    if (pdl && !c->opt_no_pdl && !c->entry_fresh) {
        attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[na].val.programmaticStreamSerializationAllowed = 1;
        ++na;
    }
    cfg.attrs = attr;
    cfg.numAttrs = na;
    c->entry_fresh = 0;
    c->launches++;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

template <typename... KArgs, typename... Args>
inline cudaError_t launch_k(ghd_ctx* c, bool pdl, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, Args&&... args) {
    return launch_kc(c, pdl, 1, kernel, grid, block, smem, std::forward<Args>(args)...);
}

size_t carve_workspace(ghd_ctx* c, char* base);   // returns bytes needed; assigns pointers when base != nullptr

// kernels_small.cu
void launch_tree_build(ghd_ctx* c, const int32_t* parent_host, ghd_tree* t);
void launch_tree_from_mask(ghd_ctx* c, ghd_tree* t, bool have_depth, const uint64_t* mask_host);   // mask/depth already copied
void launch_load_x(ghd_ctx* c, const void* x_in, int n);     // T [n][d] -> xres
void launch_store_x(ghd_ctx* c, void* x_out, int n);         // xres -> T [n][d]
void launch_embed(ghd_ctx* c, const void* embed, const int32_t* tokens, int n);
void launch_rmsnorm(ghd_ctx* c, const float* x, const void* g, int n, void* out);
// xg T [n][d] = xres * g (not normalised), ssq[0][node] = sum of squares of the row
void launch_prenorm(ghd_ctx* c, const void* g, int n, void* xg, float* ssq);
// xres += sum of the pending partial tiles; then optionally h = RMSNorm(xres) * g and/or x_out = T(xres)
void launch_fold_pending(ghd_ctx* c, int n, const void* g, void* h_out, void* x_out);
void launch_rope_append(ghd_ctx* c, const float* qkv_raw, const ghd_tree* t, const ghd_kv_layer* kv);
void launch_swiglu(ghd_ctx* c, const float* gu_raw, int n);
void launch_residual(ghd_ctx* c, const float* proj_raw, int n);
void launch_argmax(ghd_ctx* c, const float* logits, int n, int v, int32_t* out);
void launch_accept(ghd_ctx* c, const ghd_tree* t, const int32_t* tokens, const int32_t* amax, ghd_accept_result* out);
// drafting heads (kernels_small.cu)
// h_sel T [d] = hbuf[last accepted node], divided by the row's rms when hbuf is not yet normalised (ssq != nullptr)
void launch_medusa_gather(ghd_ctx* c, const ghd_accept_result* res, void* h_sel, const float* ssq, int ssq_tiles);
void launch_medusa_res(ghd_ctx* c, const void* h_sel, const float* raw, int heads, void* y);        // y T [heads][d] = h + SiLU(raw)
void launch_medusa_topk(ghd_ctx* c, const float* logits, int heads, int vocab, const int* topk, int32_t* cand);
void launch_tree_fill(ghd_ctx* c, const int32_t* cand, const ghd_accept_result* res, const int32_t* level, const int32_t* rank, int n, int32_t* tokens);
// kv_len < 0: rows relative to the device word, which a second kernel then advances by n_matched + 1
void launch_kv_commit(ghd_ctx* c, const ghd_kv_layer* kv, int n_layers, int kv_len, const ghd_accept_result* res);
void launch_kv_len_set(ghd_ctx* c, int kv_len);
// the device word when the tree's length is GHD_KV_LEN_DEVICE, else nullptr
inline const int* kv_len_dev_of(const ghd_ctx* c, const ghd_tree* t) { return t->kv_len < 0 ? c->kv_len_word : nullptr; }
// the length launch geometry is sized for
inline int kv_len_host_of(const ghd_ctx* c, const ghd_tree* t) { return t->kv_len < 0 ? c->kv_len_hint : t->kv_len; }

// gemm_simt.cu : y float [n][m] = x T [n][k] * w T [m][k]^T
void launch_gemm_simt(ghd_ctx* c, const void* x, const void* w, int n, int k, int m, float* y);

// attn_simt.cu : split-KV tree attention + combine
void launch_attn_simt(ghd_ctx* c, const void* q, const ghd_kv_layer* kv, const ghd_tree* t, void* out, bool coo);
// The sparse part from the coordinate index: every query gathers the new keys/values it sees; the result
// goes to partial slot `slot` of att_o / att_ml (natural-log maxima), to be merged with the cache splits.
void launch_attn_coo(ghd_ctx* c, const void* q, const ghd_kv_layer* kv, const ghd_tree* t, int slot);
int attn_auto_splits(const ghd_ctx* c, int n, int kv_total);

void launch_attn_combine(ghd_ctx* c, void* out, int splits, int n);   // merges att_o / att_ml into out

// attn_tc.cu : tcgen05 / TMA tree attention (GHD_F16 only)
bool attn_tc_supported(const ghd_ctx* c, const ghd_tree* t);
// the split partials go to att_o / att_ml and a second kernel merges them into `out`
// coo: the new rows are handled by launch_attn_coo (one more partial), this kernel takes the cache only
ghd_status launch_attn_tc(ghd_ctx* c, const void* q, const ghd_kv_layer* kv, const ghd_tree* t, void* out, bool coo);
// attn_tc_small.cu : the split kernel for trees of up to 64 nodes (128-key units, accumulator resident in tensor
// memory); leaves the partials in att_o / att_ml and returns the number of splits (0 and *st after an error)
int launch_attn_tc_small(ghd_ctx* c, const void* q, const ghd_kv_layer* kv, const ghd_tree* t, bool coo, ghd_status* st);

// gemm_tc.cu : tcgen05 / TMA path (GHD_F16 only)
ghd_status launch_gemm_tc(ghd_ctx* c, const void* x, const void* w, int n, int k, int m, const EpiArgs& epi);
bool gemm_tc_supported(const ghd_ctx* c, int n, int k, int m, int epi_mode);

}  // namespace ghd
