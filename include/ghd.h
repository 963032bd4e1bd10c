/*
 * ghd - tree-verification step of speculative decoding on one GPU (sm_100a).
 *
 * The operation (paper Sec. II-C, "Predict-then-Verify"): a tree of N drafted
 * token nodes (node 0 = the root, parent[i] < i) sits on top of a KV cache of
 * length L.  One forward of the decoder stack is run for all N nodes at once;
 * node i attends to the whole cache plus only its own root-to-i ancestors
 * (Sec. II-C, Fig. 3: attention between two drafted nodes is needed only
 * along a root path); the row argmax of the logits then decides which
 * drafted tokens are accepted (the longest validated prefix).
 *
 * Conventions
 *   - "dev" pointers are device memory on the context's GPU, "host" pointers
 *     are ordinary host memory.  The library never allocates or frees device
 *     memory: every buffer, the workspace included, belongs to the caller and
 *     must stay alive until the work enqueued on the stream has finished.
 *   - All calls enqueue work on the stream given to ghd_create and return
 *     without synchronising, except ghd_sync_status.
 *   - Every call returns a ghd_status.  Arguments are validated on the host
 *     before anything is launched; a failing call launches nothing.
 *   - Storage type T is float (GHD_F32) or IEEE half (GHD_F16, accumulation in
 *     float).  Matrices are row-major; weights are stored [out][in].
 *   - One context per stream; a context is not thread-safe.
 */
#ifndef GHD_H_
#define GHD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define GHD_MAX_NODES 256

typedef enum ghd_status {
    GHD_OK = 0,
    GHD_EINVAL = 1,       /* null pointer or bad scalar argument                     */
    GHD_ESHAPE = 2,       /* model shape the kernels do not cover                    */
    GHD_ETREE = 3,        /* parent array / mask is not a valid tree description     */
    GHD_ENOSPACE = 4,     /* kv_len + n > max_kv_len, or workspace too small         */
    GHD_ECUDA = 5,        /* a CUDA runtime/driver call failed                       */
    GHD_ETIMEOUT = 6,     /* a bounded device-side wait gave up (see ghd_sync_status) */
    GHD_EUNSUPPORTED = 7
} ghd_status;

typedef enum ghd_dtype { GHD_F32 = 0, GHD_F16 = 1 } ghd_dtype;

/* Knobs for tests and sweeps (ghd_set_option).  0 always means "automatic". */
typedef enum ghd_option {
    GHD_OPT_GEMM_PATH = 0,    /* 0 auto, 1 SIMT kernels, 2 tcgen05 kernels (GHD_F16 only)   */
    GHD_OPT_ATTN_SPLITS = 1,  /* number of KV splits of the attention (>= 1), 0 auto         */
    GHD_OPT_ATTN_PATH = 2,    /* 0 auto, 1 SIMT kernel, 2 tcgen05 kernel (GHD_F16 only)      */
    GHD_OPT_GRAPH = 3,        /* ghd_verify_step: 0/1 = launch kernels directly, 2 = replay a
                                 CUDA graph captured on first use for the same arguments    */
    GHD_OPT_GEMM_CTAS = 4,    /* CTAs of the tcgen05 GEMM (0 = one per SM)                   */
    GHD_OPT_GEMM_BURST = 5,   /* k-steps whose weight loads the tcgen05 GEMM issues together  */
    GHD_OPT_NO_PDL = 6,       /* 1 = launch every kernel fully serialised (no programmatic
                                 dependent launch overlap between consecutive kernels)        */
    GHD_OPT_GEMM_STAGES = 7,  /* pipeline stages of the tcgen05 GEMM (0 = automatic)          */
    GHD_OPT_GEMM_EPI = 8,     /* epilogue warp groups of the tcgen05 GEMM: 0 auto, 1, 2        */
    GHD_OPT_CHAIN_CALLS = 10, /* 1 = the caller promises that whatever runs before a call on the stream does not
                                 write anything the call reads ahead of its dependency wait (weights, cache
                                 rows below kv_len): the first kernel of every call may then start while
                                 its predecessor drains, like the kernels inside a call do (0 = it waits)  */
    GHD_OPT_FUSED_NORM = 11,  /* tcgen05 path: 1 = the RMSNorms live in the projections' epilogues (the projection into
                                 the residual stream leaves gain-weighted rows and per-tile sums of squares, its
                                 consumer multiplies by 1 / rms); 0 = separate reduction + norm kernels (default:
                                 faster as measured, the split tiles of the narrow projections finish in parallel)  */
    GHD_OPT_GEMM_PAIR = 12,   /* tcgen05 GEMM on clusters of two CTAs (cta_group::2: a pair shares the activation slab of
                                 two neighbouring weight tiles, each CTA loading half of it): 0 = for trees of more
                                 than 128 nodes, 1 = never, 2 = whenever the shape allows (even tile count)          */
    GHD_OPT_ATTN_ROWS = 13,   /* tcgen05 attention, trees of more than 64 nodes: 0 = two softmax threads per query row
                                 (two groups of four warps on the same tensor-memory lanes), 1 = one thread per row     */
    GHD_OPT_GEMM_SKEW = 14,   /* tcgen05 GEMM with three CTAs per two tiles: k-chunks taken from the middle CTA of every
                                 group (0 = automatic, 1 = none, s + 1 = s chunks), so that it is done before its neighbours */
    GHD_OPT_ATTN_SMALL = 15,  /* tcgen05 attention: the kernel with 128-key units, four softmax threads per query row and
                                 the output accumulator resident in tensor memory: 0 = over a cache of at least 1024 rows
                                 (where it measured faster), 1 = always, 2 = never (64-key units, k_attn_tc)        */
    GHD_OPT_ATTN_SPARSE = 9   /* how the attention handles the new (drafted) keys, the sparse part of
                                 Sec. III-B-3: 0 = packed ancestor bitmask, 64-node groups skipped when
                                 nobody sees them (default); 1 = per-query list of visible nodes (the
                                 COO index): each query gathers only the keys it sees                */
} ghd_option;

/* LLaMA-style decoder (paper Sec. IV-A: Vicuna-7B / LLaMA-7B): RMSNorm, rotary
 * embedding (rotate-half pairing), SwiGLU MLP, no biases, n_kv_heads == n_heads. */
typedef struct ghd_model_cfg {
    int32_t d_model, n_heads, n_kv_heads, d_head, d_ffn, vocab, n_layers;
    int32_t max_kv_len;   /* rows of every K/V cache                              */
    int32_t max_nodes;    /* largest tree, <= GHD_MAX_NODES                        */
    int32_t dtype;        /* ghd_dtype of weights, caches, activations             */
    float rms_eps;
    float rope_theta;
} ghd_model_cfg;

/* dev pointers, storage type T.  wqkv [3*d_model][d_model] (q rows, then k, then v),
 * wo [d_model][d_model], w_gate_up [2*d_ffn][d_model] (gate rows, then up rows),
 * w_down [d_model][d_ffn], rms1/rms2 [d_model]. */
typedef struct ghd_layer_weights {
    const void *wqkv, *wo, *w_gate_up, *w_down, *rms1, *rms2;
} ghd_layer_weights;

typedef struct ghd_model_weights {
    const void *embed;                /* dev T [vocab][d_model]            */
    const ghd_layer_weights *layers;  /* HOST array [n_layers]             */
    const void *rms_final;            /* dev T [d_model]                   */
    const void *lm_head;              /* dev T [vocab][d_model]            */
} ghd_model_weights;

/* One layer's cache (paper Sec. II-A: decode appends the new K/V).  k, v: dev T
 * [n_heads][max_kv_len][d_head]; keys are stored already rotated.  A verify call
 * reads rows [0, len) and writes the N new rows to [len, len + N) in tree order;
 * it does not change len. */
typedef struct ghd_kv_layer {
    void *k, *v;
    int32_t len;
} ghd_kv_layer;

/* A built tree.  The caller fills the five dev pointers with buffers of at least
 * mask: max_nodes * 4 uint64, parent/depth/pos: max_nodes int32,
 * rope: max_nodes * d_head float; ghd_tree_build / ghd_tree_from_mask fill the
 * scalars and enqueue the kernel that fills the buffers.
 *   mask[i * n_words + w] bit b  = 1 iff new node (64 w + b) is visible to node i
 *                                  (ancestor or i itself), LSB first;
 *   depth[i] = edges from the root, pos[i] = kv_len + depth[i] (position id);
 *   rope[i * d_head + 2 t], [.. + 2 t + 1] = cos, sin of pos[i] * theta^(-2 t / d_head).
 * Optional (both NULL, or both given): the same visibility as a sparse index in coordinate order
 * (Sec. III-B-3: the index of the token pairs to verify is generated before the inference),
 *   coo_ptr: int32 [max_nodes + 1], coo_col: int32 [max_nodes * (max_nodes + 1) / 2];
 *   the visible new nodes of query i are coo_col[coo_ptr[i] .. coo_ptr[i + 1]), ascending; nnz = coo_ptr[n].
 * GHD_OPT_ATTN_SPARSE = 1 needs it. */
typedef struct ghd_tree {
    int32_t n, kv_len, n_words, has_parent;       /* kv_len = GHD_KV_LEN_DEVICE: taken from the context's device word */
    uint64_t *mask;
    int32_t *parent, *depth, *pos;
    float *rope;
    int32_t *coo_ptr, *coo_col;
    int32_t nnz;
} ghd_tree;

/* The cache length kept on the device (paper Sec. II-A: every step extends the cache by the tokens it
 * produced; Sec. II-C: by the accepted ones only).  A context owns one int32 device word.  Wherever a call
 * takes a cache length (ghd_tree_build, ghd_tree_from_mask, ghd_kv_layer.len, ghd_kv_commit) the value
 * GHD_KV_LEN_DEVICE means "read the word on the device when the kernel runs": positions, the rows a step
 * appends and the keys the attention walks then follow the word, and ghd_kv_commit advances it by
 * n_matched + 1, so that a loop of draft / verify / accept / commit steps needs no host read between
 * steps (and, with GHD_OPT_GRAPH = 2, replays one graph for every step).  Every kernel clamps the word to
 * [0, max_kv_len - n]; the tree kernels record a word outside that range in the status word
 * (ghd_sync_status -> GHD_ENOSPACE).  In this mode the attention kernels may fetch cache rows past
 * kv_len + n (their weights are exactly zero): every row of the cache buffers must hold finite numbers,
 * e.g. buffers that were zero-filled when they were allocated. */
#define GHD_KV_LEN_DEVICE (-1)

/* dev struct written by ghd_accept.  nodes[0..n_matched] is the accepted root
 * path (nodes[0] = 0); tokens[j] = argmax at nodes[j]; n_emitted = n_matched + 1
 * (the last token is the one the target model adds itself; paper Table I counts
 * n_emitted: width 1 gives acceptance length 1). */
typedef struct ghd_accept_result {
    int32_t n_matched, n_emitted;
    int32_t nodes[GHD_MAX_NODES];
    int32_t tokens[GHD_MAX_NODES];
} ghd_accept_result;

typedef struct ghd_ctx ghd_ctx;

/* Creates a context bound to `cuda_stream` (a cudaStream_t; NULL = default stream)
 * on the current device.  GHD_ESHAPE unless d_model == n_heads * d_head,
 * n_kv_heads == n_heads, d_head in {64, 128}, d_model % 8 == 0, d_ffn % 8 == 0. */
ghd_status ghd_create(const ghd_model_cfg *cfg, void *cuda_stream, ghd_ctx **out);
void ghd_destroy(ghd_ctx *ctx);

/* Bytes of scratch the context needs (for cfg.max_nodes and cfg.max_kv_len). */
size_t ghd_workspace_bytes(const ghd_ctx *ctx);
/* Hands the context its scratch (dev, 256-byte aligned, caller-owned) and enqueues
 * the one-time clearing of the parts that must start at zero. */
ghd_status ghd_set_workspace(ghd_ctx *ctx, void *dev_ptr, size_t bytes);
ghd_status ghd_set_option(ghd_ctx *ctx, int32_t option, int32_t value);

/* Diagnostics (no counterpart in the paper): how many launches so far went to each kernel family,
 * so that a test can tell which path really ran. */
typedef enum ghd_path {
    GHD_PATH_GEMM_TILE = 0,   /* tcgen05 projection, stream-K over 128-row tiles      */
    GHD_PATH_GEMM_SIMT = 1,   /* CUDA-core projection                                 */
    GHD_PATH_ATTN_TC = 2,     /* tcgen05 tree attention                               */
    GHD_PATH_ATTN_SIMT = 3,   /* CUDA-core tree attention                             */
    GHD_PATH_ATTN_COO = 4,    /* sparse part gathered from the coordinate index        */
    GHD_PATH_GEMM_PAIR = 5    /* tcgen05 projection on CTA pairs (counted besides GEMM_TILE) */
} ghd_path;
int64_t ghd_path_count(const ghd_ctx *ctx, int32_t path);

/* Sec. II-C / III-C-1 (verification tree): parent_host[n], parent[0] = -1,
 * 0 <= parent[i] < i.  Fills tree->mask/parent/depth/pos/rope (see ghd_tree).
 * GHD_ETREE on a bad parent array or n outside [1, max_nodes]; GHD_ENOSPACE if
 * kv_len + n > max_kv_len. */
ghd_status ghd_tree_build(ghd_ctx *ctx, const int32_t *parent_host, int32_t n, int32_t kv_len, ghd_tree *tree);

/* Same from an explicit visibility mask (Fig. 3d, lookahead-style patterns):
 * mask_host [n][ceil(n/64)] packed as in ghd_tree; row i must have bit i set and
 * no bit above i.  depth_host (may be NULL) gives depth[i]; NULL means
 * popcount(row i) - 1.  parent_host may be NULL (then ghd_accept is refused). */
ghd_status ghd_tree_from_mask(ghd_ctx *ctx, const uint64_t *mask_host, const int32_t *depth_host,
                              const int32_t *parent_host, int32_t n, int32_t kv_len, ghd_tree *tree);

/* Sec. II-B (one Transformer layer: MHA block then MLP block) for all tree nodes:
 *   h = RMSNorm(x) ; q,k,v = h Wqkv^T ; RoPE(q,k) ; K/V rows -> cache[len + i] ;
 *   o_i = softmax(q_i K_S^T / sqrt(d_head)) V_S over S = cache rows [0,len) plus
 *   visible new rows (Eq. (1) restricted to the tree) ; y = x + o Wo^T ;
 *   z = y + (SiLU(h2 Wg^T) * (h2 Wu^T)) Wd^T with h2 = RMSNorm(y).
 * x_in, x_out: dev T [n][d_model] (may alias).  kv->len must equal tree->kv_len. */
ghd_status ghd_verify_layer(ghd_ctx *ctx, const ghd_layer_weights *w, ghd_kv_layer *kv, const ghd_tree *tree,
                            const void *x_in, void *x_out);

/* The whole verify forward: embedding rows of tokens_dev[n], cfg.n_layers layers
 * (kv[l] is layer l's cache, HOST array), final RMSNorm, lm_head, row argmax
 * (first index among equal maxima).  logits_dev: float [n][vocab] or NULL (then
 * the logits live only in the workspace); argmax_dev: int32 [n]. */
ghd_status ghd_verify_step(ghd_ctx *ctx, const ghd_model_weights *w, ghd_kv_layer *kv, const ghd_tree *tree,
                           const int32_t *tokens_dev, float *logits_dev, int32_t *argmax_dev);

/* The hidden states the last ghd_verify_step of this context produced: the output of the last layer
 * (Sec. II-B: what the layer stack hands to the final norm and the lm_head), float, before the final
 * RMSNorm.  Copies rows [0, n) of width d_model to dst_dev (dev float [n][d_model]) on the context's stream.
 * GHD_EINVAL on a null pointer or n outside [1, max_nodes]; GHD_ENOSPACE without a workspace. */
ghd_status ghd_copy_hidden(ghd_ctx *ctx, int32_t n, float *dst_dev);

/* Greedy acceptance (Sec. II-C: fall back to the longest validated prefix): node
 * c is valid iff every edge (p -> c') on its root path has tokens[c'] == argmax[p];
 * the deepest valid node wins (lowest index among equals).  out_dev: dev struct. */
ghd_status ghd_accept(ghd_ctx *ctx, const ghd_tree *tree, const int32_t *tokens_dev, const int32_t *argmax_dev,
                      ghd_accept_result *out_dev);

/* KV commit: what a step keeps of the rows it appended (paper Sec. II-A: each step extends the KV
 * cache by the tokens it produced; Sec. II-C: only the longest validated prefix survives).
 * For each of the n_layers caches kv[l] (dev pointers, [n_kv_heads][max_kv_len][d_head]) the rows of
 * the accepted path move from slots kv_len + nodes[j] (tree order, where the verify call wrote
 * them) to slots kv_len + j, j = 0 .. n_matched, so that rows [0, kv_len + n_matched + 1) are the
 * cache of the accepted sequence; later rows keep stale tree rows.  `result_dev` is the struct
 * ghd_accept filled (read on the device: no host round trip).  kv[l].len is a host field and is
 * NOT changed: the caller raises it to kv_len + n_matched + 1 once it has read n_matched.
 * With kv_len = GHD_KV_LEN_DEVICE the rows move relative to the context's device word, which is then
 * advanced to word + n_matched + 1 (clamped to max_kv_len - 1) by a kernel enqueued behind the moves.
 * Enqueued on the context's stream.  GHD_EINVAL on null pointers, GHD_ENOSPACE when
 * kv_len + max_nodes > max_kv_len could be exceeded (kv_len < 0 or kv_len + 1 > max_kv_len). */
ghd_status ghd_kv_commit(ghd_ctx *ctx, const ghd_kv_layer *kv, int32_t n_layers, int32_t kv_len,
                         const ghd_accept_result *result_dev);

/* The device word with the cache length (see GHD_KV_LEN_DEVICE). */
/* Sets the word (enqueued on the context's stream).  GHD_ENOSPACE: no workspace, or kv_len outside [0, max_kv_len). */
ghd_status ghd_kv_len_set(ghd_ctx *ctx, int32_t kv_len);
/* Waits for the context's stream and copies the word to *kv_len_host. */
ghd_status ghd_kv_len_get(ghd_ctx *ctx, int32_t *kv_len_host);

/* Self-drafting with extra heads (paper Sec. II-C: Medusa-style heads attached after the last layer each
 * draft the token of one later position; the paper's default drafter).  The paper does not
 * spell out a head; the reading taken is the Medusa head: y_k = h + SiLU(W1_k h), logits_k = W2_k y_k, where h is
 * the model's last hidden state (after the final RMSNorm) at the LAST ACCEPTED node, head k drafts the token
 * k + 1 positions after the bonus token, and its top-t_k tokens (ties: lower id first) are the candidates of
 * tree level k + 1.
 *   w1: dev T [n_heads][d_model][d_model], w2: dev T [n_heads][vocab][d_model]. */
typedef struct ghd_medusa_weights {
    int32_t n_heads;                  /* <= GHD_MAX_DRAFT_HEADS */
    const void *w1, *w2;
} ghd_medusa_weights;
#define GHD_MAX_DRAFT_HEADS 8
#define GHD_MAX_TOPK 16

/* Runs the heads on the hidden state that the last ghd_verify_step of this context left for node
 * result_dev->nodes[n_matched] (read on the device) and writes, for head k, its topk_host[k] best token ids
 * to cand_dev[k * GHD_MAX_TOPK ..] (int32, best first; unused entries -1).  logits_dev: float
 * [n_heads][vocab] or NULL.  Must follow ghd_verify_step on the same context and stream with nothing of this
 * library in between except ghd_accept / ghd_kv_commit.  GHD_EINVAL: null pointer, n_heads or a top-k out of
 * range. */
ghd_status ghd_medusa_draft(ghd_ctx *ctx, const ghd_medusa_weights *w, const ghd_accept_result *result_dev,
                            const int32_t *topk_host, int32_t *cand_dev, float *logits_dev);

/* Fills the token slots of the next tree from the candidates: node 0 gets the bonus token
 * result_dev->tokens[n_matched]; node i > 0 gets cand[level[i] - 1][rank[i]] (level_dev / rank_dev: int32 [n],
 * the node's depth and its rank among the candidates of its head, e.g. from the tree design).  tokens_dev: int32 [n]. */
ghd_status ghd_tree_fill_tokens(ghd_ctx *ctx, const int32_t *cand_dev, const ghd_accept_result *result_dev,
                                const int32_t *level_dev, const int32_t *rank_dev, int32_t n, int32_t *tokens_dev);

/* Building blocks of the layer, exposed for unit tests (same kernels the layer uses).
 * ghd_linear: y float [n][m] = x T[n][k] * w T[m][k]^T.
 * ghd_gate_up: u T [n][d_ffn] = SiLU(h Wg^T) * (h Wu^T) for h T [n][d_model], w_gate_up T [2*d_ffn][d_model]
 *   (gate rows, then up rows): the first half of the MLP block with its activation fused, as the layer runs it.
 * ghd_rmsnorm: out T [n][d_model] = RMSNorm(x float [n][d_model]) * g.
 * ghd_tree_attention: q T [n][n_heads*d_head] (rotated), caches already holding the
 *   n new rows at [kv_len, kv_len+n) -> out T [n][n_heads*d_head].
 * ghd_argmax: float [n][v] -> int32 [n]. */
ghd_status ghd_linear(ghd_ctx *ctx, const void *x, const void *w, int32_t n, int32_t k, int32_t m, float *y);
ghd_status ghd_gate_up(ghd_ctx *ctx, const void *h, const void *w_gate_up, int32_t n, void *u);
ghd_status ghd_rmsnorm(ghd_ctx *ctx, const float *x, const void *g, int32_t n, void *out);
ghd_status ghd_tree_attention(ghd_ctx *ctx, const void *q, const ghd_kv_layer *kv, const ghd_tree *tree, void *out);
ghd_status ghd_argmax(ghd_ctx *ctx, const float *logits, int32_t n, int32_t v, int32_t *out);

/* (The paper has no counterpart of this call; it exists for deployment reasons only.)
 * ghd_tree_attention for callers that must not allocate device memory - code that runs
 * inside another framework's fixed memory pool, plugins of a serving process whose memory
 * budget is frozen at start-up, or loops in which cudaMalloc (it may synchronise the whole
 * device) is forbidden.  Such callers cannot provide the workspace that holds the per-split
 * partial results, so this variant keeps them in an array built into the library image
 * (about 8.25 MiB, present on every GPU that loads the library until the process exits).
 * It needs no context and calls no allocating routine.
 *   stream: cudaStream_t (NULL = default).  dtype: ghd_dtype of q, caches and out.
 *   q, out: dev T [n][n_heads*d_head]; k_cache, v_cache: dev T [n_heads][max_kv_len][d_head]
 *   already holding the n new rows at [kv_len, kv_len + n); mask_dev: dev uint64
 *   [n][ceil(n/64)] as in ghd_tree.  err_buf (host, may be NULL) receives a message on failure.
 * Limits: n <= 64 and n_heads * d_head <= 4096, else GHD_ENOSPACE; d_head in {64, 128}.
 * The first call on each device looks up the array's device address; make that first call
 * outside any stream capture.  All calls on a device share the one array (it keeps whatever
 * the previous call left; every slot that is read is rewritten first, so nothing needs
 * clearing): two calls whose kernels may overlap on the GPU - different streams without an
 * ordering between them - race on it.  Calls on one stream are safe. */
ghd_status ghd_tree_attention_static(void *cuda_stream, int32_t dtype, int32_t n_heads, int32_t d_head,
                                     int32_t max_kv_len, const void *q, const void *k_cache, const void *v_cache,
                                     const uint64_t *mask_dev, int32_t n, int32_t kv_len, void *out,
                                     char *err_buf, size_t err_len);

/* Synchronises the stream and returns GHD_OK, GHD_ECUDA (with the CUDA error kept
 * for ghd_last_error) or GHD_ETIMEOUT when a kernel's bounded wait expired. */
ghd_status ghd_sync_status(ghd_ctx *ctx);
const char *ghd_status_str(ghd_status s);
const char *ghd_last_error(const ghd_ctx *ctx);
/* Kernels this context has launched so far (for launch accounting in benchmarks). */
int64_t ghd_launch_count(const ghd_ctx *ctx);

#ifdef __cplusplus
}
#endif
#endif /* GHD_H_ */
