// Tree attention on CUDA cores (float math): the attention of the float32 mode,
// and the fallback of the half mode.
//
// Keys/values of one head are the cache rows [0, kv_len) followed by the n new
// rows [kv_len, kv_len + n) that the projection step already appended.  Query i
// sees every cache row (the dense part) and new row j only when bit j of its
// ancestor mask is set (the sparse part).  The key range is cut into splits; a
// block handles QB queries of one head for one split with a running (max, sum)
// softmax, and a second kernel merges the splits by rescaling with exp(m_s - m)
// (paper Sec. III-B-2: each partition keeps its own softmax and the results are
// aligned by a scaling factor at the end).  32-key tiles of the new-row region in
// which no query of the block has a visible key are skipped without being loaded.
#include <cstdio>
#include <mutex>

#include "internal.h"

namespace ghd {

namespace {

constexpr int QB = 8;      // queries (warps) per block
constexpr int TK = 32;     // keys per tile

template <typename T> __device__ __forceinline__ float ld_f32(const T* p);
template <> __device__ __forceinline__ float ld_f32<float>(const float* p) { return *p; }
template <> __device__ __forceinline__ float ld_f32<__half>(const __half* p) { return __half2float(*p); }
template <typename T> __device__ __forceinline__ T st_cvt(float v);
template <> __device__ __forceinline__ float st_cvt<float>(float v) { return v; }
template <> __device__ __forceinline__ __half st_cvt<__half>(float v) { return __float2half_rn(v); }

template <typename T, int DH>
__global__ void __launch_bounds__(QB * 32)
k_attn_simt(const T* __restrict__ q, const T* __restrict__ kc, const T* __restrict__ vc,
            const uint64_t* __restrict__ mask, int n_words, int n, int n_new, int heads, int kv_len, int max_kv,
            int chunk, float* __restrict__ part_o, float* __restrict__ part_ml, int max_nodes, const int* __restrict__ kv_len_dev) {
    constexpr int R = DH / 32;
    if (kv_len_dev) {          // the length lives on the device: deal the keys to the splits here
        kv_len = resolve_kv_len(kv_len, kv_len_dev, max_kv, n);
        chunk = (kv_len + n_new + (int)gridDim.z - 1) / (int)gridDim.z;
        chunk = ((chunk + TK - 1) / TK) * TK;
    }
    __shared__ float sq[QB][DH];
    __shared__ float sk[TK][DH + 1];
    __shared__ float sv[TK][DH + 1];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int h = blockIdx.y, split = blockIdx.z;
    const int i = blockIdx.x * QB + warp;
    const bool live = i < n;
    const int d = heads * DH;
    const int kt = kv_len + n_new;                         // n_new = n, or 0 when the new rows are handled elsewhere
    const int j_begin = split * chunk, j_end = min(kt, j_begin + chunk);
    const float scale = rsqrtf((float)DH);
    for (int c = lane; c < DH; c += 32) sq[warp][c] = live ? ld_f32<T>(q + (size_t)i * d + h * DH + c) * scale : 0.f;
    float m = -INFINITY, l = 0.f, o[R];
#pragma unroll
    for (int r = 0; r < R; ++r) o[r] = 0.f;
    const T* kbase = kc + (size_t)h * max_kv * DH;
    const T* vbase = vc + (size_t)h * max_kv * DH;
    __syncthreads();
    for (int t0 = j_begin; t0 < j_end; t0 += TK) {
        const int j = t0 + lane;
        bool vis = live && j < j_end;
        if (vis && j >= kv_len) {
            const int b = j - kv_len;
            vis = (mask[(size_t)i * n_words + (b >> 6)] >> (b & 63)) & 1ull;
        }
        const bool warp_any = __any_sync(0xffffffffu, vis);
        if (!__syncthreads_or(warp_any ? 1 : 0)) continue;   // nobody in the block needs this tile
        for (int e = threadIdx.x; e < TK * DH; e += QB * 32) {
            const int r = e / DH, c = e % DH;
            const bool in = t0 + r < j_end;
            sk[r][c] = in ? ld_f32<T>(kbase + (size_t)(t0 + r) * DH + c) : 0.f;
            sv[r][c] = in ? ld_f32<T>(vbase + (size_t)(t0 + r) * DH + c) : 0.f;
        }
        __syncthreads();
        if (warp_any) {
            float s = 0.f;
#pragma unroll 8
            for (int c = 0; c < DH; ++c) s = fmaf(sq[warp][c], sk[lane][c], s);
            s = vis ? s : -INFINITY;
            float tmax = s;
            for (int sh = 16; sh > 0; sh >>= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, sh));
            const float m_new = fmaxf(m, tmax);
            const float corr = (m == -INFINITY) ? 0.f : expf(m - m_new);
            const float p = vis ? expf(s - m_new) : 0.f;
            float psum = p;
            for (int sh = 16; sh > 0; sh >>= 1) psum += __shfl_xor_sync(0xffffffffu, psum, sh);
            l = l * corr + psum;
#pragma unroll
            for (int r = 0; r < R; ++r) o[r] *= corr;
            for (int jj = 0; jj < TK; ++jj) {
                const float pj = __shfl_sync(0xffffffffu, p, jj);
#pragma unroll
                for (int r = 0; r < R; ++r) o[r] = fmaf(pj, sv[jj][lane + 32 * r], o[r]);
            }
            m = m_new;
        }
        __syncthreads();
    }
    if (live) {
        float* po = part_o + ((size_t)split * max_nodes + i) * d + h * DH;
#pragma unroll
        for (int r = 0; r < R; ++r) po[lane + 32 * r] = o[r];
        if (lane == 0) {
            float* pm = part_ml + (((size_t)split * max_nodes + i) * heads + h) * 2;
            pm[0] = m;
            pm[1] = l;
        }
    }
}

// Sparse part of the tree attention from a coordinate index (paper Sec. III-B-3: the visible (query, key)
// pairs are listed before the inference; Q K^T touches one row of Q and one row of K per pair, A V adds
// A[i][j] * V[j] into row i of O, which stays in registers until the row's pairs are exhausted).  One warp per
// (query, head): lane t holds DH / 32 consecutive columns of q, of the output row and of every K / V row it
// reads (a row is one coalesced request of the warp); a query with depth + 1 visible nodes reads exactly that
// many rows, whatever the size of the tree.  Leaves the un-normalised (o, max, sum) of the new-row part.
constexpr int COO_WARPS = 4;

// R consecutive elements (R = 2 or 4, the address R-element aligned) in one request, widened to float.
template <typename T, int R>
__device__ __forceinline__ void ld_row_piece(const T* p, float (&v)[R]) {
    if constexpr (sizeof(T) == 4) {
        if constexpr (R == 4) { const float4 t = *reinterpret_cast<const float4*>(p); v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w; }
        else { const float2 t = *reinterpret_cast<const float2*>(p); v[0] = t.x; v[1] = t.y; }
    } else {
        if constexpr (R == 4) {
            const uint2 t = *reinterpret_cast<const uint2*>(p);
            const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&t.x)), b = __half22float2(*reinterpret_cast<const __half2*>(&t.y));
            v[0] = a.x; v[1] = a.y; v[2] = b.x; v[3] = b.y;
        } else {
            const float2 a = __half22float2(*reinterpret_cast<const __half2*>(p));
            v[0] = a.x; v[1] = a.y;
        }
    }
}

template <typename T, int DH>
__global__ void __launch_bounds__(COO_WARPS * 32)
k_attn_coo(const T* __restrict__ q, const T* __restrict__ kc, const T* __restrict__ vc, const int32_t* __restrict__ coo_ptr,
           const int32_t* __restrict__ coo_col, int n, int heads, int kv_len, int max_kv,
           float* __restrict__ part_o, float* __restrict__ part_ml, const int* __restrict__ kv_len_dev) {
    constexpr int R = DH / 32;
    pdl_wait();
    pdl_trigger();
    kv_len = resolve_kv_len(kv_len, kv_len_dev, max_kv, n);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int i = blockIdx.x * COO_WARPS + warp, h = blockIdx.y;
    if (i >= n) return;
    const int d = heads * DH;
    const float scale = rsqrtf((float)DH);
    float qv[R], o[R];
    ld_row_piece<T, R>(q + (size_t)i * d + h * DH + lane * R, qv);
#pragma unroll
    for (int r = 0; r < R; ++r) { qv[r] *= scale; o[r] = 0.f; }
    const T* kbase = kc + ((size_t)h * max_kv + kv_len) * DH + lane * R;
    const T* vbase = vc + ((size_t)h * max_kv + kv_len) * DH + lane * R;
    float m = -INFINITY, l = 0.f;
    const int e0 = coo_ptr[i], e1 = coo_ptr[i + 1];
    for (int e = e0; e < e1; ++e) {
        const int j = coo_col[e];
        float kr[R], vr[R], s = 0.f;
        ld_row_piece<T, R>(kbase + (size_t)j * DH, kr);
        ld_row_piece<T, R>(vbase + (size_t)j * DH, vr);
#pragma unroll
        for (int r = 0; r < R; ++r) s = fmaf(qv[r], kr[r], s);
        for (int sh = 16; sh > 0; sh >>= 1) s += __shfl_xor_sync(0xffffffffu, s, sh);
        const float m_new = fmaxf(m, s);
        const float corr = (m == -INFINITY) ? 0.f : expf(m - m_new);
        const float pj = expf(s - m_new);
        l = l * corr + pj;
#pragma unroll
        for (int r = 0; r < R; ++r) o[r] = fmaf(pj, vr[r], o[r] * corr);
        m = m_new;
    }
    float* po = part_o + (size_t)i * d + h * DH + lane * R;
#pragma unroll
    for (int r = 0; r < R; ++r) po[r] = o[r];
    if (lane == 0) {
        float* pm = part_ml + ((size_t)i * heads + h) * 2;
        pm[0] = m;
        pm[1] = l;
    }
}

// out[i][h*DH + c] = sum_s e^{m_s - m} o_s / sum_s e^{m_s - m} l_s ; splits that saw no key have m_s = -inf.
template <typename T>
__global__ void k_attn_combine(const float* __restrict__ part_o, const float* __restrict__ part_ml, T* __restrict__ out,
                               int splits, int heads, int dh, int max_nodes) {
    pdl_wait();
    pdl_trigger();
    const int i = blockIdx.x, h = blockIdx.y, d = heads * dh;
    float m = -INFINITY;
    for (int s = 0; s < splits; ++s) m = fmaxf(m, part_ml[(((size_t)s * max_nodes + i) * heads + h) * 2]);
    float den = 0.f;
    for (int s = 0; s < splits; ++s) {
        const float* pm = part_ml + (((size_t)s * max_nodes + i) * heads + h) * 2;
        if (pm[0] != -INFINITY) den += pm[1] * expf(pm[0] - m);
    }
    for (int c = threadIdx.x; c < dh; c += blockDim.x) {
        float acc = 0.f;
        for (int s = 0; s < splits; ++s) {
            const float ms = part_ml[(((size_t)s * max_nodes + i) * heads + h) * 2];
            if (ms != -INFINITY) acc += part_o[((size_t)s * max_nodes + i) * d + h * dh + c] * expf(ms - m);
        }
        out[(size_t)i * d + h * dh + c] = st_cvt<T>(acc / den);
    }
}

// Same merge, one block per node and four consecutive features per thread (16-byte loads):
// used when the row width is a multiple of 4, i.e. always for the supported head sizes.
template <typename T>
__global__ void __launch_bounds__(1024) k_attn_combine_rows(const float* __restrict__ part_o, const float* __restrict__ part_ml, T* __restrict__ out,
                                    int splits, int heads, int dh, int max_nodes) {
    pdl_wait();
    pdl_trigger();
    const int i = blockIdx.x, d = heads * dh;
    for (int f = 4 * threadIdx.x; f < d; f += 4 * blockDim.x) {
        const int h = f / dh;
        // all loads of up to four splits go out together, then the weights are worked out
        float ms[4], ls[4];
        float4 ov[4];
        float m = -INFINITY, den = 0.f;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int s0 = 0; s0 < splits; s0 += 4) {
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int s = s0 + q;
                ms[q] = -INFINITY; ls[q] = 0.f; ov[q] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (s < splits) {
                    const float2 ml = *reinterpret_cast<const float2*>(part_ml + (((size_t)s * max_nodes + i) * heads + h) * 2);
                    ms[q] = ml.x; ls[q] = ml.y;
                    ov[q] = *reinterpret_cast<const float4*>(part_o + ((size_t)s * max_nodes + i) * d + f);
                }
            }
            float m_new = m;
#pragma unroll
            for (int q = 0; q < 4; ++q) m_new = fmaxf(m_new, ms[q]);
            if (m_new == -INFINITY) continue;
            const float rescale = (m == -INFINITY) ? 0.f : expf(m - m_new);
            den *= rescale; acc.x *= rescale; acc.y *= rescale; acc.z *= rescale; acc.w *= rescale;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                if (ms[q] == -INFINITY) continue;
                const float w = expf(ms[q] - m_new);
                den += ls[q] * w;
                acc.x += ov[q].x * w; acc.y += ov[q].y * w; acc.z += ov[q].z * w; acc.w += ov[q].w * w;
            }
            m = m_new;
        }
        const float inv = 1.f / den;
        T* dst = out + (size_t)i * d + f;
        dst[0] = st_cvt<T>(acc.x * inv); dst[1] = st_cvt<T>(acc.y * inv);
        dst[2] = st_cvt<T>(acc.z * inv); dst[3] = st_cvt<T>(acc.w * inv);
    }
}

}  // namespace

int attn_auto_splits(const ghd_ctx* c, int n, int kv_total) {
    const int blocks = ((n + QB - 1) / QB) * c->cfg.n_heads;
    int s = (2 * c->sm_count + blocks - 1) / blocks;
    const int by_len = (kv_total + 127) / 128;      // at least 128 keys per split
    if (s > by_len) s = by_len;
    if (s > c->max_splits) s = c->max_splits;
    return s < 1 ? 1 : s;
}

void launch_attn_simt(ghd_ctx* c, const void* q, const ghd_kv_layer* kv, const ghd_tree* t, void* out, bool coo) {
    const ghd_model_cfg& m = c->cfg;
    const int n_new = coo ? 0 : t->n;
    const int kt = kv_len_host_of(c, t) + n_new;
    int splits = c->opt_attn_splits > 0 ? c->opt_attn_splits : attn_auto_splits(c, t->n, kt);
    if (splits > c->max_splits - (coo ? 1 : 0)) splits = c->max_splits - (coo ? 1 : 0);
    int chunk = (kt + splits - 1) / splits;
    chunk = ((chunk + TK - 1) / TK) * TK;
    dim3 grid((t->n + QB - 1) / QB, m.n_heads, splits);
#define GHD_ATTN(T, DH)                                                                                          \
    k_attn_simt<T, DH><<<grid, QB * 32, 0, c->cur>>>((const T*)q, (const T*)kv->k, (const T*)kv->v, t->mask,  \
                                                        t->n_words, t->n, n_new, m.n_heads, t->kv_len, m.max_kv_len, \
                                                        chunk, c->att_o, c->att_ml, m.max_nodes, kv_len_dev_of(c, t))
    if (m.dtype == GHD_F32) { if (m.d_head == 64) GHD_ATTN(float, 64); else GHD_ATTN(float, 128); }
    else { if (m.d_head == 64) GHD_ATTN(__half, 64); else GHD_ATTN(__half, 128); }
#undef GHD_ATTN
    c->launches++;
    if (coo) { launch_attn_coo(c, q, kv, t, splits); ++splits; }      // the sparse part as one more partial
    dim3 cgrid(t->n, m.n_heads);
    if (m.dtype == GHD_F32)
        k_attn_combine<float><<<cgrid, m.d_head, 0, c->cur>>>(c->att_o, c->att_ml, (float*)out, splits, m.n_heads,
                                                                 m.d_head, m.max_nodes);
    else
        k_attn_combine<__half><<<cgrid, m.d_head, 0, c->cur>>>(c->att_o, c->att_ml, (__half*)out, splits, m.n_heads,
                                                                  m.d_head, m.max_nodes);
    c->launches++;
}

void launch_attn_coo(ghd_ctx* c, const void* q, const ghd_kv_layer* kv, const ghd_tree* t, int slot) {
    const ghd_model_cfg& m = c->cfg;
    dim3 grid((t->n + COO_WARPS - 1) / COO_WARPS, m.n_heads);
#define GHD_COO(T, DH)                                                                                              \
    launch_k(c, true, k_attn_coo<T, DH>, grid, dim3(COO_WARPS * 32), 0, (const T*)q, (const T*)kv->k, (const T*)kv->v,   \
             (const int32_t*)t->coo_ptr, (const int32_t*)t->coo_col, t->n, m.n_heads, t->kv_len, m.max_kv_len,      \
             c->att_o + (size_t)slot * m.max_nodes * m.d_model, c->att_ml + (size_t)slot * m.max_nodes * m.n_heads * 2, \
             kv_len_dev_of(c, t))
    if (m.dtype == GHD_F32) { if (m.d_head == 64) GHD_COO(float, 64); else GHD_COO(float, 128); }
    else { if (m.d_head == 64) GHD_COO(__half, 64); else GHD_COO(__half, 128); }
#undef GHD_COO
}

void launch_attn_combine(ghd_ctx* c, void* out, int splits, int n) {
    const ghd_model_cfg& m = c->cfg;
    if (splits <= 16) {
        int threads = ((m.d_model / 4 + 31) / 32) * 32;
        if (threads > 1024) threads = 1024;
        if (m.dtype == GHD_F32)
            launch_k(c, true, k_attn_combine_rows<float>, n, threads, 0, (const float*)c->att_o, (const float*)c->att_ml,
                     (float*)out, splits, m.n_heads, m.d_head, m.max_nodes);
        else
            launch_k(c, true, k_attn_combine_rows<__half>, n, threads, 0, (const float*)c->att_o, (const float*)c->att_ml,
                     (__half*)out, splits, m.n_heads, m.d_head, m.max_nodes);
        return;
    }
    dim3 cgrid(n, m.n_heads);
    if (m.dtype == GHD_F32)
        launch_k(c, true, k_attn_combine<float>, cgrid, m.d_head, 0, (const float*)c->att_o, (const float*)c->att_ml, (float*)out,
                 splits, m.n_heads, m.d_head, m.max_nodes);
    else
        launch_k(c, true, k_attn_combine<__half>, cgrid, m.d_head, 0, (const float*)c->att_o, (const float*)c->att_ml, (__half*)out,
                 splits, m.n_heads, m.d_head, m.max_nodes);
}

// ---------------------------------------------------------------------------
// Tree attention for callers that cannot allocate device memory.
//
// Some hosts of this library are not allowed to call cudaMalloc at all: code
// running inside another framework's pre-sized memory pool, a plugin in a
// serving process whose memory budget is fixed at start-up, or a latency-critical
// loop where an allocation (which may synchronise the device) is forbidden.
// They cannot give ghd_tree_attention the workspace it needs for its per-split
// partial results.  This variant keeps those partials in a fixed array that is
// part of the library image instead; every GPU that loads the library carries
// the array (about 8.25 MiB) until the process exits.
// ---------------------------------------------------------------------------
namespace {

constexpr int ST_MAX_NODES = 64;       // tree nodes
constexpr int ST_MAX_WIDTH = 4096;     // n_heads * d_head
constexpr int ST_MAX_HEADS = ST_MAX_WIDTH / 64;
constexpr int ST_MAX_SPLITS = 8;
constexpr size_t ST_O_FLOATS = (size_t)ST_MAX_SPLITS * ST_MAX_NODES * ST_MAX_WIDTH;
constexpr size_t ST_ML_FLOATS = (size_t)ST_MAX_SPLITS * ST_MAX_NODES * ST_MAX_HEADS * 2;

// Split partials: numerators first, then (running max, running sum) pairs.
static __device__ __align__(256) float g_static_scratch[ST_O_FLOATS + ST_ML_FLOATS];

constexpr int ST_MAX_DEVICES = 64;
float* g_static_scratch_addr[ST_MAX_DEVICES];   // device address of the array, per device, once known
std::mutex g_static_scratch_lock;

void st_error(char* buf, size_t len, const char* msg) {
    if (buf && len) snprintf(buf, len, "%s", msg);
}

}  // namespace
}  // namespace ghd

extern "C" ghd_status ghd_tree_attention_static(void* cuda_stream, int32_t dtype, int32_t n_heads, int32_t d_head,
                                                int32_t max_kv_len, const void* q, const void* k_cache,
                                                const void* v_cache, const uint64_t* mask_dev, int32_t n,
                                                int32_t kv_len, void* out, char* err_buf, size_t err_len) {
    using namespace ghd;
    if (!q || !k_cache || !v_cache || !mask_dev || !out) { st_error(err_buf, err_len, "null pointer argument"); return GHD_EINVAL; }
    if (dtype != GHD_F32 && dtype != GHD_F16) { st_error(err_buf, err_len, "dtype must be GHD_F32 or GHD_F16"); return GHD_EINVAL; }
    if (d_head != 64 && d_head != 128) { st_error(err_buf, err_len, "d_head must be 64 or 128"); return GHD_ESHAPE; }
    if (n_heads < 1 || n < 1 || kv_len < 0 || max_kv_len < 1) { st_error(err_buf, err_len, "non-positive size"); return GHD_EINVAL; }
    if (n > ST_MAX_NODES || (int64_t)n_heads * d_head > ST_MAX_WIDTH) {
        st_error(err_buf, err_len, "beyond the built-in scratch: at most 64 tree nodes and n_heads * d_head <= 4096");
        return GHD_ENOSPACE;
    }
    if ((int64_t)kv_len + n > max_kv_len) { st_error(err_buf, err_len, "kv_len + n > max_kv_len"); return GHD_ENOSPACE; }

    // Set-up, once per device: in host code `g_static_scratch` is only a handle of the
    // symbol, so ask the runtime where the array lives on the current device.
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= ST_MAX_DEVICES) {
        st_error(err_buf, err_len, "cannot identify the current device");
        return GHD_ECUDA;
    }
    float* scratch = nullptr;
    {
        std::lock_guard<std::mutex> hold(g_static_scratch_lock);
        if (!g_static_scratch_addr[dev]) {
            void* p = nullptr;
            const cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
            if (e != cudaSuccess || !p) {
                st_error(err_buf, err_len, cudaGetErrorString(e));
                return GHD_ECUDA;
            }
            g_static_scratch_addr[dev] = static_cast<float*>(p);
        }
        scratch = g_static_scratch_addr[dev];
    }
    float* part_o = scratch;
    float* part_ml = scratch + ST_O_FLOATS;

    // Nothing in the array has to start at zero: every (split, node, head) slot that the merge
    // kernel reads is written by the split kernel of this same call (splits without a visible
    // key write max = -inf, sum = 0), so what an earlier call left behind is never observed.
    const int kt = kv_len + n;
    int splits = (kt + 255) / 256;
    if (splits > ST_MAX_SPLITS) splits = ST_MAX_SPLITS;
    if (splits < 1) splits = 1;
    int chunk = (kt + splits - 1) / splits;
    chunk = ((chunk + TK - 1) / TK) * TK;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    dim3 grid((n + QB - 1) / QB, n_heads, splits);
    const int n_words = (n + 63) / 64;
#define GHD_ATTN_ST(T, DH)                                                                                  \
    k_attn_simt<T, DH><<<grid, QB * 32, 0, stream>>>((const T*)q, (const T*)k_cache, (const T*)v_cache,      \
                                                     mask_dev, n_words, n, n, n_heads, kv_len, max_kv_len,   \
                                                     chunk, part_o, part_ml, ST_MAX_NODES, (const int*)nullptr)
    if (dtype == GHD_F32) { if (d_head == 64) GHD_ATTN_ST(float, 64); else GHD_ATTN_ST(float, 128); }
    else { if (d_head == 64) GHD_ATTN_ST(__half, 64); else GHD_ATTN_ST(__half, 128); }
#undef GHD_ATTN_ST
    dim3 cgrid(n, n_heads);
    if (dtype == GHD_F32)
        k_attn_combine<float><<<cgrid, d_head, 0, stream>>>(part_o, part_ml, (float*)out, splits, n_heads, d_head, ST_MAX_NODES);
    else
        k_attn_combine<__half><<<cgrid, d_head, 0, stream>>>(part_o, part_ml, (__half*)out, splits, n_heads, d_head, ST_MAX_NODES);
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { st_error(err_buf, err_len, cudaGetErrorString(e)); return GHD_ECUDA; }
    return GHD_OK;
}
