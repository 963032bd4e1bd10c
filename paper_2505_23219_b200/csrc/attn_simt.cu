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
            const uint64_t* __restrict__ mask, int n_words, int n, int heads, int kv_len, int max_kv,
            int chunk, float* __restrict__ part_o, float* __restrict__ part_ml, int max_nodes) {
    constexpr int R = DH / 32;
    __shared__ float sq[QB][DH];
    __shared__ float sk[TK][DH + 1];
    __shared__ float sv[TK][DH + 1];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int h = blockIdx.y, split = blockIdx.z;
    const int i = blockIdx.x * QB + warp;
    const bool live = i < n;
    const int d = heads * DH;
    const int kt = kv_len + n;
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

// out[i][h*DH + c] = sum_s e^{m_s - m} o_s / sum_s e^{m_s - m} l_s ; splits that saw no key have m_s = -inf.
template <typename T>
__global__ void k_attn_combine(const float* __restrict__ part_o, const float* __restrict__ part_ml, T* __restrict__ out,
                               int splits, int heads, int dh, int max_nodes) {
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

}  // namespace

int attn_auto_splits(const ghd_ctx* c, int n, int kv_total) {
    const int blocks = ((n + QB - 1) / QB) * c->cfg.n_heads;
    int s = (2 * c->sm_count + blocks - 1) / blocks;
    const int by_len = (kv_total + 127) / 128;      // at least 128 keys per split
    if (s > by_len) s = by_len;
    if (s > c->max_splits) s = c->max_splits;
    return s < 1 ? 1 : s;
}

void launch_attn_simt(ghd_ctx* c, const void* q, const ghd_kv_layer* kv, const ghd_tree* t, void* out) {
    const ghd_model_cfg& m = c->cfg;
    const int kt = t->kv_len + t->n;
    int splits = c->opt_attn_splits > 0 ? c->opt_attn_splits : attn_auto_splits(c, t->n, kt);
    if (splits > c->max_splits) splits = c->max_splits;
    int chunk = (kt + splits - 1) / splits;
    chunk = ((chunk + TK - 1) / TK) * TK;
    dim3 grid((t->n + QB - 1) / QB, m.n_heads, splits);
#define GHD_ATTN(T, DH)                                                                                          \
    k_attn_simt<T, DH><<<grid, QB * 32, 0, c->cur>>>((const T*)q, (const T*)kv->k, (const T*)kv->v, t->mask,  \
                                                        t->n_words, t->n, m.n_heads, t->kv_len, m.max_kv_len,    \
                                                        chunk, c->att_o, c->att_ml, m.max_nodes)
    if (m.dtype == GHD_F32) { if (m.d_head == 64) GHD_ATTN(float, 64); else GHD_ATTN(float, 128); }
    else { if (m.d_head == 64) GHD_ATTN(__half, 64); else GHD_ATTN(__half, 128); }
#undef GHD_ATTN
    c->launches++;
    dim3 cgrid(t->n, m.n_heads);
    if (m.dtype == GHD_F32)
        k_attn_combine<float><<<cgrid, m.d_head, 0, c->cur>>>(c->att_o, c->att_ml, (float*)out, splits, m.n_heads,
                                                                 m.d_head, m.max_nodes);
    else
        k_attn_combine<__half><<<cgrid, m.d_head, 0, c->cur>>>(c->att_o, c->att_ml, (__half*)out, splits, m.n_heads,
                                                                  m.d_head, m.max_nodes);
    c->launches++;
}

}  // namespace ghd
