// Small kernels of the verify step: tree build, embedding gather, RMSNorm,
// RoPE + KV append, SwiGLU, residual add, row argmax, acceptance walk.
#include "internal.h"

namespace ghd {

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__half>(__half v) { return __half2float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __half from_f32<__half>(float v) { return __float2half_rn(v); }

#define GHD_DISPATCH_T(c, expr_f32, expr_f16) \
    do { if ((c)->cfg.dtype == GHD_F32) { expr_f32; } else { expr_f16; } } while (0)

// ---------------------------------------------------------------- tree build
struct ParentArg { int16_t p[GHD_MAX_NODES]; };
// Row starts of the coordinate index (nnz <= 256 * 257 / 2 fits 16 bits), worked out on the host.
struct CooPtrArg { uint16_t ptr[GHD_MAX_NODES + 1]; };

// Block b takes nodes 8b .. 8b+7: one thread per node walks to the root, setting one mask bit per
// ancestor; then the block fills those nodes' rows of the rotary table.  The table is computed in
// double so that the angle pos * theta^(-2t/dh) carries no float rounding of the frequency; that is
// the slow part (pow and sincos in double), hence several blocks.
constexpr int TREE_NODES_PER_BLOCK = 8;

// Length of the cache for a tree kernel: the host's value, or the device word (clamped into the cache; a word
// outside [0, max_kv_len - n] is recorded in the status word by the kernel's first thread).
__device__ __forceinline__ int tree_kv_len(int host, const int* dev, int max_kv_len, int n, int* status, bool reporter) {
    if (dev && reporter) {
        const int raw = __ldcg(dev);
        if (raw < 0 || raw > max_kv_len - n) atomicCAS(status, DEV_OK, DEV_KV_RANGE);
    }
    return resolve_kv_len(host, dev, max_kv_len, n);
}

__global__ void k_tree_build(ParentArg pa, CooPtrArg cp, int n, int n_words, int kv_len, int d_head, double theta,
                             uint64_t* mask, int32_t* parent, int32_t* depth, int32_t* pos, float* rope,
                             int32_t* coo_ptr, int32_t* coo_col, const int* kv_len_dev, int max_kv_len, int* status) {
    __shared__ int spos[TREE_NODES_PER_BLOCK];
    kv_len = tree_kv_len(kv_len, kv_len_dev, max_kv_len, n, status, blockIdx.x == 0 && threadIdx.x == 0);
    const int first = blockIdx.x * TREE_NODES_PER_BLOCK;
    if (threadIdx.x < TREE_NODES_PER_BLOCK) {
        const int i = first + threadIdx.x;
        int p = kv_len;
        if (i < n) {
            uint64_t row[GHD_MAX_NODES / 64] = {0, 0, 0, 0};
            int steps = 0;
            for (int a = i; a >= 0 && steps <= n; a = pa.p[a]) { row[a >> 6] |= 1ull << (a & 63); ++steps; }
            for (int w = 0; w < n_words; ++w) mask[i * n_words + w] = row[w];
            if (coo_ptr) {
                // the same walk again, filling the row's list from its end: ancestors come out in descending order
                coo_ptr[i] = cp.ptr[i];
                if (i == n - 1) coo_ptr[n] = cp.ptr[n];
                int at = cp.ptr[i + 1], left = steps;
                for (int a = i; a >= 0 && left > 0 && at > cp.ptr[i]; a = pa.p[a], --left) coo_col[--at] = a;
            }
            parent[i] = pa.p[i];
            depth[i] = steps - 1;
            p = kv_len + steps - 1;
            pos[i] = p;
        }
        spos[threadIdx.x] = p;
    }
    __syncthreads();
    const int half = d_head / 2;
    for (int e = threadIdx.x; e < TREE_NODES_PER_BLOCK * half; e += blockDim.x) {
        const int local = e / half, t = e % half, node = first + local;
        if (node >= n) break;
        const double ang = (double)spos[local] * pow(theta, -2.0 * t / d_head);
        double s, c;
        sincos(ang, &s, &c);
        rope[node * d_head + 2 * t] = (float)c;
        rope[node * d_head + 2 * t + 1] = (float)s;
    }
}

// Explicit-mask variant: mask (and optionally depth, parent) were copied in.
__global__ void k_tree_from_mask(CooPtrArg cp, int n, int n_words, int kv_len, int d_head, double theta, int have_depth,
                                 const uint64_t* mask, int32_t* depth, int32_t* pos, float* rope, int32_t* coo_ptr, int32_t* coo_col,
                                 const int* kv_len_dev, int max_kv_len, int* status) {
    const int i = threadIdx.x;
    kv_len = tree_kv_len(kv_len, kv_len_dev, max_kv_len, n, status, threadIdx.x == 0);
    if (i < n && coo_ptr) {
        coo_ptr[i] = cp.ptr[i];
        if (i == n - 1) coo_ptr[n] = cp.ptr[n];
        int at = cp.ptr[i];
        for (int w = 0; w < n_words; ++w)
            for (uint64_t bits = mask[i * n_words + w]; bits && at < cp.ptr[i + 1]; bits &= bits - 1) coo_col[at++] = 64 * w + __ffsll((long long)bits) - 1;
    }
    if (i < n) {
        int dep;
        if (have_depth) dep = depth[i];
        else {
            int bits = 0;
            for (int w = 0; w < n_words; ++w) bits += __popcll(mask[i * n_words + w]);
            dep = bits - 1;
            depth[i] = dep;
        }
        pos[i] = kv_len + dep;
    }
    __syncthreads();
    const int half = d_head / 2;
    for (int e = threadIdx.x; e < n * half; e += blockDim.x) {
        const int node = e / half, t = e % half;
        const double ang = (double)pos[node] * pow(theta, -2.0 * t / d_head);
        double s, c;
        sincos(ang, &s, &c);
        rope[node * d_head + 2 * t] = (float)c;
        rope[node * d_head + 2 * t + 1] = (float)s;
    }
}

void launch_tree_build(ghd_ctx* c, const int32_t* parent_host, ghd_tree* t) {
    ParentArg pa;
    CooPtrArg cp;
    int depth[GHD_MAX_NODES];
    cp.ptr[0] = 0;
    for (int i = 0; i < GHD_MAX_NODES; ++i) {
        pa.p[i] = (int16_t)(i < t->n ? parent_host[i] : -1);
        if (i < t->n) {                                   // row i lists node i and its ancestors: depth + 1 entries
            depth[i] = i == 0 ? 0 : depth[parent_host[i]] + 1;
            cp.ptr[i + 1] = (uint16_t)(cp.ptr[i] + depth[i] + 1);
        } else {
            cp.ptr[i + 1] = cp.ptr[i];
        }
    }
    t->nnz = cp.ptr[t->n];
    k_tree_build<<<(t->n + TREE_NODES_PER_BLOCK - 1) / TREE_NODES_PER_BLOCK, 256, 0, c->cur>>>(pa, cp, t->n, t->n_words, t->kv_len, c->cfg.d_head,
                                                     (double)c->cfg.rope_theta, t->mask, t->parent, t->depth,
                                                     t->pos, t->rope, t->coo_ptr, t->coo_col, kv_len_dev_of(c, t), c->cfg.max_kv_len, c->status);
    c->launches++;
}

void launch_tree_from_mask(ghd_ctx* c, ghd_tree* t, bool have_depth, const uint64_t* mask_host) {
    CooPtrArg cp;
    cp.ptr[0] = 0;
    for (int i = 0; i < GHD_MAX_NODES; ++i) {
        int bits = 0;
        if (i < t->n)
            for (int w = 0; w < t->n_words; ++w) bits += __builtin_popcountll(mask_host[(size_t)i * t->n_words + w]);
        cp.ptr[i + 1] = (uint16_t)(cp.ptr[i] + bits);
    }
    t->nnz = cp.ptr[t->n];
    k_tree_from_mask<<<1, GHD_MAX_NODES, 0, c->cur>>>(cp, t->n, t->n_words, t->kv_len, c->cfg.d_head,
                                                         (double)c->cfg.rope_theta, have_depth ? 1 : 0, t->mask,
                                                         t->depth, t->pos, t->rope, t->coo_ptr, t->coo_col, kv_len_dev_of(c, t),
                                                         c->cfg.max_kv_len, c->status);
    c->launches++;
}

// ---------------------------------------------------------------- x in / out, embedding
template <typename T>
__global__ void k_load_x(const T* __restrict__ x, float* __restrict__ xres, size_t count) {
    for (size_t e = blockIdx.x * (size_t)blockDim.x + threadIdx.x; e < count; e += (size_t)gridDim.x * blockDim.x)
        xres[e] = to_f32<T>(x[e]);
}

template <typename T>
__global__ void k_store_x(const float* __restrict__ xres, T* __restrict__ x, size_t count) {
    for (size_t e = blockIdx.x * (size_t)blockDim.x + threadIdx.x; e < count; e += (size_t)gridDim.x * blockDim.x)
        x[e] = from_f32<T>(xres[e]);
}

template <typename T>
__global__ void k_embed(const T* __restrict__ table, const int32_t* __restrict__ tokens, float* __restrict__ xres, int d) {
    pdl_wait();
    pdl_trigger();
    const T* row = table + (size_t)tokens[blockIdx.x] * d;
    for (int cidx = threadIdx.x; cidx < d; cidx += blockDim.x) xres[(size_t)blockIdx.x * d + cidx] = to_f32<T>(row[cidx]);
}

static int grid_for(size_t count, int block, int cap) {
    size_t g = (count + block - 1) / block;
    return (int)(g < 1 ? 1 : (g > (size_t)cap ? cap : g));
}

void launch_load_x(ghd_ctx* c, const void* x_in, int n) {
    const size_t count = (size_t)n * c->cfg.d_model;
    const int g = grid_for(count, 256, 4 * c->sm_count);
    GHD_DISPATCH_T(c, (k_load_x<float><<<g, 256, 0, c->cur>>>((const float*)x_in, c->xres, count)),
                   (k_load_x<__half><<<g, 256, 0, c->cur>>>((const __half*)x_in, c->xres, count)));
    c->launches++;
}

void launch_store_x(ghd_ctx* c, void* x_out, int n) {
    const size_t count = (size_t)n * c->cfg.d_model;
    const int g = grid_for(count, 256, 4 * c->sm_count);
    GHD_DISPATCH_T(c, (k_store_x<float><<<g, 256, 0, c->cur>>>(c->xres, (float*)x_out, count)),
                   (k_store_x<__half><<<g, 256, 0, c->cur>>>(c->xres, (__half*)x_out, count)));
    c->launches++;
}

void launch_embed(ghd_ctx* c, const void* embed, const int32_t* tokens, int n) {
    GHD_DISPATCH_T(c, launch_k(c, true, k_embed<float>, n, 256, 0, (const float*)embed, tokens, c->xres, c->cfg.d_model),
                   launch_k(c, true, k_embed<__half>, n, 256, 0, (const __half*)embed, tokens, c->xres, c->cfg.d_model));
}

// ---------------------------------------------------------------- RMSNorm
__device__ __forceinline__ float block_sum(float v, float* red) {
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
    if (l == 0) red[w] = v;
    __syncthreads();
    const int nw = (blockDim.x + 31) >> 5;
    float t = (threadIdx.x < nw) ? red[threadIdx.x] : 0.f;
    if (w == 0) {
        for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
        if (l == 0) red[0] = t;
    }
    __syncthreads();
    const float r = red[0];
    __syncthreads();
    return r;
}

// One block per row: out = x * g / sqrt(mean(x^2) + eps), math in float.  The row is read
// once with 16-byte loads and kept in registers (up to RMS_V float4 per thread).
constexpr int RMS_V = 4;

template <typename T> __device__ __forceinline__ void store4(T* p, float a, float b, float c, float d);
template <> __device__ __forceinline__ void store4<float>(float* p, float a, float b, float c, float d) {
    *reinterpret_cast<float4*>(p) = make_float4(a, b, c, d);
}
template <> __device__ __forceinline__ void store4<__half>(__half* p, float a, float b, float c, float d) {
    const __half2 lo = __floats2half2_rn(a, b), hi = __floats2half2_rn(c, d);
    uint2 u;
    u.x = *reinterpret_cast<const uint32_t*>(&lo);
    u.y = *reinterpret_cast<const uint32_t*>(&hi);
    *reinterpret_cast<uint2*>(p) = u;
}
template <typename T> __device__ __forceinline__ float4 load4(const T* p);
template <> __device__ __forceinline__ float4 load4<float>(const float* p) { return *reinterpret_cast<const float4*>(p); }
template <> __device__ __forceinline__ float4 load4<__half>(const __half* p) {
    const uint2 u = *reinterpret_cast<const uint2*>(p);
    const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&u.x)), b = __half22float2(*reinterpret_cast<const __half2*>(&u.y));
    return make_float4(a.x, a.y, b.x, b.y);
}

template <typename T>
__global__ void __launch_bounds__(1024) k_rmsnorm(const float* __restrict__ x, const T* __restrict__ g, T* __restrict__ out, int d, float eps) {
    __shared__ float red[32];
    pdl_wait();
    pdl_trigger();
    const float* row = x + (size_t)blockIdx.x * d;
    const int nv = d >> 2;                        // d is a multiple of 8
    float4 v[RMS_V];
    float ss = 0.f;
#pragma unroll
    for (int k = 0; k < RMS_V; ++k) {
        const int idx = threadIdx.x + k * blockDim.x;
        v[k] = (idx < nv) ? *reinterpret_cast<const float4*>(row + 4 * idx) : make_float4(0.f, 0.f, 0.f, 0.f);
        ss += v[k].x * v[k].x + v[k].y * v[k].y + v[k].z * v[k].z + v[k].w * v[k].w;
    }
    for (int idx = threadIdx.x + RMS_V * blockDim.x; idx < nv; idx += blockDim.x) {      // very wide rows
        const float4 w = *reinterpret_cast<const float4*>(row + 4 * idx);
        ss += w.x * w.x + w.y * w.y + w.z * w.z + w.w * w.w;
    }
    ss = block_sum(ss, red);
    const float r = rsqrtf(ss / (float)d + eps);
    T* orow = out + (size_t)blockIdx.x * d;
#pragma unroll
    for (int k = 0; k < RMS_V; ++k) {
        const int idx = threadIdx.x + k * blockDim.x;
        if (idx < nv) {
            const float4 gg = load4<T>(g + 4 * idx);
            store4<T>(orow + 4 * idx, v[k].x * r * gg.x, v[k].y * r * gg.y, v[k].z * r * gg.z, v[k].w * r * gg.w);
        }
    }
    for (int idx = threadIdx.x + RMS_V * blockDim.x; idx < nv; idx += blockDim.x) {
        const float4 w = *reinterpret_cast<const float4*>(row + 4 * idx);
        const float4 gg = load4<T>(g + 4 * idx);
        store4<T>(orow + 4 * idx, w.x * r * gg.x, w.y * r * gg.y, w.z * r * gg.z, w.w * r * gg.w);
    }
}

void launch_rmsnorm(ghd_ctx* c, const float* x, const void* g, int n, void* out) {
    const int d = c->cfg.d_model;
    int threads = ((d / 4 + 31) / 32) * 32;
    if (threads > 1024) threads = 1024;
    GHD_DISPATCH_T(c, launch_k(c, true, k_rmsnorm<float>, n, threads, 0, x, (const float*)g, (float*)out, d, c->cfg.rms_eps),
                   launch_k(c, true, k_rmsnorm<__half>, n, threads, 0, x, (const __half*)g, (__half*)out, d, c->cfg.rms_eps));
}

// The first norm of a call when the projections normalise in their epilogues: xg = x * g (gain-weighted,
// not divided by the rms) and the row's sum of squares as the single "tile" of a sum-of-squares buffer.
__global__ void __launch_bounds__(1024) k_prenorm(const float* __restrict__ x, const __half* __restrict__ g, __half* __restrict__ xg,
                                                  float* __restrict__ ssq, int d) {
    __shared__ float red[32];
    pdl_wait();
    pdl_trigger();
    const float* row = x + (size_t)blockIdx.x * d;
    __half* orow = xg + (size_t)blockIdx.x * d;
    const int nv = d >> 2;
    float ss = 0.f;
    for (int idx = threadIdx.x; idx < nv; idx += blockDim.x) {
        const float4 w = *reinterpret_cast<const float4*>(row + 4 * idx);
        const float4 gg = load4<__half>(g + 4 * idx);
        ss += w.x * w.x + w.y * w.y + w.z * w.z + w.w * w.w;
        store4<__half>(orow + 4 * idx, w.x * gg.x, w.y * gg.y, w.z * gg.z, w.w * gg.w);
    }
    ss = block_sum(ss, red);
    if (threadIdx.x == 0) ssq[blockIdx.x] = ss;
}

void launch_prenorm(ghd_ctx* c, const void* g, int n, void* xg, float* ssq) {
    const int d = c->cfg.d_model;
    int threads = ((d / 4 + 31) / 32) * 32;
    if (threads > 1024) threads = 1024;
    launch_k(c, true, k_prenorm, n, threads, 0, (const float*)c->xres, (const __half*)g, (__half*)xg, ssq, d);
}

// Folds the partial tiles of a deferred-reduction projection into the residual stream and,
// in the same pass, produces the next RMSNorm output.  One block per node; a thread owns four
// consecutive features (all inside one 128-row tile), adds that tile's contributors in CTA
// order (fixed order -> reproducible), then the row's mean square is reduced across the block.
template <typename T>
__global__ void __launch_bounds__(1024) k_fold_pending(float* __restrict__ xres, const float* __restrict__ part, PendingPartials pp,
                               const T* __restrict__ g, T* __restrict__ h_out, T* __restrict__ x_out, int d, float eps) {
    __shared__ float red[32];
    pdl_wait();
    pdl_trigger();
    const int node = blockIdx.x;
    const int nv = d >> 2;
    float4 v[RMS_V];
    float ss = 0.f;
#pragma unroll
    for (int k = 0; k < RMS_V; ++k) {
        const int idx = threadIdx.x + k * blockDim.x;
        v[k] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (idx < nv) {
            const int f = 4 * idx, tile = f >> 7, row = f & 127;
            const int c_first = pp.first_cta[tile], cnt = pp.n_contrib[tile], slot0 = pp.first_slot[tile];
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int cb = 0; cb < cnt; cb += 8) {          // up to eight loads in flight, summed in CTA order
                float4 t[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    t[q] = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (cb + q < cnt) {
                        const int slot = (cb + q == 0) ? slot0 : 0;
                        t[q] = __ldcg(reinterpret_cast<const float4*>(part + ((size_t)(c_first + (cb + q) * pp.stride) * 2 + slot) * pp.slot_elems +
                                                                      (size_t)node * 128 + row));
                    }
                }
#pragma unroll
                for (int q = 0; q < 8; ++q) { acc.x += t[q].x; acc.y += t[q].y; acc.z += t[q].z; acc.w += t[q].w; }
            }
            float4 x = *reinterpret_cast<const float4*>(xres + (size_t)node * d + f);
            x.x += acc.x; x.y += acc.y; x.z += acc.z; x.w += acc.w;
            *reinterpret_cast<float4*>(xres + (size_t)node * d + f) = x;
            v[k] = x;
            ss += x.x * x.x + x.y * x.y + x.z * x.z + x.w * x.w;
        }
    }
    if (x_out) {
#pragma unroll
        for (int k = 0; k < RMS_V; ++k) {
            const int idx = threadIdx.x + k * blockDim.x;
            if (idx < nv) store4<T>(x_out + (size_t)node * d + 4 * idx, v[k].x, v[k].y, v[k].z, v[k].w);
        }
    }
    if (h_out) {
        ss = block_sum(ss, red);
        const float r = rsqrtf(ss / (float)d + eps);
#pragma unroll
        for (int k = 0; k < RMS_V; ++k) {
            const int idx = threadIdx.x + k * blockDim.x;
            if (idx < nv) {
                const float4 gg = load4<T>(g + 4 * idx);
                store4<T>(h_out + (size_t)node * d + 4 * idx, v[k].x * r * gg.x, v[k].y * r * gg.y, v[k].z * r * gg.z, v[k].w * r * gg.w);
            }
        }
    }
}

void launch_fold_pending(ghd_ctx* c, int n, const void* g, void* h_out, void* x_out) {
    const int d = c->cfg.d_model;
    int threads = (((d / 4 + RMS_V - 1) / RMS_V + 31) / 32) * 32;      // d/4 float4 per row, up to RMS_V per thread
    if (d / 4 <= 1024) threads = ((d / 4 + 31) / 32) * 32;
    launch_k(c, true, k_fold_pending<__half>, n, threads, 0, c->xres, (const float*)c->gemm_part, c->pending, (const __half*)g,
             (__half*)h_out, (__half*)x_out, d, c->cfg.rms_eps);
    c->pending.active = 0;
}

// ---------------------------------------------------------------- RoPE + KV append (un-fused path)
// qkv float [n][3 d].  Thread per (node, head, t < dh/2): rotates the q and k pairs
// (t, t + dh/2), writes q to the query buffer and k, v to cache row kv_len + node.
template <typename T>
__global__ void k_rope_append(const float* __restrict__ qkv, const float* __restrict__ rope, T* __restrict__ q,
                              T* __restrict__ kc, T* __restrict__ vc, int n, int heads, int dh, int kv_len, int max_kv,
                              const int* __restrict__ kv_len_dev) {
    kv_len = resolve_kv_len(kv_len, kv_len_dev, max_kv, n);
    const int half = dh / 2, d = heads * dh;
    const size_t total = (size_t)n * heads * half;
    for (size_t e = blockIdx.x * (size_t)blockDim.x + threadIdx.x; e < total; e += (size_t)gridDim.x * blockDim.x) {
        const int t = (int)(e % half), h = (int)((e / half) % heads), i = (int)(e / ((size_t)half * heads));
        const float cs = rope[i * dh + 2 * t], sn = rope[i * dh + 2 * t + 1];
        const float* base = qkv + (size_t)i * 3 * d + h * dh;
        const float qa = base[t], qb = base[t + half];
        const float ka = base[d + t], kb = base[d + t + half];
        T* qo = q + (size_t)i * d + h * dh;
        qo[t] = from_f32<T>(qa * cs - qb * sn);
        qo[t + half] = from_f32<T>(qb * cs + qa * sn);
        const size_t crow = ((size_t)h * max_kv + kv_len + i) * dh;
        kc[crow + t] = from_f32<T>(ka * cs - kb * sn);
        kc[crow + t + half] = from_f32<T>(kb * cs + ka * sn);
        vc[crow + t] = from_f32<T>(base[2 * d + t]);
        vc[crow + t + half] = from_f32<T>(base[2 * d + t + half]);
    }
}

void launch_rope_append(ghd_ctx* c, const float* qkv_raw, const ghd_tree* t, const ghd_kv_layer* kv) {
    const ghd_model_cfg& m = c->cfg;
    const size_t total = (size_t)t->n * m.n_heads * (m.d_head / 2);
    const int g = grid_for(total, 256, 8 * c->sm_count);
    GHD_DISPATCH_T(c,
        (k_rope_append<float><<<g, 256, 0, c->cur>>>(qkv_raw, t->rope, (float*)c->qbuf, (float*)kv->k, (float*)kv->v,
                                                         t->n, m.n_heads, m.d_head, t->kv_len, m.max_kv_len, kv_len_dev_of(c, t))),
        (k_rope_append<__half><<<g, 256, 0, c->cur>>>(qkv_raw, t->rope, (__half*)c->qbuf, (__half*)kv->k, (__half*)kv->v,
                                                          t->n, m.n_heads, m.d_head, t->kv_len, m.max_kv_len, kv_len_dev_of(c, t))));
    c->launches++;
}

// ---------------------------------------------------------------- SwiGLU, residual (un-fused path)
template <typename T>
__global__ void k_swiglu(const float* __restrict__ gu, T* __restrict__ u, int n, int f) {
    const size_t total = (size_t)n * f;
    for (size_t e = blockIdx.x * (size_t)blockDim.x + threadIdx.x; e < total; e += (size_t)gridDim.x * blockDim.x) {
        const size_t i = e / f, cidx = e % f;
        const float g = gu[i * 2 * f + cidx], up = gu[i * 2 * f + f + cidx];
        u[e] = from_f32<T>(g / (1.f + expf(-g)) * up);
    }
}

void launch_swiglu(ghd_ctx* c, const float* gu_raw, int n) {
    const size_t total = (size_t)n * c->cfg.d_ffn;
    const int g = grid_for(total, 256, 8 * c->sm_count);
    GHD_DISPATCH_T(c, (k_swiglu<float><<<g, 256, 0, c->cur>>>(gu_raw, (float*)c->ubuf, n, c->cfg.d_ffn)),
                   (k_swiglu<__half><<<g, 256, 0, c->cur>>>(gu_raw, (__half*)c->ubuf, n, c->cfg.d_ffn)));
    c->launches++;
}

__global__ void k_residual(float* __restrict__ xres, const float* __restrict__ proj, size_t count) {
    for (size_t e = blockIdx.x * (size_t)blockDim.x + threadIdx.x; e < count; e += (size_t)gridDim.x * blockDim.x)
        xres[e] += proj[e];
}

void launch_residual(ghd_ctx* c, const float* proj_raw, int n) {
    const size_t count = (size_t)n * c->cfg.d_model;
    k_residual<<<grid_for(count, 256, 8 * c->sm_count), 256, 0, c->cur>>>(c->xres, proj_raw, count);
    c->launches++;
}

// ---------------------------------------------------------------- row argmax
// One block per row; each warp scans a strided slice, lanes keep (value, index)
// with "greater value, or equal value and smaller index" as the order, so equal
// maxima resolve to the first index.  NaN never wins.
__device__ __forceinline__ void amax_merge(float& v, int& i, float ov, int oi) {
    if (ov > v || (ov == v && oi < i)) { v = ov; i = oi; }
}

__global__ void k_argmax(const float* __restrict__ logits, int v, int32_t* __restrict__ out) {
    __shared__ float sv[32];
    __shared__ int si[32];
    pdl_wait();
    pdl_trigger();
    const float* row = logits + (size_t)blockIdx.x * v;
    float best = -INFINITY;
    int bi = 0x7fffffff;
    if ((v & 3) == 0 && (reinterpret_cast<uintptr_t>(logits) & 15) == 0) {   // 16-byte aligned rows: four columns per load
        const float4* row4 = reinterpret_cast<const float4*>(row);
#pragma unroll 4
        for (int q = threadIdx.x; q < (v >> 2); q += blockDim.x) {
            const float4 w = __ldcs(row4 + q);
            amax_merge(best, bi, w.x, 4 * q);
            amax_merge(best, bi, w.y, 4 * q + 1);
            amax_merge(best, bi, w.z, 4 * q + 2);
            amax_merge(best, bi, w.w, 4 * q + 3);
        }
    } else {
        for (int cidx = threadIdx.x; cidx < v; cidx += blockDim.x) amax_merge(best, bi, row[cidx], cidx);
    }
    for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, best, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        amax_merge(best, bi, ov, oi);
    }
    const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
    if (l == 0) { sv[w] = best; si[w] = bi; }
    __syncthreads();
    if (w == 0) {
        const int nw = blockDim.x >> 5;
        best = l < nw ? sv[l] : -INFINITY;
        bi = l < nw ? si[l] : 0x7fffffff;
        for (int o = 16; o > 0; o >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, best, o);
            const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
            amax_merge(best, bi, ov, oi);
        }
        if (l == 0) out[blockIdx.x] = (bi == 0x7fffffff) ? 0 : bi;
    }
}

void launch_argmax(ghd_ctx* c, const float* logits, int n, int v, int32_t* out) {
    launch_k(c, true, k_argmax, n, 1024, 0, logits, v, out);
}

// ---------------------------------------------------------------- acceptance
// Thread i checks every edge on the root path of node i; the deepest valid node
// wins, the lowest index among equally deep ones.  Thread 0 then writes the path.
__global__ void k_accept(int n, const int32_t* __restrict__ parent,
                         const int32_t* __restrict__ tokens, const int32_t* __restrict__ amax,
                         ghd_accept_result* __restrict__ out) {
    __shared__ int key[GHD_MAX_NODES];
    const int i = threadIdx.x;
    int k = -1;
    if (i < n) {
        bool ok = true;
        int dep = 0;
        for (int cnode = i; cnode > 0 && dep <= n; ++dep) {
            const int p = parent[cnode];
            if (tokens[cnode] != amax[p]) ok = false;
            cnode = p;
        }
        if (ok) k = dep * GHD_MAX_NODES + (GHD_MAX_NODES - 1 - i);
    }
    key[i] = k;
    __syncthreads();
    for (int s = GHD_MAX_NODES / 2; s > 0; s >>= 1) {
        if (i < s) key[i] = max(key[i], key[i + s]);
        __syncthreads();
    }
    if (i == 0) {
        const int best = key[0];
        const int dep = best / GHD_MAX_NODES, win = GHD_MAX_NODES - 1 - (best % GHD_MAX_NODES);
        out->n_matched = dep;
        out->n_emitted = dep + 1;
        int cnode = win;
        for (int j = dep; j >= 0; --j) {
            out->nodes[j] = cnode;
            out->tokens[j] = amax[cnode];
            cnode = (j > 0) ? parent[cnode] : 0;
        }
    }
}

void launch_accept(ghd_ctx* c, const ghd_tree* t, const int32_t* tokens, const int32_t* amax, ghd_accept_result* out) {
    k_accept<<<1, GHD_MAX_NODES, 0, c->cur>>>(t->n, t->parent, tokens, amax, out);
    c->launches++;
}

// ---------------------------------------------------------------- drafting heads
// h_sel = hidden state (after the final norm) of the last accepted node, picked on the device.
template <typename T>
__global__ void k_medusa_gather(const T* __restrict__ hbuf, const ghd_accept_result* __restrict__ res, int d, int max_nodes, T* __restrict__ h_sel,
                                const float* __restrict__ ssq, int ssq_tiles, float eps) {
    int m = res->n_matched;
    if (m < 0 || m >= GHD_MAX_NODES) m = 0;
    int node = res->nodes[m];
    if (node < 0 || node >= max_nodes) node = 0;
    float r = 1.f;
    if (ssq) {      // hbuf holds gain-weighted rows that still want their 1 / rms
        float ss = 0.f;
        for (int t = 0; t < ssq_tiles; ++t) ss += ssq[(size_t)t * SSQ_PITCH + node];
        r = rsqrtf(ss / (float)d + eps);
    }
    for (int j = blockIdx.x * blockDim.x + threadIdx.x; j < d; j += gridDim.x * blockDim.x) h_sel[j] = (T)((float)hbuf[(size_t)node * d + j] * r);
}
// y[k][j] = h[j] + SiLU(raw[k * d + j])
template <typename T>
__global__ void k_medusa_res(const T* __restrict__ h, const float* __restrict__ raw, int heads, int d, T* __restrict__ y) {
    const int total = heads * d;
    for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < total; e += gridDim.x * blockDim.x) {
        const float a = raw[e];
        y[e] = from_f32<T>(to_f32<T>(h[e % d]) + a / (1.f + expf(-a)));
    }
}

// Block k: the topk[k] largest logits of head k, best first, ties to the lower id: one block-wide
// argmax per rank, each excluding what the earlier ranks took (a taken id is greater in the order).
struct TopkArg { int t[GHD_MAX_DRAFT_HEADS]; };

__global__ void __launch_bounds__(1024) k_medusa_topk(const float* __restrict__ logits, int vocab, TopkArg topk, int32_t* __restrict__ cand) {
    __shared__ float sv[32];
    __shared__ int si[32];
    __shared__ float last_v;
    __shared__ int last_i;
    const float* row = logits + (size_t)blockIdx.x * vocab;
    const int t = topk.t[blockIdx.x];
    const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
    if (threadIdx.x == 0) { last_v = INFINITY; last_i = -1; }
    __syncthreads();
    for (int r = 0; r < GHD_MAX_TOPK; ++r) {
        if (r >= t) {
            if (threadIdx.x == 0) cand[blockIdx.x * GHD_MAX_TOPK + r] = -1;
            continue;
        }
        const float lv = last_v;
        const int li = last_i;
        float best = -INFINITY;
        int bi = 0x7fffffff;
        for (int cidx = threadIdx.x; cidx < vocab; cidx += blockDim.x) {
            const float v = row[cidx];
            // still available: strictly after (lv, li) in the order "greater value, then smaller id"
            if (v < lv || (v == lv && cidx > li)) amax_merge(best, bi, v, cidx);
        }
        for (int o = 16; o > 0; o >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, best, o);
            const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
            amax_merge(best, bi, ov, oi);
        }
        if (l == 0) { sv[w] = best; si[w] = bi; }
        __syncthreads();
        if (w == 0) {
            const int nw = blockDim.x >> 5;
            best = l < nw ? sv[l] : -INFINITY;
            bi = l < nw ? si[l] : 0x7fffffff;
            for (int o = 16; o > 0; o >>= 1) {
                const float ov = __shfl_xor_sync(0xffffffffu, best, o);
                const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
                amax_merge(best, bi, ov, oi);
            }
            if (l == 0) {
                cand[blockIdx.x * GHD_MAX_TOPK + r] = (bi == 0x7fffffff) ? -1 : bi;
                last_v = best;
                last_i = bi;
            }
        }
        __syncthreads();
    }
}

__global__ void k_tree_fill(const int32_t* __restrict__ cand, const ghd_accept_result* __restrict__ res, const int32_t* __restrict__ level,
                            const int32_t* __restrict__ rank, int n, int32_t* __restrict__ tokens) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    if (i == 0) {
        int m = res->n_matched;
        if (m < 0 || m >= GHD_MAX_NODES) m = 0;
        tokens[0] = res->tokens[m];
        return;
    }
    const int lv = level[i], rk = rank[i];
    tokens[i] = (lv >= 1 && lv <= GHD_MAX_DRAFT_HEADS && rk >= 0 && rk < GHD_MAX_TOPK) ? cand[(lv - 1) * GHD_MAX_TOPK + rk] : -1;
}

void launch_medusa_gather(ghd_ctx* c, const ghd_accept_result* res, void* h_sel, const float* ssq, int ssq_tiles) {
    const int d = c->cfg.d_model;
    const float eps = c->cfg.rms_eps;
    GHD_DISPATCH_T(c, (k_medusa_gather<float><<<1, 1024, 0, c->cur>>>((const float*)c->hbuf, res, d, c->cfg.max_nodes, (float*)h_sel, ssq, ssq_tiles, eps)),
                   (k_medusa_gather<__half><<<1, 1024, 0, c->cur>>>((const __half*)c->hbuf, res, d, c->cfg.max_nodes, (__half*)h_sel, ssq, ssq_tiles, eps)));
    c->launches++;
}

void launch_medusa_res(ghd_ctx* c, const void* h_sel, const float* raw, int heads, void* y) {
    const int d = c->cfg.d_model;
    const int g = grid_for((size_t)heads * d, 256, 8 * c->sm_count);
    GHD_DISPATCH_T(c, (k_medusa_res<float><<<g, 256, 0, c->cur>>>((const float*)h_sel, raw, heads, d, (float*)y)),
                   (k_medusa_res<__half><<<g, 256, 0, c->cur>>>((const __half*)h_sel, raw, heads, d, (__half*)y)));
    c->launches++;
}

void launch_medusa_topk(ghd_ctx* c, const float* logits, int heads, int vocab, const int* topk, int32_t* cand) {
    TopkArg a{};
    for (int k = 0; k < heads; ++k) a.t[k] = topk[k];
    k_medusa_topk<<<heads, 1024, 0, c->cur>>>(logits, vocab, a, cand);
    c->launches++;
}

void launch_tree_fill(ghd_ctx* c, const int32_t* cand, const ghd_accept_result* res, const int32_t* level, const int32_t* rank, int n, int32_t* tokens) {
    k_tree_fill<<<(n + 255) / 256, 256, 0, c->cur>>>(cand, res, level, rank, n, tokens);
    c->launches++;
}

// ---------------------------------------------------------------- KV commit
// Block (layer, head, K or V); thread = one 16-byte piece of a row.  Row kv_len + nodes[j] moves to
// row kv_len + j for j = 1 .. n_matched (j = 0 is the root, already in place).  nodes[] increases
// and nodes[j] >= j, so a thread that copies its piece in ascending j never reads a piece it has
// already overwritten, and threads own disjoint pieces: no synchronisation is needed.
constexpr int COMMIT_LAYERS = 64;
struct CommitPtrs {
    void* k[COMMIT_LAYERS];
    void* v[COMMIT_LAYERS];
};

__global__ void k_kv_commit(CommitPtrs ptrs, int heads, int max_kv_len, int row_bytes, int kv_len,
                            const ghd_accept_result* __restrict__ res, const int* __restrict__ kv_len_dev) {
    kv_len = resolve_kv_len(kv_len, kv_len_dev, max_kv_len, 1);
    const int layer = blockIdx.x / heads, head = blockIdx.x - layer * heads;
    char* base = (char*)(blockIdx.y == 0 ? ptrs.k[layer] : ptrs.v[layer]) + (size_t)head * max_kv_len * row_bytes;
    int m = res->n_matched;
    if (m > GHD_MAX_NODES - 1) m = GHD_MAX_NODES - 1;
    for (int j = 1; j <= m; ++j) {
        const int src = res->nodes[j];
        if (src == j || src < 0 || src >= GHD_MAX_NODES || kv_len + src >= max_kv_len) continue;
        const uint4* from = reinterpret_cast<const uint4*>(base + (size_t)(kv_len + src) * row_bytes);
        uint4* to = reinterpret_cast<uint4*>(base + (size_t)(kv_len + j) * row_bytes);
        for (int q = threadIdx.x; q < row_bytes / 16; q += blockDim.x) to[q] = from[q];
    }
}

// The cache length after a step: the accepted path adds n_matched + 1 rows (Sec. II-C).
__global__ void k_kv_len_advance(int* word, const ghd_accept_result* __restrict__ res, int max_kv_len) {
    int m = res->n_matched;
    if (m < 0) m = 0;
    if (m > GHD_MAX_NODES - 1) m = GHD_MAX_NODES - 1;
    int v = *word;
    if (v < 0) v = 0;
    v += m + 1;
    *word = v > max_kv_len - 1 ? max_kv_len - 1 : v;
}
__global__ void k_kv_len_set(int* word, int v) { *word = v; }

void launch_kv_commit(ghd_ctx* c, const ghd_kv_layer* kv, int n_layers, int kv_len, const ghd_accept_result* res) {
    const ghd_model_cfg& m = c->cfg;
    const int row_bytes = m.d_head * (m.dtype == GHD_F32 ? 4 : 2);
    for (int l0 = 0; l0 < n_layers; l0 += COMMIT_LAYERS) {
        CommitPtrs ptrs{};
        const int cnt = n_layers - l0 < COMMIT_LAYERS ? n_layers - l0 : COMMIT_LAYERS;
        for (int l = 0; l < cnt; ++l) { ptrs.k[l] = kv[l0 + l].k; ptrs.v[l] = kv[l0 + l].v; }
        k_kv_commit<<<dim3(cnt * m.n_kv_heads, 2), 32, 0, c->cur>>>(ptrs, m.n_kv_heads, m.max_kv_len, row_bytes, kv_len, res,
                                                                    kv_len < 0 ? c->kv_len_word : nullptr);
        c->launches++;
    }
    if (kv_len < 0) {          // every move above read the old length: advance the word behind them
        k_kv_len_advance<<<1, 1, 0, c->cur>>>(c->kv_len_word, res, m.max_kv_len);
        c->launches++;
        if (c->kv_len_hint + 1 < m.max_kv_len) c->kv_len_hint += 1;      // a step emits at least one token
    }
}

void launch_kv_len_set(ghd_ctx* c, int kv_len) {
    k_kv_len_set<<<1, 1, 0, c->cur>>>(c->kv_len_word, kv_len);
    c->launches++;
    c->kv_len_hint = kv_len;
}

}  // namespace ghd
