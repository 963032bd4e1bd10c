// Plain CUDA-core projection GEMM: y float [n][m] = x T [n][k] * w T [m][k]^T,
// float accumulation.  It is the only GEMM of the float32 mode (tensor cores have
// no exact float32 product) and the fallback of the half mode for shapes the
// tcgen05 kernel does not take.
//
// One warp owns one output feature for a group of NG nodes: its lanes stride
// over k with 16-byte loads of the weight row (read exactly once per group) and
// of the NG activation rows, keep NG partial sums, and finish with a shuffle
// reduction in a fixed order, so results are run-to-run identical.
#include "internal.h"

namespace ghd {

namespace {

constexpr int NG = 8;        // nodes per warp pass
constexpr int WARPS = 8;     // output features per block

template <typename T> struct Vec;
template <> struct Vec<float> {
    static constexpr int W = 4;
    __device__ static void load(const float* p, float (&o)[4]) {
        const float4 v = *reinterpret_cast<const float4*>(p);
        o[0] = v.x; o[1] = v.y; o[2] = v.z; o[3] = v.w;
    }
    __device__ static float one(const float* p) { return *p; }
};
template <> struct Vec<__half> {
    static constexpr int W = 8;
    __device__ static void load(const __half* p, float (&o)[8]) {
        const uint4 v = *reinterpret_cast<const uint4*>(p);
        const __half2* h = reinterpret_cast<const __half2*>(&v);
#pragma unroll
        for (int j = 0; j < 4; ++j) { const float2 f = __half22float2(h[j]); o[2 * j] = f.x; o[2 * j + 1] = f.y; }
    }
    __device__ static float one(const __half* p) { return __half2float(*p); }
};

template <typename T>
__global__ void __launch_bounds__(WARPS * 32)
k_gemm_simt(const T* __restrict__ x, const T* __restrict__ w, float* __restrict__ y, int n, int k, int m) {
    constexpr int W = Vec<T>::W;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int o = blockIdx.x * WARPS + warp;
    const int i0 = blockIdx.y * NG;
    if (o >= m) return;
    const T* wrow = w + (size_t)o * k;
    float acc[NG];
#pragma unroll
    for (int g = 0; g < NG; ++g) acc[g] = 0.f;
    const int kvec = (k / W) * W;
    for (int c = lane * W; c < kvec; c += 32 * W) {
        float wv[W];
        Vec<T>::load(wrow + c, wv);
#pragma unroll
        for (int g = 0; g < NG; ++g) {
            if (i0 + g < n) {
                float xv[W];
                Vec<T>::load(x + (size_t)(i0 + g) * k + c, xv);
#pragma unroll
                for (int j = 0; j < W; ++j) acc[g] = fmaf(wv[j], xv[j], acc[g]);
            }
        }
    }
    for (int c = kvec + lane; c < k; c += 32) {
        const float wv = Vec<T>::one(wrow + c);
#pragma unroll
        for (int g = 0; g < NG; ++g)
            if (i0 + g < n) acc[g] = fmaf(wv, Vec<T>::one(x + (size_t)(i0 + g) * k + c), acc[g]);
    }
#pragma unroll
    for (int g = 0; g < NG; ++g) {
        float v = acc[g];
        for (int s = 16; s > 0; s >>= 1) v += __shfl_xor_sync(0xffffffffu, v, s);
        if (lane == 0 && i0 + g < n) y[(size_t)(i0 + g) * m + o] = v;
    }
}

}  // namespace

void launch_gemm_simt(ghd_ctx* c, const void* x, const void* w, int n, int k, int m, float* y) {
    dim3 grid((m + WARPS - 1) / WARPS, (n + NG - 1) / NG);
    if (c->cfg.dtype == GHD_F32)
        k_gemm_simt<float><<<grid, WARPS * 32, 0, c->cur>>>((const float*)x, (const float*)w, y, n, k, m);
    else
        k_gemm_simt<__half><<<grid, WARPS * 32, 0, c->cur>>>((const __half*)x, (const __half*)w, y, n, k, m);
    c->launches++;
}

}  // namespace ghd
