// Device-side pieces shared by the tcgen05 projection kernels: tile constants, the parameter
// block of one projection, the shared-memory control block, and the fused epilogues.
#pragma once

#include "internal.h"
#include "tc_common.cuh"

namespace ghd {
namespace gemmdev {

constexpr int TILE_M = 128;          // output features per tile (MMA M)
constexpr int TILE_K = 64;           // halfs per k-step = one 128-byte swizzle row
constexpr int UMMA_K = 16;           // k per tcgen05.mma of kind::f16
constexpr int MAX_STAGES = 10;
constexpr int EPI_CHUNK = 32;        // accumulator columns per tcgen05.ld
constexpr int THREADS = 192;
constexpr int THREADS_TC = 320;      // k_gemm_tc: producer warp, MMA warp, two groups of four epilogue warps
constexpr int MAX_TILES = 256;
constexpr int MAX_WORKERS = 256;    // CTAs (or CTA pairs) of one launch
constexpr int DONE_OFF = 2048;       // counters[DONE_OFF + tile]: contributors that have finished their slice of a split tile

struct GemmParams {
    int n, nb, k, m;                 // nodes, padded nodes (MMA N), reduction length, output features
    int n_tiles, kiters, stages;     // kiters = k-chunks per tile; a chunk = ks column slabs of 64 = one pipeline stage
    int n_work, pair;                // work units dealt to the workers: tiles (one CTA each), or tile pairs (pair = 1: one cluster of two CTAs each)
    int ks, kslabs;                  // slabs per stage, slabs per weight row (k / 64)
    int swiglu_f;                    // d_ffn when the tile is [64 gate rows | 64 up rows], else 0
    int ctas;                        // CTAs of the launch; ctas / (1 + pair) workers share the flattened (work unit, k-chunk) space
    float* part;                     // [ctas][2][nb][128] float partial tiles
    int* counters;                   // [n_tiles] arrival counters, zero on entry and on exit
    int* status;
    EpiArgs epi;
    // per work unit, worked out on the host (64-bit divisions are slow on the device): first contributing
    // worker, number of contributors, slot of the first contributor (the others use slot 0)
    unsigned short tile_first[MAX_TILES];
    unsigned char tile_count[MAX_TILES], tile_slot[MAX_TILES];
    unsigned char tile_fin[MAX_TILES];   // which contributor (offset from the first) finishes a split tile: the one that ends last
    // first (work unit, k-chunk) iteration of every worker, and the end of the last: equal shares, except where the
    // host skews them so that the contributors of a tile do not all end together
    int range_beg[MAX_WORKERS + 1];
};

using namespace tc;

struct Smem {
    uint64_t full[MAX_STAGES];
    uint64_t empty[MAX_STAGES];
    uint64_t tmem_full[2];
    uint64_t tmem_empty[2];
    uint64_t drain;
    uint32_t tmem_base;
    int abort_flag;
    int last_flag;
    float stage_x[EPI_CHUNK][TILE_M + 1];   // epilogue exchange buffer (rotary pairs, gate/up pairs)
    float colscale[GHD_MAX_NODES];          // 1 / rms of every input row (projections that read un-normalised rows)
    float ssq_part[2][4][32];               // per epilogue group and warp: sums of squares of 32 rows x 32 nodes
    float ssq_slice[4][GHD_MAX_NODES / 2];  // slice finishing: per 32-row warp, sums of squares of the slice's columns
};

// s[j] (j < 32) summed over the 32 lanes of the warp; lane L returns the total of column L.
// Each step halves the columns a lane is responsible for: 16 + 8 + 4 + 2 + 1 shuffles.
template <int N>
__device__ __forceinline__ void warp_transpose_sum_step(float (&s)[32], int lane) {
    constexpr int H = N / 2;
    const bool up = (lane & H) != 0;
#pragma unroll
    for (int i = 0; i < H; ++i) {
        const float send = up ? s[i] : s[i + H];
        const float keep = up ? s[i + H] : s[i];
        s[i] = keep + __shfl_xor_sync(0xffffffffu, send, H);
    }
}
__device__ __forceinline__ float warp_transpose_sum(float (&s)[32], int lane) {
    warp_transpose_sum_step<32>(s, lane);
    warp_transpose_sum_step<16>(s, lane);
    warp_transpose_sum_step<8>(s, lane);
    warp_transpose_sum_step<4>(s, lane);
    warp_transpose_sum_step<2>(s, lane);
    return s[0];
}

// ---------------------------------------------------------------- fused epilogue
// Thread `row` (0..127) of the tile holds the final sums v[j] of its output feature for nodes
// c0 .. c0+31.  GROUPS = 1: four epilogue warps; GROUPS = 2: eight epilogue warps in two groups of
// four, group g taking the 32-column chunks g, g + 2, ... of a tile (so that the epilogue of a
// 64-node tile takes the time of one chunk).  The rotary and SwiGLU epilogues exchange values
// between threads through `stage_x`, XR = 32 / GROUPS node columns at a time, each group in its
// own rows of the buffer and with its own named barrier.
__device__ __forceinline__ void grp_bar(int grp) { asm volatile("bar.sync %0, 128;" ::"r"(1 + grp) : "memory"); }
__device__ __forceinline__ void all_epi_bar() { asm volatile("bar.sync 3, 256;" ::: "memory"); }

template <int GROUPS>
__device__ __forceinline__ void epilogue_chunk(const GemmParams& p, Smem* sm, int grp, int tile, int row, int c0, float (&v)[32]) {
    constexpr int XR = 32 / GROUPS;      // node columns per exchange pass
    constexpr int PASSES = GROUPS;
    const EpiArgs& e = p.epi;
    float (*xb)[TILE_M + 1] = sm->stage_x + grp * XR;
    if (e.ssq_in) {
#pragma unroll
        for (int j = 0; j < 32; ++j) v[j] *= sm->colscale[c0 + j];
    }
    if (e.mode == EPI_RESID_NORM) {
        // residual add, the gain-weighted copy for the next projection, and this tile's share of every
        // node's sum of squares (the consumer turns the sums into 1 / rms); m is a multiple of 128
        const int f = tile * TILE_M + row, lane = row & 31, quad = row >> 5;
        float* xr = e.out_f32 + (size_t)c0 * p.m + f;
        __half* xg = (__half*)e.xg_out + (size_t)c0 * p.m + f;
        const unsigned m = (unsigned)p.m;
        {
            float old[32];      // all loads first: a load after a store through another pointer would wait for it
#pragma unroll
            for (int j = 0; j < 32; ++j) old[j] = (c0 + j < p.n) ? __ldcg(xr + j * m) : 0.f;
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = (c0 + j < p.n) ? v[j] + old[j] : 0.f;
        }
        const float g = __half2float(__ldg((const __half*)e.gain + f));
#pragma unroll
        for (int j = 0; j < 32; ++j)
            if (c0 + j < p.n) {
                xr[j * m] = v[j];
                xg[j * m] = __float2half_rn(v[j] * g);
                v[j] *= v[j];
            }
        sm->ssq_part[grp][quad][lane] = warp_transpose_sum(v, lane);
        grp_bar(grp);
        if (quad == 0 && c0 + lane < p.n)
            e.ssq_out[(size_t)tile * SSQ_PITCH + c0 + lane] =
                (sm->ssq_part[grp][0][lane] + sm->ssq_part[grp][1][lane]) + (sm->ssq_part[grp][2][lane] + sm->ssq_part[grp][3][lane]);
        grp_bar(grp);
        return;
    }
    if (e.mode == EPI_RAW || e.mode == EPI_RESID) {
        const int f = tile * TILE_M + row;
        if (f < p.m) {
            float* dst = e.out_f32 + (size_t)c0 * p.m + f;
            if (e.mode == EPI_RESID) {
                // all loads first, then all stores: a load placed after a store through another
                // pointer would have to wait for it, turning 32 round trips into a chain
                float old[32];
#pragma unroll
                for (int j = 0; j < 32; ++j) old[j] = (c0 + j < p.n) ? __ldcg(dst + (size_t)j * p.m) : 0.f;
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] += old[j];
            }
#pragma unroll
            for (int j = 0; j < 32; ++j)
                if (c0 + j < p.n) dst[(size_t)j * p.m] = v[j];
        }
        return;
    }
    if (e.mode == EPI_SWIGLU) {
        // rows 0..63: gate pre-activations of features tile*64 + row; rows 64..127: the matching up rows.
        // Per pass thread `row` finishes XR/2 nodes of feature row & 63 (inputs gathered first, stores last:
        // a store between two loads would serialise them, the compiler cannot prove the pointers distinct).
        constexpr int HALF = XR / 2;
        const int f = row & 63, jb = (row >> 6) * HALF;
        __half res[PASSES * HALF];
#pragma unroll
        for (int hh = 0; hh < PASSES; ++hh) {
#pragma unroll
            for (int j = 0; j < XR; ++j) xb[j][row] = v[hh * XR + j];
            grp_bar(grp);
#pragma unroll
            for (int j = 0; j < HALF; ++j) {      // SiLU(g) * up = g * up / (1 + 2^(-g log2 e))
                const float g = xb[jb + j][f], up = xb[jb + j][f + 64];
                res[hh * HALF + j] = __float2half_rn(__fdividef(g * up, 1.f + exp2f(-1.4426950408889634f * g)));
            }
            grp_bar(grp);
        }
        __half* u = (__half*)e.out_t + (size_t)(c0 + jb) * p.swiglu_f + tile * 64 + f;
#pragma unroll
        for (int hh = 0; hh < PASSES; ++hh)
#pragma unroll
            for (int j = 0; j < HALF; ++j)
                if (c0 + hh * XR + jb + j < p.n) u[(size_t)(hh * XR + j) * p.swiglu_f] = res[hh * HALF + j];
        return;
    }
    // EPI_ROPE_KV: output features [0,d) = q, [d,2d) = k, [2d,3d) = v; tiles never straddle sections
    const int d = e.d_model, dh = e.d_head, half = dh >> 1;
    const int kv_len = resolve_kv_len(e.kv_len, e.kv_len_dev, e.max_kv_len, p.n);
    const int f = tile * TILE_M + row;
    const int section = f / d, el = f - section * d;
    const int head = el / dh, idx = el - head * dh;
    if (section < 2) {
        const int prow = (idx < half) ? row + half : row - half;
        const int t = (idx < half) ? idx : idx - half;
        const float sign = (idx < half) ? -1.f : 1.f;
        // the table loads go out first so that their latency overlaps the exchange through shared memory
        float2 cs[32];
        const float2* tab = reinterpret_cast<const float2*>(e.rope + (size_t)c0 * dh + 2 * t);
#pragma unroll
        for (int j = 0; j < 32; ++j) cs[j] = (c0 + j < p.n) ? __ldg(tab + (size_t)j * half) : make_float2(1.f, 0.f);
#pragma unroll
        for (int hh = 0; hh < PASSES; ++hh) {
#pragma unroll
            for (int j = 0; j < XR; ++j) xb[j][row] = v[hh * XR + j];
            grp_bar(grp);
            float partner[XR];
#pragma unroll
            for (int j = 0; j < XR; ++j) partner[j] = xb[j][prow];
            grp_bar(grp);
#pragma unroll
            for (int j = 0; j < XR; ++j) v[hh * XR + j] = fmaf(sign * partner[j], cs[hh * XR + j].y, v[hh * XR + j] * cs[hh * XR + j].x);
        }
        __half* dst;
        size_t pitch;
        if (section == 0) { dst = (__half*)e.out_t + (size_t)c0 * d + el; pitch = (size_t)d; }
        else { dst = (__half*)e.k_cache + ((size_t)head * e.max_kv_len + kv_len + c0) * dh + idx; pitch = (size_t)dh; }
#pragma unroll
        for (int j = 0; j < 32; ++j)
            if (c0 + j < p.n) dst[(size_t)j * pitch] = __float2half_rn(v[j]);
    } else {
#pragma unroll
        for (int j = 0; j < 32; ++j) {
            const int node = c0 + j;
            if (node < p.n)
                ((__half*)e.v_cache)[((size_t)head * e.max_kv_len + kv_len + node) * dh + idx] = __float2half_rn(v[j]);
        }
    }
}

}  // namespace gemmdev

// Host: everything one projection launch needs.  `pending` describes the partial tiles an
// EPI_DEFER projection leaves behind (active = 0 for the other epilogues).
struct GemmPlan {
    gemmdev::GemmParams p;
    CUtensorMap tm_w, tm_x;
    size_t smem;
    PendingPartials pending;
};
ghd_status plan_gemm_tc(ghd_ctx* c, const void* x, const void* w, int n, int k, int m, const EpiArgs& epi, GemmPlan* plan);

}  // namespace ghd
