// A chain of dependent phases of one decoder layer in ONE persistent kernel (sm_100a):
// skinny projections on the tensor cores (the same tiles, stream-K split and fused epilogues
// as k_gemm_tc) interleaved with the element-wise phases between them (attention split merge,
// split-K fold + residual + RMSNorm).
//
// Why: a verify step of a tree of <= 256 nodes is bound by streaming the weights from HBM once.
// With one kernel per projection every kernel boundary stalls that stream: the ring of weight
// tiles in shared memory drains, the next kernel sets up, and the first loads pay full latency.
// Here the weights of ALL projections of the chain form one stream per CTA.  A dedicated
// producer thread keeps requesting weight tiles (constant data, no dependency) as fast as the ring
// frees slots, across phase boundaries; only the activation operand of a phase (small, L2
// resident) waits until the previous phase has finished on every CTA.  While the CTAs sit in a
// grid-wide dependency or run an element-wise phase, the ring (about 190 KB per SM, 28 MB per
// GPU) keeps HBM busy.
//
// Per CTA (one per SM, 224 threads): warp 0 = weight producer (TMA), warp 6 = activation
// producer (TMA, gated by the phase dependency), warp 1 = MMA issuer (tcgen05.mma) and TMEM
// owner, warps 2..5 = epilogue of the projections and all element-wise phases.
//
// Phase dependency: phase p may read what phase p-1 wrote once every CTA has counted itself in
// at sync[p-1] (release add after a CTA-wide barrier; acquire poll).  Activations written with
// ordinary stores are read back through TMA, so writers and readers also fence the async proxy.
// All CTAs of the grid must be resident together: the grid never exceeds the SM count and a CTA
// takes a whole SM; the launch asks for a cooperative grid so that the driver checks this.
// Every wait is bounded; on expiry the CTA records a status code, stops issuing, waits for its
// loads and MMAs in flight, frees its TMEM and returns, and the other CTAs follow.
#include <cuda.h>

#include <cstdio>
#include <cstring>

#include "gemm_tc_dev.cuh"

namespace ghd {

using namespace gemmdev;

namespace {

constexpr int CH_THREADS = 224;
constexpr int SSQ_TILES = 64;         // row stride of the per-tile mean-square shares: d_model <= 128 * SSQ_TILES
constexpr int TRACE_SLOTS = 8;

struct FoldArgs {
    float* xres;                      // [n][d] residual stream, updated in place
    const float* part;                // partial tiles of the projection folded in (gemm >= 0)
    const __half* g;                  // RMSNorm gain (h_out != null)
    __half* h_out;                    // [n][d] xres * g in storage type (the consumer applies 1/rms), or null
    float* ssq;                       // [n][SSQ_TILES] per-tile shares of the rows' sums of squares (h_out != null)
    __half* x_out;                    // [n][d] residual stream in storage type, or null
    int d, gemm;                      // gemm: index of the projection whose partial tiles are summed, -1 = none
    float eps;
    unsigned long long slot_elems;
};

struct CombineArgs {
    const float* part_o;              // [splits][max_nodes][d] attention numerators
    const float* part_ml;             // [splits][max_nodes][heads][2] running max / sum
    __half* out;                      // [n][d]
    int splits, heads, dh, max_nodes;
};

struct ChainParams {
    int n_phases, n, nb, stages, ks;
    int type[CHAIN_MAX_PHASES], arg[CHAIN_MAX_PHASES];
    int* sync;                        // [CHAIN_MAX_PHASES] phase arrival counters + exit counter; zero between launches
    int* status;
    long long* trace;                 // optional [CHAIN_MAX_PHASES + 1][grid][4] nanosecond stamps (diagnostics), or null
    CombineArgs comb;
    const float* ssq[CHAIN_MAX_GEMMS];   // per projection: shares of its input rows' sums of squares (scale columns by 1/rms), or null
    int norm_d;
    float norm_eps;
    FoldArgs f[CHAIN_MAX_FOLDS];
    GemmParams g[CHAIN_MAX_GEMMS];
};

struct alignas(64) ChainMaps {
    CUtensorMap w[CHAIN_MAX_GEMMS], x[CHAIN_MAX_GEMMS];
};

struct ChainSmem {
    Smem base;
    volatile int a_issued, b_issued;  // stages requested so far by the two producers (read on the abort path)
    int sync_ok;
    float colscale[GHD_MAX_NODES];    // 1/rms per node for the current projection
};

__device__ __forceinline__ long long global_ns() {
    long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async;" ::: "memory"); }

// One thread, after a CTA-wide barrier that follows every thread's global writes of the phase.
__device__ __forceinline__ void grid_arrive(int* counter) {
    __threadfence();
    asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(counter) : "memory");
}

// Bounded wait until `target` CTAs have counted themselves in.
__device__ __forceinline__ bool grid_wait(const int* counter, int target, volatile int* abort_flag, int* status) {
    for (uint32_t spin = 0; spin < SPIN_LIMIT; ++spin) {
        if (ld_acquire_gpu(counter) >= target) {
            fence_proxy_async();
            return true;
        }
        if (*abort_flag) return false;
        if ((spin & 1023u) == 1023u && ld_acquire_gpu(status) != DEV_OK) { *abort_flag = 1; return false; }   // another CTA gave up
        __nanosleep(spin > 4096 ? 256 : 64);
    }
    *abort_flag = 1;
    atomicCAS(status, DEV_OK, DEV_TIMEOUT_GRID);
    return false;
}

struct Range {
    long long it_beg, it_end;
    int tile, k0;
};

// CTA `cta` of the p.ctas that share a projection owns k-chunks [it_beg, it_end) of the flattened
// (tile, k-chunk) space; (tile, k0) is where it starts.
__device__ __forceinline__ Range cta_range(const GemmParams& p, int cta) {
    Range r;
    const long long total = (long long)p.n_tiles * p.kiters;
    r.it_beg = total * cta / p.ctas;
    r.it_end = total * (cta + 1) / p.ctas;
    r.tile = (int)(r.it_beg / p.kiters);
    r.k0 = (int)(r.it_beg - (long long)r.tile * p.kiters);
    return r;
}

// Walks one CTA's k-chunks through every projection of the chain, in execution order.
struct Cursor {
    int ph, gi, tile, kc, kiters, left, row_step;
};

__device__ __forceinline__ void cursor_init(Cursor& c) { c.ph = -1; c.left = 0; }

template <typename Params>
__device__ __forceinline__ bool cursor_next_phase(Cursor& c, const Params& P, int cta) {
    for (++c.ph; c.ph < P.n_phases; ++c.ph) {
        if (P.type[c.ph] != CHAIN_GEMM) continue;
        const GemmParams& p = P.g[P.arg[c.ph]];
        if (cta >= p.ctas) continue;
        const Range r = cta_range(p, cta);
        if (r.it_end <= r.it_beg) continue;
        c.gi = P.arg[c.ph];
        c.tile = r.tile;
        c.kc = r.k0;
        c.kiters = p.kiters;
        c.left = (int)(r.it_end - r.it_beg);
        c.row_step = p.swiglu_f ? 64 : TILE_M;
        return true;
    }
    return false;
}

template <typename Params>
__device__ __forceinline__ bool cursor_step(Cursor& c, const Params& P, int cta) {
    if (--c.left == 0) return cursor_next_phase(c, P, cta);
    if (++c.kc == c.kiters) { c.kc = 0; ++c.tile; }
    return true;
}

// ---------------------------------------------------------------- epilogue of one projection phase
// Same unit walk as k_gemm_tc: whole tiles go through the fused epilogue, partial tiles are
// stored (EPI_DEFER) or handed to whichever contributor arrives last.
__device__ __forceinline__ bool epilogue_phase(const GemmParams& p, Smem* sm, int cta, uint32_t tmem_base, uint32_t buf_cols,
                                               uint32_t& buf, uint32_t& buf_phase, int quad, int lane, int et,
                                               volatile int* abort_flag, const float* cscale, long long* tr) {
    const int row = quad * 32 + lane;
    const Range r = cta_range(p, cta);
    long long it = r.it_beg;
    const size_t slot_elems = (size_t)buf_cols * TILE_M;
    int tile = r.tile, k0 = r.k0;
    for (; it < r.it_end; ++tile, k0 = 0) {
        const long long left = r.it_end - it;
        const int k1 = (p.kiters - k0 < left) ? p.kiters : (int)(k0 + left);
        const bool whole = (k0 == 0 && k1 == p.kiters) && p.epi.mode != EPI_DEFER;
        mbar_wait(smem_u32(&sm->tmem_full[buf]), buf_phase, abort_flag, p.status, DEV_TIMEOUT_EPI);
        epi_bar();                                             // all 128 threads take the same decision
        if (*abort_flag != 0) return false;
        tc_fence_after();
        if (tr && et == 0) { if (it == r.it_beg) tr[7] = global_ns(); tr[1] = global_ns(); }
        const uint32_t t_addr = tmem_base + buf * buf_cols + ((uint32_t)(quad * 32) << 16);
        if (whole) {
            for (int c0 = 0; c0 < p.nb; c0 += EPI_CHUNK) {
                float v[32];
                tc_ld32(t_addr + c0, v);
                if (c0 < p.n) epilogue_chunk(p, sm, tile, row, c0, v, cscale);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sm->tmem_empty[buf]));
        } else {
            const int slot = (it == r.it_beg) ? 0 : 1;
            float* mine = p.part + ((size_t)cta * 2 + slot) * slot_elems;
            const int c_first = p.tile_first[tile], c_last = c_first + p.tile_count[tile] - 1;
            bool finish = false, dumped = false;
            if (p.epi.mode != EPI_DEFER) {
                if (et == 0) sm->last_flag = (ld_acquire_gpu(p.counters + tile) == c_last - c_first) ? 1 : 0;
                epi_bar();
                finish = sm->last_flag != 0;
                epi_bar();
            }
            if (!finish) {
                for (int c0 = 0; c0 < p.nb; c0 += EPI_CHUNK) {
                    float v[32];
                    tc_ld32(t_addr + c0, v);
#pragma unroll
                    for (int j = 0; j < 32; ++j) __stcg(mine + (size_t)(c0 + j) * TILE_M + row, v[j]);
                }
                dumped = true;
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&sm->tmem_empty[buf]));
                if (p.epi.mode != EPI_DEFER) {
                    epi_bar();
                    if (et == 0) sm->last_flag = (atom_add_acq_rel_gpu(p.counters + tile, 1) == c_last - c_first) ? 1 : 0;
                    epi_bar();
                    finish = sm->last_flag != 0;
                    epi_bar();
                }
            }
            if (finish) {
                for (int c0 = 0; c0 < p.nb && c0 < p.n; c0 += EPI_CHUNK) {
                    float v[32], own[32];
                    if (!dumped) tc_ld32(t_addr + c0, own);
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = 0.f;
                    for (int c = c_first; c <= c_last; ++c) {      // CTA order: reproducible sums
                        if (c == cta && !dumped) {
#pragma unroll
                            for (int j = 0; j < 32; ++j) v[j] += own[j];
                            continue;
                        }
                        const int cslot = (c == c_first) ? p.tile_slot[tile] : 0;
                        const float* src = p.part + ((size_t)c * 2 + cslot) * slot_elems + (size_t)c0 * TILE_M + row;
                        float t[32];
#pragma unroll
                        for (int j = 0; j < 32; ++j) t[j] = __ldcg(src + (size_t)j * TILE_M);
#pragma unroll
                        for (int j = 0; j < 32; ++j) v[j] += t[j];
                    }
                    epilogue_chunk(p, sm, tile, row, c0, v, cscale);
                }
                if (!dumped) {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&sm->tmem_empty[buf]));
                }
                if (et == 0) p.counters[tile] = 0;
            }
        }
        if (++buf == 2) { buf = 0; buf_phase ^= 1; }
        it += (k1 - k0);
    }
    return true;
}

// ---------------------------------------------------------------- element-wise phases (128 epilogue threads)
// Both phases deal (128-column tile, group of 16 nodes) units to the CTAs round robin, so that
// every SM takes part and a thread owns four float4 (one per node row r, r + 4, r + 8, r + 12 of the
// group) whose loads all go out together: with HBM saturated by the weight stream an L2 round
// trip costs more than a microsecond, and the phase is one round trip long.
__device__ __forceinline__ uint2 pack_half4(float a, float b, float c, float d) {
    const __half2 lo = __floats2half2_rn(a, b), hi = __floats2half2_rn(c, d);
    uint2 pk;
    pk.x = *reinterpret_cast<const uint32_t*>(&lo);
    pk.y = *reinterpret_cast<const uint32_t*>(&hi);
    return pk;
}

// xres += partial tiles of projection `gp` (contributors summed in CTA order); x_out = T(xres);
// h_out = T(xres * g), WITHOUT the 1/rms factor: the mean square of a row is only known once all
// its tiles are folded, so each unit leaves its share in ssq[node][tile] and the projection that
// consumes h_out scales its accumulator columns by rsqrt(sum_tiles ssq / d + eps) (the scale of a
// node is a factor of the whole row, so it commutes with the projection).
__device__ __forceinline__ void fold_phase(const FoldArgs& a, const GemmParams* gp, int n, int cta, int G, int et, int lane) {
    const int d = a.d, d_tiles = d >> 7;
    const int units = d_tiles * ((n + 15) >> 4);
    const int c4 = et & 31, r = et >> 5;
    for (int u = cta; u < units; u += G) {
        const int tile = u % d_tiles, group = u / d_tiles;
        const int col = tile * TILE_M + 4 * c4;
        float4 x[4];
        bool live[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int node = group * 16 + r + 4 * q;
            live[q] = node < n;
            x[q] = live[q] ? __ldcg(reinterpret_cast<const float4*>(a.xres + (size_t)node * d + col)) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
        uint2 gr = make_uint2(0u, 0u);
        if (a.h_out) gr = __ldg(reinterpret_cast<const uint2*>(a.g + col));
        if (gp) {
            const int c_first = gp->tile_first[tile], cnt = gp->tile_count[tile], slot0 = gp->tile_slot[tile];
            const float* base = a.part + (size_t)(group * 16 + r) * TILE_M + 4 * c4;
            float4 acc[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) acc[q] = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int c0 = 0; c0 < cnt; c0 += 8) {
                float4 t[8][4];
#pragma unroll
                for (int ci = 0; ci < 8; ++ci) {
                    const int c = c0 + ci;
                    const float* src = base + ((size_t)(c_first + c) * 2 + (c == 0 ? slot0 : 0)) * (size_t)a.slot_elems;
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        t[ci][q] = (c < cnt && live[q]) ? __ldcg(reinterpret_cast<const float4*>(src + (size_t)(4 * q) * TILE_M)) : make_float4(0.f, 0.f, 0.f, 0.f);
                }
#pragma unroll
                for (int ci = 0; ci < 8; ++ci)
#pragma unroll
                    for (int q = 0; q < 4; ++q) { acc[q].x += t[ci][q].x; acc[q].y += t[ci][q].y; acc[q].z += t[ci][q].z; acc[q].w += t[ci][q].w; }
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                x[q].x += acc[q].x; x[q].y += acc[q].y; x[q].z += acc[q].z; x[q].w += acc[q].w;
                if (live[q]) *reinterpret_cast<float4*>(a.xres + (size_t)(group * 16 + r + 4 * q) * d + col) = x[q];
            }
        }
        const float2 g01 = __half22float2(*reinterpret_cast<const __half2*>(&gr.x));
        const float2 g23 = __half22float2(*reinterpret_cast<const __half2*>(&gr.y));
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int node = group * 16 + r + 4 * q;
            if (a.x_out && live[q]) *reinterpret_cast<uint2*>(a.x_out + (size_t)node * d + col) = pack_half4(x[q].x, x[q].y, x[q].z, x[q].w);
            if (a.h_out) {
                if (live[q]) *reinterpret_cast<uint2*>(a.h_out + (size_t)node * d + col) = pack_half4(x[q].x * g01.x, x[q].y * g01.y, x[q].z * g23.x, x[q].w * g23.y);
                // the warp holds exactly this node's 128 columns of the tile: fixed-order tree sum
                float ss = x[q].x * x[q].x + x[q].y * x[q].y + x[q].z * x[q].z + x[q].w * x[q].w;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
                if (lane == 0 && live[q]) a.ssq[(size_t)node * SSQ_TILES + tile] = ss;
            }
        }
    }
}

// 1/rms of every node from the per-tile shares a fold phase left behind -> colscale[node] (shared memory).
__device__ __forceinline__ void norm_scales(const float* ssq, int d, float eps, int n, int et, float* colscale) {
    const int d_tiles = d >> 7;
    for (int node = et; node < n; node += 128) {
        float s = 0.f;
        for (int t0 = 0; t0 < d_tiles; t0 += 16) {
            float v[16];
#pragma unroll
            for (int t = 0; t < 16; ++t) v[t] = (t0 + t < d_tiles) ? __ldcg(ssq + (size_t)node * SSQ_TILES + t0 + t) : 0.f;
#pragma unroll
            for (int t = 0; t < 16; ++t) s += v[t];
        }
        colscale[node] = rsqrtf(s / (float)d + eps);
    }
}

// Online-softmax merge of the attention KV splits (paper Sec. III-B-2): out = sum_s w_s o_s / sum_s w_s l_s
// with w_s = exp(m_s - max m).
__device__ __forceinline__ void combine_phase(const CombineArgs& a, int n, int cta, int G, int et) {
    const int d = a.heads * a.dh, d_tiles = d >> 7;
    const int units = d_tiles * ((n + 15) >> 4);
    const int c4 = et & 31, r = et >> 5;
    for (int u = cta; u < units; u += G) {
        const int tile = u % d_tiles, group = u / d_tiles;
        const int col = tile * TILE_M + 4 * c4, h = col / a.dh;
        float m[4], den[4];
        float4 acc[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) { m[q] = -INFINITY; den[q] = 0.f; acc[q] = make_float4(0.f, 0.f, 0.f, 0.f); }
        for (int s0 = 0; s0 < a.splits; s0 += 4) {
            float2 ml[4][4];
            float4 ov[4][4];
#pragma unroll
            for (int s = 0; s < 4; ++s)
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const int node = group * 16 + r + 4 * q;
                    ml[s][q] = make_float2(-INFINITY, 0.f);
                    ov[s][q] = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (node < n && s0 + s < a.splits) {
                        ml[s][q] = __ldcg(reinterpret_cast<const float2*>(a.part_ml + (((size_t)(s0 + s) * a.max_nodes + node) * a.heads + h) * 2));
                        ov[s][q] = __ldcg(reinterpret_cast<const float4*>(a.part_o + ((size_t)(s0 + s) * a.max_nodes + node) * d + col));
                    }
                }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                float m_new = m[q];
#pragma unroll
                for (int s = 0; s < 4; ++s) m_new = fmaxf(m_new, ml[s][q].x);
                if (m_new == -INFINITY) continue;
                const float rescale = (m[q] == -INFINITY) ? 0.f : expf(m[q] - m_new);
                den[q] *= rescale; acc[q].x *= rescale; acc[q].y *= rescale; acc[q].z *= rescale; acc[q].w *= rescale;
#pragma unroll
                for (int s = 0; s < 4; ++s) {
                    if (ml[s][q].x == -INFINITY) continue;
                    const float w = expf(ml[s][q].x - m_new);
                    den[q] += ml[s][q].y * w;
                    acc[q].x += ov[s][q].x * w; acc[q].y += ov[s][q].y * w; acc[q].z += ov[s][q].z * w; acc[q].w += ov[s][q].w * w;
                }
                m[q] = m_new;
            }
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int node = group * 16 + r + 4 * q;
            if (node < n) {
                const float inv = 1.f / den[q];
                *reinterpret_cast<uint2*>(a.out + (size_t)node * d + col) = pack_half4(acc[q].x * inv, acc[q].y * inv, acc[q].z * inv, acc[q].w * inv);
            }
        }
    }
}

// ---------------------------------------------------------------- kernel
__global__ void __launch_bounds__(CH_THREADS, 1)
k_chain_tc(const __grid_constant__ ChainMaps maps, const __grid_constant__ ChainParams P) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t pad = (1024u - (raw_addr & 1023u)) & 1023u;
    uint8_t* tiles = smem_raw + pad;
    const uint32_t a_slab = TILE_M * TILE_K * 2, b_slab = (uint32_t)P.nb * TILE_K * 2;
    const uint32_t a_bytes = P.ks * a_slab, b_bytes = P.ks * b_slab;
    const uint32_t stage_bytes = a_bytes + b_bytes;
    ChainSmem* cs = reinterpret_cast<ChainSmem*>(tiles + (size_t)P.stages * stage_bytes);
    Smem* sm = &cs->base;
    const uint32_t tiles_addr = smem_u32(tiles);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = gridDim.x, cta = blockIdx.x;

    const uint32_t buf_cols = (uint32_t)((P.nb + EPI_CHUNK - 1) / EPI_CHUNK * EPI_CHUNK);
    uint32_t tmem_cols = 32;
    while (tmem_cols < 2u * buf_cols) tmem_cols <<= 1;

    if (threadIdx.x == 32) {
        for (int ph = 0; ph < P.n_phases; ++ph)
            if (P.type[ph] == CHAIN_GEMM) {
                asm volatile("prefetch.tensormap [%0];" ::"l"(&maps.w[P.arg[ph]]) : "memory");
                asm volatile("prefetch.tensormap [%0];" ::"l"(&maps.x[P.arg[ph]]) : "memory");
            }
    }
    if (threadIdx.x == 0) {
        for (int s = 0; s < P.stages; ++s) { mbar_init(smem_u32(&sm->full[s]), 2); mbar_init(smem_u32(&sm->empty[s]), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(smem_u32(&sm->tmem_full[b]), 1); mbar_init(smem_u32(&sm->tmem_empty[b]), 4); }
        mbar_init(smem_u32(&sm->drain), 1);
        sm->abort_flag = 0;
        sm->last_flag = 0;
        cs->a_issued = 0;
        cs->b_issued = 0;
        cs->sync_ok = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm->tmem_base)), "r"(tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = sm->tmem_base;
    volatile int* abort_flag = &sm->abort_flag;
    if (threadIdx.x == 0) pdl_trigger();
    if (P.trace && threadIdx.x == 0) P.trace[((size_t)CHAIN_MAX_PHASES * G + cta) * TRACE_SLOTS] = global_ns();

    if (warp == 0) {
        // ------------------------------------------------ weight producer: one stream over all projections
        if (lane == 0) {
            uint64_t pol_stream;
            asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol_stream));
            uint32_t stage = 0, phase = 0;
            int issued = 0;
            bool ok = true;
            Cursor ld;
            cursor_init(ld);
            bool live = cursor_next_phase(ld, P, cta);
            int traced_ph = -1;
            while (live) {
                if (issued >= P.stages) ok = mbar_wait(smem_u32(&sm->empty[stage]), phase ^ 1, abort_flag, P.status, DEV_TIMEOUT_TMA);
                if (!ok) break;
                if (P.trace && traced_ph != ld.ph) { traced_ph = ld.ph; P.trace[((size_t)ld.ph * G + cta) * TRACE_SLOTS + 4] = global_ns(); }
                const uint32_t full = smem_u32(&sm->full[stage]);
                mbar_expect_tx(full, a_bytes);
                tma_load_4d(tiles_addr + stage * stage_bytes, &maps.w[ld.gi], 0, ld.tile * ld.row_step, 0, ld.kc * P.ks, full, pol_stream);
                cs->a_issued = ++issued;
                if (++stage == (uint32_t)P.stages) { stage = 0; phase ^= 1; }
                if (P.trace && ld.left == 1) P.trace[((size_t)ld.ph * G + cta) * TRACE_SLOTS + 5] = global_ns();
                live = cursor_step(ld, P, cta);
            }
        }
    } else if (warp == 6) {
        // ------------------------------------------------ activation producer: waits for the phase's input
        if (lane == 0) {
            pdl_wait();
            uint64_t pol_keep;
            asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol_keep));
            uint32_t stage = 0, phase = 0;
            int issued = 0;
            bool ok = true;
            for (int ph = 0; ph < P.n_phases && ok; ++ph) {
                if (P.type[ph] != CHAIN_GEMM) continue;
                const int gi = P.arg[ph];
                const GemmParams& p = P.g[gi];
                if (cta >= p.ctas) continue;
                if (ph > 0) {
                                ok = grid_wait(P.sync + ph - 1, G, abort_flag, P.status);
                }
                if (!ok) break;
                if (P.trace) P.trace[((size_t)ph * G + cta) * TRACE_SLOTS + 3] = global_ns();
                const Range r = cta_range(p, cta);
                int kc = r.k0;
                const int my_iters = (int)(r.it_end - r.it_beg);
                for (int i = 0; i < my_iters; ++i) {
                    if (issued >= P.stages) ok = mbar_wait(smem_u32(&sm->empty[stage]), phase ^ 1, abort_flag, P.status, DEV_TIMEOUT_TMA);
                    if (!ok) break;
                    const uint32_t full = smem_u32(&sm->full[stage]);
                    mbar_expect_tx(full, b_bytes);
                    tma_load_4d(tiles_addr + stage * stage_bytes + a_bytes, &maps.x[gi], 0, 0, 0, kc * P.ks, full, pol_keep);
                    cs->b_issued = ++issued;
                    if (++stage == (uint32_t)P.stages) { stage = 0; phase ^= 1; }
                    if (++kc == p.kiters) kc = 0;
                }
                if (P.trace) P.trace[((size_t)ph * G + cta) * TRACE_SLOTS + 6] = global_ns();
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idesc = instr_desc_f16(P.nb);
            uint32_t stage = 0, phase = 0, buf = 0, buf_phase = 0;
            long long units = 0;
            bool ok = true;
            for (int ph = 0; ph < P.n_phases && ok; ++ph) {
                if (P.type[ph] != CHAIN_GEMM) continue;
                const GemmParams& p = P.g[P.arg[ph]];
                if (cta >= p.ctas) continue;
                const Range r = cta_range(p, cta);
                long long it = r.it_beg;
                int k0 = r.k0;
                while (it < r.it_end && ok) {
                    const long long left = r.it_end - it;
                    const int k1 = (p.kiters - k0 < left) ? p.kiters : (int)(k0 + left);
                    if (units >= 2) ok = mbar_wait(smem_u32(&sm->tmem_empty[buf]), buf_phase ^ 1, abort_flag, P.status, DEV_TIMEOUT_TMEM);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t d_tmem = tmem_base + buf * buf_cols;
                    for (int kc = k0; kc < k1; ++kc) {
                        ok = mbar_wait(smem_u32(&sm->full[stage]), phase, abort_flag, P.status, DEV_TIMEOUT_MMA);
                        if (!ok) break;
                        tc_fence_after();
                        const uint32_t a_addr = tiles_addr + stage * stage_bytes, b_addr = a_addr + a_bytes;
                        const int nslab = (p.kslabs - kc * P.ks < P.ks) ? p.kslabs - kc * P.ks : P.ks;
                        for (int sl = 0; sl < nslab; ++sl) {
                            const uint64_t adesc = smem_desc_sw128(a_addr + sl * a_slab), bdesc = smem_desc_sw128(b_addr + sl * b_slab);
#pragma unroll
                            for (int j = 0; j < TILE_K / UMMA_K; ++j)
                                tc_mma_f16(d_tmem, adesc + (uint64_t)(j * 2), bdesc + (uint64_t)(j * 2), idesc, (kc > k0 || sl > 0 || j > 0) ? 1u : 0u);
                        }
                        tc_commit(smem_u32(&sm->empty[stage]));
                        if (++stage == (uint32_t)P.stages) { stage = 0; phase ^= 1; }
                    }
                    if (!ok) break;
                    tc_commit(smem_u32(&sm->tmem_full[buf]));
                    ++units;
                    if (++buf == 2) { buf = 0; buf_phase ^= 1; }
                    it += (k1 - k0);
                    k0 = 0;
                }
            }
            if (!ok) {
                tc_commit(smem_u32(&sm->drain));
                for (uint32_t spin = 0; spin < SPIN_LIMIT && !mbar_try(smem_u32(&sm->drain), 0); ++spin) __nanosleep(64);
            }
        }
    } else {
        // ------------------------------------------------ epilogue / element-wise warps
        const int quad = warp & 3;
        const int et = threadIdx.x - 64;
        pdl_wait();
        uint32_t buf = 0, buf_phase = 0;
        bool ok = true;
        for (int ph = 0; ph < P.n_phases && ok; ++ph) {
            const int type = P.type[ph], arg = P.arg[ph];
            long long* tr = P.trace ? P.trace + ((size_t)ph * G + cta) * TRACE_SLOTS : nullptr;
            if (tr && et == 0) tr[0] = global_ns();
            if (type == CHAIN_GEMM) {
                const GemmParams& p = P.g[arg];
                if (cta < p.ctas) {
                    const float* cscale = nullptr;
                    if (P.ssq[arg]) {
                        // the rows' mean squares are complete once the fold phase before this one is
                        if (ph > 0) {
                            if (et == 0) cs->sync_ok = grid_wait(P.sync + ph - 1, G, abort_flag, P.status) ? 1 : 0;
                            epi_bar();
                            ok = cs->sync_ok != 0;
                            epi_bar();
                        }
                        if (ok) {
                            norm_scales(P.ssq[arg], P.norm_d, P.norm_eps, P.n, et, cs->colscale);
                            epi_bar();
                            cscale = cs->colscale;
                        }
                    }
                    if (ok) ok = epilogue_phase(p, sm, cta, tmem_base, buf_cols, buf, buf_phase, quad, lane, et, abort_flag, cscale, tr);
                }
            } else if (cta < (P.norm_d >> 7) * ((P.n + 15) >> 4)) {
                if (ph > 0) {
                    if (et == 0) cs->sync_ok = grid_wait(P.sync + ph - 1, G, abort_flag, P.status) ? 1 : 0;
                    epi_bar();
                    ok = cs->sync_ok != 0;
                    epi_bar();
                }
                if (tr && et == 0) tr[1] = global_ns();
                if (ok) {
                    if (type == CHAIN_FOLD) {
                        const FoldArgs& a = P.f[arg];
                        fold_phase(a, a.gemm >= 0 ? &P.g[a.gemm] : nullptr, P.n, cta, G, et, lane);
                    } else {
                        combine_phase(P.comb, P.n, cta, G, et);
                    }
                }
            }
            if (!ok) break;
            if (ph + 1 < P.n_phases) {
                fence_proxy_async();          // this thread's stores, before TMA reads them elsewhere
                epi_bar();
                if (et == 0) grid_arrive(P.sync + ph);
            }
            if (tr && et == 0) tr[2] = global_ns();
        }
    }

    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0) {
        if (*abort_flag) {
            // A stage may hold only one of its two loads: stand in for the missing producer so that
            // the stage's barrier completes when the issued load lands, then wait for every load in flight.
            const int na = cs->a_issued, nb_ = cs->b_issued;
            const int lo = na < nb_ ? na : nb_, hi = na < nb_ ? nb_ : na;
            for (int j = lo; j < hi; ++j) mbar_arrive(smem_u32(&sm->full[j % P.stages]));
            for (int j = (hi > P.stages ? hi - P.stages : 0); j < hi; ++j) {
                const uint32_t bar = smem_u32(&sm->full[j % P.stages]), par = (uint32_t)(j / P.stages) & 1u;
                for (uint32_t spin = 0; spin < SPIN_LIMIT && !mbar_try(bar, par); ++spin) __nanosleep(64);
            }
        }
        // the last CTA out clears the phase counters for the next launch: by then nobody polls them
        if (atom_add_acq_rel_gpu(P.sync + CHAIN_MAX_PHASES, 1) == G - 1) {
            for (int ph = 0; ph <= CHAIN_MAX_PHASES; ++ph) P.sync[ph] = 0;
            __threadfence();
        }
    }
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
    }
}

size_t chain_smem_bytes(int nb, int ks, int stages) {
    return 1024 + (size_t)stages * ks * (TILE_M * TILE_K * 2 + (size_t)nb * TILE_K * 2) + sizeof(ChainSmem);
}

}  // namespace

bool chain_supported(const ghd_ctx* c, int n) {
    if (c->cfg.dtype != GHD_F16 || n < 1 || n > GHD_MAX_NODES) return false;
    if (c->cfg.d_model % 128 || c->cfg.d_model > 128 * SSQ_TILES) return false;
    return c->sm_count >= 1;
}

ghd_status launch_chain(ghd_ctx* c, const ChainPhase* phases, int count, int n) {
    if (count < 1 || count > CHAIN_MAX_PHASES) return GHD_EINVAL;
    ChainParams P{};
    ChainMaps M{};
    P.n_phases = count;
    P.n = n;
    P.nb = ((n + 15) / 16) * 16;
    P.sync = c->counters + CHAIN_SYNC_OFFSET;
    P.status = c->status;
    P.trace = c->trace;
    P.norm_d = c->cfg.d_model;
    P.norm_eps = c->cfg.rms_eps;
    int n_gemm = 0, n_fold = 0, n_comb = 0, last_defer = -1, grid = 1;
    bool h_unscaled = false;      // hbuf holds xres * g without the 1/rms factor
    for (int i = 0; i < count; ++i) {
        const ChainPhase& ph = phases[i];
        P.type[i] = ph.type;
        if (ph.type == CHAIN_GEMM) {
            if (n_gemm == CHAIN_MAX_GEMMS) return GHD_EINVAL;
            GemmPlan plan;
            const ghd_status s = plan_gemm_tc(c, ph.x, ph.w, n, ph.k, ph.m, ph.epi, &plan);
            if (s != GHD_OK) return s;
            P.g[n_gemm] = plan.p;
            M.w[n_gemm] = plan.tm_w;
            M.x[n_gemm] = plan.tm_x;
            P.ks = plan.p.ks;
            if (plan.p.ctas > grid) grid = plan.p.ctas;
            if (ph.epi.mode == EPI_DEFER) last_defer = n_gemm;
            P.ssq[n_gemm] = (h_unscaled && ph.x == c->hbuf) ? c->ssq : nullptr;
            P.arg[i] = n_gemm++;
        } else if (ph.type == CHAIN_FOLD) {
            if (n_fold == CHAIN_MAX_FOLDS) return GHD_EINVAL;
            FoldArgs& f = P.f[n_fold];
            f.xres = c->xres;
            f.part = c->gemm_part;
            f.g = (const __half*)ph.gain;
            f.h_out = ph.gain ? (__half*)ph.h_out : nullptr;
            f.x_out = (__half*)ph.x_out;
            f.ssq = c->ssq;
            if (f.h_out) h_unscaled = true;
            f.d = c->cfg.d_model;
            f.eps = c->cfg.rms_eps;
            f.gemm = ph.fold_partials ? last_defer : -1;
            if (ph.fold_partials && last_defer < 0) return GHD_EINVAL;
            f.slot_elems = (unsigned long long)((P.nb + EPI_CHUNK - 1) / EPI_CHUNK * EPI_CHUNK) * TILE_M;
            last_defer = ph.fold_partials ? -1 : last_defer;
            P.arg[i] = n_fold++;
        } else if (ph.type == CHAIN_COMBINE) {
            if (n_comb++) return GHD_EINVAL;
            P.comb.part_o = c->att_o;
            P.comb.part_ml = c->att_ml;
            P.comb.out = (__half*)ph.x_out;
            P.comb.splits = ph.splits;
            P.comb.heads = c->cfg.n_heads;
            P.comb.dh = c->cfg.d_head;
            P.comb.max_nodes = c->cfg.max_nodes;
        } else {
            return GHD_EINVAL;
        }
    }
    if (n_gemm == 0) return GHD_EINVAL;
    if (grid > c->sm_count) return GHD_EUNSUPPORTED;
    int stages = MAX_STAGES;
    while (stages > 2 && chain_smem_bytes(P.nb, P.ks, stages) > 227 * 1024) --stages;
    P.stages = stages;
    const size_t smem = chain_smem_bytes(P.nb, P.ks, stages);
    static bool attr_set = false;
    if (!attr_set) {
        if (cudaFuncSetAttribute(k_chain_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess) {
            snprintf(c->err, sizeof(c->err), "projection chain: cannot raise dynamic shared memory: %s", cudaGetErrorString(cudaGetLastError()));
            return GHD_ECUDA;
        }
        attr_set = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(CH_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = c->cur;
    cudaLaunchAttribute attr[2];
    int na = 0;
    if (!c->opt_no_pdl) {
        attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[na].val.programmaticStreamSerializationAllowed = 1;
        ++na;
    }
    if (c->opt_chain_coop != 1) {
        attr[na].id = cudaLaunchAttributeCooperative;
        attr[na].val.cooperative = 1;
        ++na;
    }
    cfg.attrs = attr;
    cfg.numAttrs = na;
    c->launches++;
    c->path_count[GHD_PATH_CHAIN]++;
    if (cudaLaunchKernelEx(&cfg, k_chain_tc, M, P) != cudaSuccess) {
        snprintf(c->err, sizeof(c->err), "projection chain: launch failed: %s", cudaGetErrorString(cudaGetLastError()));
        return GHD_ECUDA;
    }
    c->pending.active = 0;
    return GHD_OK;
}

}  // namespace ghd
