// Skinny projection GEMM on the 5th-generation tensor cores (sm_100a), half in,
// float accumulate:  Y[n][m] = X[n][k] * W[m][k]^T  with n <= 256 tree nodes.
//
// The problem is transposed for the hardware ("swap A/B"): a tile is 128 output
// features (rows of W, the MMA M dimension) by all NB = roundup16(n) nodes (the
// MMA N dimension), so each weight byte is fetched from HBM exactly once and the
// node columns stay on-chip.  The accumulator tile [128 x NB] float lives in
// tensor memory (TMEM), double-buffered so that the epilogue of one tile overlaps
// the MMAs of the next.
//
// Work split (stream-K): the (tile, 64-wide k-step) iteration space is flattened
// and cut into equal contiguous ranges, one per CTA (one CTA per SM), so every SM
// streams the same number of weight bytes whatever the tile count.  A CTA whose
// range covers only part of a tile's k-steps writes its float partial tile to the
// workspace and bumps the tile's arrival counter; the tile's first contributor (for
// which the tile comes last) keeps its share in tensor memory, waits - bounded - for
// that counter, sums the partials in CTA order (fixed order -> bit-reproducible) and
// runs the epilogue.  Contributors that store never wait.
//
// Per CTA: warp 0 = TMA producer (weights and activations into a ring of
// 128B-swizzled shared-memory stages), warp 1 = MMA issuer (tcgen05.mma, one
// thread) and TMEM owner, warps 2..5 = epilogue (tcgen05.ld, fused epilogue).
// All mbarrier waits are bounded: on expiry the kernel records a status code,
// stops issuing work, drains what it issued, frees its TMEM and returns.
#include <cuda.h>

#include <cstdio>
#include <cstring>

#include "gemm_tc_dev.cuh"

namespace ghd {

using namespace gemmdev;

namespace {

// ---------------------------------------------------------------- kernel
// TWO: eight epilogue warps in two groups (trees of more than 32 nodes: several 32-column chunks per tile);
// otherwise four epilogue warps, which a single chunk cannot keep more of busy and which leaves each thread
// the full register budget.
template <bool TWO>
__global__ void __launch_bounds__(TWO ? THREADS_TC : THREADS, 1)
k_gemm_tc(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_x, const GemmParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t pad = (1024u - (raw_addr & 1023u)) & 1023u;
    uint8_t* tiles = smem_raw + pad;
    const uint32_t a_slab = TILE_M * TILE_K * 2, b_slab = (uint32_t)p.nb * TILE_K * 2;
    const uint32_t a_bytes = p.ks * a_slab, b_bytes = p.ks * b_slab;
    const uint32_t stage_bytes = a_bytes + b_bytes;
    Smem* sm = reinterpret_cast<Smem*>(tiles + (size_t)p.stages * stage_bytes);
    const uint32_t tiles_addr = smem_u32(tiles);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = gridDim.x, cta = blockIdx.x;
    const long long total = (long long)p.n_tiles * p.kiters;
    const long long it_beg = total * cta / G, it_end = total * (cta + 1) / G;
    const int my_iters = (int)(it_end - it_beg);
    const int prefill = my_iters < p.stages ? my_iters : p.stages;    // weight stages requested during set-up

    // accumulator buffers are EPI_CHUNK-aligned so that a 32-column read never leaves the allocation
    const uint32_t buf_cols = (uint32_t)((p.nb + EPI_CHUNK - 1) / EPI_CHUNK * EPI_CHUNK);
    uint32_t tmem_cols = 32;
    while (tmem_cols < 2u * buf_cols) tmem_cols <<= 1;

    if (threadIdx.x == 32) {        // descriptor fetches overlap the barrier set-up
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_w) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_x) : "memory");
    }
    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) { mbar_init(smem_u32(&sm->full[s]), 1); mbar_init(smem_u32(&sm->empty[s]), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(smem_u32(&sm->tmem_full[b]), 1); mbar_init(smem_u32(&sm->tmem_empty[b]), TWO ? 8 : 4); }
        mbar_init(smem_u32(&sm->drain), 1);
        sm->abort_flag = 0;
        sm->last_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        // This thread is also the TMA producer.  Weights never change, so the first ring-full of weight
        // stages is requested right here: their latency overlaps the rest of the set-up (tensor-memory
        // allocation, CTA barrier) and the tail of the preceding kernel; the activations of those stages
        // follow after the dependency wait.
        uint64_t pol_first;
        asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol_first));
        int tile = (int)(it_beg / p.kiters), kc = (int)(it_beg - (long long)tile * p.kiters);
        for (int i = 0; i < prefill; ++i) {
            const uint32_t full = smem_u32(&sm->full[i]);
            mbar_expect_tx(full, stage_bytes);
            tma_load_4d(tiles_addr + i * stage_bytes, &tm_w, 0, p.swiglu_f ? tile * 64 : tile * TILE_M, 0, kc * p.ks, full, pol_first);
            if (++kc == p.kiters) { kc = 0; ++tile; }
        }
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
    if (threadIdx.x == 0) pdl_trigger();       // this CTA now owns its shared and tensor memory

    if (warp == 0) {
        // ------------------------------------------------ TMA producer
        if (lane == 0) {
            uint64_t pol_stream, pol_keep;
            asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol_stream));
            asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol_keep));
            uint32_t stage = 0, phase = 0;
            int issued = 0;
            bool ok = true;
            // (tile, kc) advance incrementally: a 64-bit division per stage would cost this single thread
            // more cycles than the loads it issues
            int tile = (int)(it_beg / p.kiters), kc = (int)(it_beg - (long long)tile * p.kiters);
            if (prefill > 0) {
                pdl_wait();                                    // the activations belong to the preceding kernel until now
                for (int q = 0; q < prefill; ++q) {            // activations of the stages whose weights went out during set-up
                    tma_load_4d(tiles_addr + q * stage_bytes + a_bytes, &tm_x, 0, 0, 0, kc * p.ks, smem_u32(&sm->full[q]), pol_keep);
                    if (++kc == p.kiters) { kc = 0; ++tile; }
                }
                issued = prefill;
                if (prefill == p.stages) phase = 1; else stage = (uint32_t)prefill;
            }
            for (int i = prefill; i < my_iters && ok; ++i) {
                ok = mbar_wait(smem_u32(&sm->empty[stage]), phase ^ 1, abort_flag, p.status, DEV_TIMEOUT_TMA);
                if (!ok) break;
                const uint32_t full = smem_u32(&sm->full[stage]);
                const uint32_t a_dst = tiles_addr + stage * stage_bytes, b_dst = a_dst + a_bytes;
                mbar_expect_tx(full, stage_bytes);
                tma_load_4d(a_dst, &tm_w, 0, p.swiglu_f ? tile * 64 : tile * TILE_M, 0, kc * p.ks, full, pol_stream);
                tma_load_4d(b_dst, &tm_x, 0, 0, 0, kc * p.ks, full, pol_keep);
                ++issued;
                if (++stage == (uint32_t)p.stages) { stage = 0; phase ^= 1; }
                if (++kc == p.kiters) { kc = 0; ++tile; }
            }
            if (!ok) {
                // drain: wait (bounded) until every load issued into the ring has landed
                const int inflight = issued < p.stages ? issued : p.stages;
                uint32_t s = stage, ph = phase;
                for (int q = 0; q < inflight; ++q) {
                    if (s == 0) { s = p.stages - 1; ph ^= 1; } else --s;
                    for (uint32_t spin = 0; spin < SPIN_LIMIT && !mbar_try(smem_u32(&sm->full[s]), ph); ++spin) __nanosleep(64);
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idesc = instr_desc_f16(p.nb);
            uint32_t stage = 0, phase = 0, buf = 0, buf_phase = 0;
            long long units = 0;
            bool ok = true;
            long long it = it_beg;
            int tile = (int)(it_beg / p.kiters), k0 = (int)(it_beg - (long long)tile * p.kiters);   // later units: next tile, k0 = 0
            while (it < it_end && ok) {
                const long long left = it_end - it;
                const int k1 = (p.kiters - k0 < left) ? p.kiters : (int)(k0 + left);
                if (units >= 2) ok = mbar_wait(smem_u32(&sm->tmem_empty[buf]), buf_phase ^ 1, abort_flag, p.status, DEV_TIMEOUT_TMEM);
                if (!ok) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * buf_cols;
                for (int kc = k0; kc < k1; ++kc) {
                    ok = mbar_wait(smem_u32(&sm->full[stage]), phase, abort_flag, p.status, DEV_TIMEOUT_MMA);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t a_addr = tiles_addr + stage * stage_bytes, b_addr = a_addr + a_bytes;
                    const int nslab = (p.kslabs - kc * p.ks < p.ks) ? p.kslabs - kc * p.ks : p.ks;   // the row's last chunk may be short
                    for (int sl = 0; sl < nslab; ++sl) {
                        const uint64_t adesc = smem_desc_sw128(a_addr + sl * a_slab), bdesc = smem_desc_sw128(b_addr + sl * b_slab);
#pragma unroll
                        for (int j = 0; j < TILE_K / UMMA_K; ++j)   // +32 bytes along k inside the swizzle row per step
                            tc_mma_f16(d_tmem, adesc + (uint64_t)(j * 2), bdesc + (uint64_t)(j * 2), idesc, (kc > k0 || sl > 0 || j > 0) ? 1u : 0u);
                    }
                    tc_commit(smem_u32(&sm->empty[stage]));    // stage is free once these MMAs have read it
                    if (++stage == (uint32_t)p.stages) { stage = 0; phase ^= 1; }
                }
                if (!ok) break;
                tc_commit(smem_u32(&sm->tmem_full[buf]));       // accumulator complete
                ++units;
                if (++buf == 2) { buf = 0; buf_phase ^= 1; }
                it += (k1 - k0);
                ++tile;
                k0 = 0;
            }
            if (!ok) {
                // make sure no MMA is still running before TMEM goes away
                tc_commit(smem_u32(&sm->drain));
                for (uint32_t spin = 0; spin < SPIN_LIMIT && !mbar_try(smem_u32(&sm->drain), 0); ++spin) __nanosleep(64);
            }
        }
    } else {
        // ------------------------------------------------ epilogue warps 2..9 (TMEM lanes 32*(warp%4) ..), two groups:
        // group g = (warp - 2) / 4 takes the 32-column chunks g, g + 2, ... of every accumulator
        const int quad = warp & 3, grp = TWO ? (warp - 2) >> 2 : 0;
        constexpr int GROUPS = TWO ? 2 : 1;
        const int row = quad * 32 + lane;
        auto epi_all = [] { if (TWO) all_epi_bar(); else grp_bar(0); };
        auto fused = [&](int tile_, int c0_, float (&v_)[32]) { epilogue_chunk<GROUPS>(p, sm, grp, tile_, row, c0_, v_); };
        const int et = threadIdx.x - 64;                       // 0..255 among epilogue threads
        const size_t slot_elems = (size_t)buf_cols * TILE_M;   // columns padded to whole 32-wide chunks
        // Epilogue of a complete tile.  split = false: the accumulator holds the whole sum.  split = true: this CTA
        // (the tile's first contributor) has its share in tensor memory and adds the other contributors' partial
        // tiles from the workspace in CTA order (fixed order -> reproducible); each one's 32 loads go out together.
        auto finish_tile = [&](int tile_, uint32_t t_addr_, bool split, int c_first_, int c_last_) {
            for (int c0 = grp * EPI_CHUNK; c0 < p.nb && c0 < p.n; c0 += GROUPS * EPI_CHUNK) {
                float v[32];
                tc_ld32(t_addr_ + c0, v);                  // may run past nb, never past the buffer
                if (split) {
                    for (int c = c_first_ + 1; c <= c_last_; ++c) {      // later contributors always use their slot 0
                        const float* src = p.part + (size_t)c * 2 * slot_elems + (size_t)c0 * TILE_M + row;
                        float t[32];
#pragma unroll
                        for (int j = 0; j < 32; ++j) t[j] = __ldcg(src + (size_t)j * TILE_M);
#pragma unroll
                        for (int j = 0; j < 32; ++j) v[j] += t[j];
                    }
                }
                fused(tile_, c0, v);
            }
        };
        pdl_wait();                                            // outputs, residual and partial buffers belong to earlier kernels until now
        if (p.epi.ssq_in) {
            // 1 / rms of every input row from the per-tile sums of squares its producer left (fixed order)
            for (int i = et; i < p.nb; i += TWO ? 256 : 128) {
                float s = 0.f;
                if (i < p.n)
                    for (int t0 = 0; t0 < p.epi.ssq_in_tiles; t0 += 8) {
                        float part[8];
#pragma unroll
                        for (int q = 0; q < 8; ++q)
                            part[q] = (t0 + q < p.epi.ssq_in_tiles) ? __ldcg(p.epi.ssq_in + (size_t)(t0 + q) * SSQ_PITCH + i) : 0.f;
#pragma unroll
                        for (int q = 0; q < 8; ++q) s += part[q];
                    }
                sm->colscale[i] = rsqrtf(s / (float)p.k + p.epi.rms_eps);
            }
            epi_all();
        }
        uint32_t buf = 0, buf_phase = 0;
        bool ok = true;
        long long it = it_beg;
        int tile = (int)(it_beg / p.kiters), k0 = (int)(it_beg - (long long)tile * p.kiters);
        for (; it < it_end && ok; ++tile, k0 = 0) {
            const long long left = it_end - it;
            const int k1 = (p.kiters - k0 < left) ? p.kiters : (int)(k0 + left);
            const bool whole = (k0 == 0 && k1 == p.kiters) && p.epi.mode != EPI_DEFER;
            mbar_wait(smem_u32(&sm->tmem_full[buf]), buf_phase, abort_flag, p.status, DEV_TIMEOUT_EPI);
            epi_all();                                     // all 256 threads take the same decision
            ok = (*abort_flag == 0);
            if (!ok) break;
            tc_fence_after();
            const uint32_t t_addr = tmem_base + buf * buf_cols + ((uint32_t)(quad * 32) << 16);
            // A tile some CTAs share is finished by its FIRST contributor: for that CTA the tile is the last unit of
            // its range, so it gets here last in time, while every other contributor handles its share as the first
            // unit of its range (or as its only one), stores it and counts itself in without ever waiting.  The
            // finisher keeps its own share in tensor memory and waits (bounded) for the others; they run at the same
            // time on other SMs and depend on nobody, so the wait is short: the store and count of a contributor
            // that ended together with the finisher.
            const int c_first = p.tile_first[tile], c_last = c_first + p.tile_count[tile] - 1;
            bool finish = whole;
            if (!whole && p.epi.mode != EPI_DEFER) {
                if (et == 0) {
                    int fl = 0;
                    if (cta == c_first) {
                        fl = 1;
                        uint32_t spin = 0;
                        while (ld_acquire_gpu(p.counters + tile) != c_last - c_first) {
                            if (++spin >= SPIN_LIMIT) { *abort_flag = 1; atomicCAS(p.status, DEV_OK, DEV_TIMEOUT_GRID); break; }
                            __nanosleep(spin > 64 ? 64 : 20);
                        }
                    }
                    sm->last_flag = fl;
                }
                epi_all();
                finish = sm->last_flag != 0;
                epi_all();
            }
            if (finish) {
                finish_tile(tile, t_addr, !whole, c_first, c_last);
                if (!whole && et == 0) p.counters[tile] = 0;   // ready for the next launch
            } else {
                // partial tile: slot 0 when this is the CTA's first unit (it starts mid-tile or is
                // its only unit of this tile), slot 1 when it is the head part of the CTA's last tile
                const int slot = (it == it_beg) ? 0 : 1;
                float* mine = p.part + ((size_t)cta * 2 + slot) * slot_elems;
                for (int c0 = grp * EPI_CHUNK; c0 < p.nb; c0 += GROUPS * EPI_CHUNK) {
                    float v[32];
                    tc_ld32(t_addr + c0, v);
#pragma unroll
                    for (int j = 0; j < 32; ++j) __stcg(mine + (size_t)(c0 + j) * TILE_M + row, v[j]);
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sm->tmem_empty[buf]));
            if (!finish && p.epi.mode != EPI_DEFER) {
                // count this arrival: the barrier orders every thread's stores before thread 0's
                // release, and the release is cumulative over them
                epi_all();
                if (et == 0) atom_add_acq_rel_gpu(p.counters + tile, 1);
            }
            if (++buf == 2) { buf = 0; buf_phase ^= 1; }
            it += (k1 - k0);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
    }
}

// ---------------------------------------------------------------- host side
size_t smem_bytes_for(int nb, int ks, int stages) {
    return 1024 + (size_t)stages * ks * (TILE_M * TILE_K * 2 + (size_t)nb * TILE_K * 2) + sizeof(Smem);
}

int pick_stages(int nb, int ks) {
    int s = MAX_STAGES;
    while (s > 2 && smem_bytes_for(nb, ks, s) > 227 * 1024) --s;
    return s;
}

}  // namespace

bool gemm_tc_supported(const ghd_ctx* c, int n, int k, int m, int epi_mode) {
    if (c->cfg.dtype != GHD_F16 || n < 1 || n > GHD_MAX_NODES || k % TILE_K || k < TILE_K) return false;
    const int n_tiles = (epi_mode == EPI_SWIGLU) ? (m / 2) / 64 : (m + TILE_M - 1) / TILE_M;
    if (n_tiles < 1 || n_tiles > MAX_TILES) return false;
    if (epi_mode == EPI_SWIGLU && (m / 2) % 64) return false;
    if (epi_mode == EPI_ROPE_KV && ((m / 3) % TILE_M || m % 3)) return false;
    if (epi_mode == EPI_RESID_NORM && (m % TILE_M || m / TILE_M > SSQ_MAX_TILES)) return false;
    if (epi_mode == EPI_DEFER) {
        int ctas = c->opt_gemm_ctas > 0 && c->opt_gemm_ctas < c->sm_count ? c->opt_gemm_ctas : c->sm_count;
        const int ks = (((n + 15) / 16) * 16 <= 128) ? 2 : 1;
        const int kch = (k / TILE_K + ks - 1) / ks;
        const long long total = (long long)n_tiles * kch;
        if (ctas > total) ctas = (int)total;
        if (m % 4 || m > 16384 || total / ctas + 1 > kch || total / ctas < 1) return false;
    }
    return true;
}

ghd_status plan_gemm_tc(ghd_ctx* c, const void* x, const void* w, int n, int k, int m, const EpiArgs& epi, GemmPlan* plan) {
    if (((uintptr_t)x & 15) || ((uintptr_t)w & 15)) {
        snprintf(c->err, sizeof(c->err), "tcgen05 GEMM: operands must be 16-byte aligned");
        return GHD_EINVAL;
    }
    GemmParams& p = plan->p;
    p = GemmParams{};
    p.n = n;
    p.nb = ((n + 15) / 16) * 16;
    p.k = k;
    p.m = m;
    p.swiglu_f = (epi.mode == EPI_SWIGLU) ? m / 2 : 0;
    p.n_tiles = p.swiglu_f ? p.swiglu_f / 64 : (m + TILE_M - 1) / TILE_M;
    p.ks = c->opt_gemm_burst > 0 ? c->opt_gemm_burst : (p.nb <= 128 ? 2 : 1);
    if (p.ks > 4) p.ks = 4;
    p.kslabs = k / TILE_K;
    p.kiters = (p.kslabs + p.ks - 1) / p.ks;
    p.stages = pick_stages(p.nb, p.ks);
    if (c->opt_gemm_stages >= 2 && c->opt_gemm_stages < p.stages) p.stages = c->opt_gemm_stages;
    p.part = c->gemm_part;
    p.counters = c->counters;
    p.status = c->status;
    p.epi = epi;
    if (!tmap_slabs(c, w, (uint64_t)m, (uint64_t)k, p.swiglu_f ? 2 : 1, p.swiglu_f ? 64 : TILE_M, (uint32_t)p.ks, &plan->tm_w) ||
        !tmap_slabs(c, x, (uint64_t)n, (uint64_t)k, 1, (uint32_t)p.nb, (uint32_t)p.ks, &plan->tm_x)) {
        snprintf(c->err, sizeof(c->err), "tcgen05 GEMM: tensor map encoding failed");
        return GHD_ECUDA;
    }
    const long long total = (long long)p.n_tiles * p.kiters;
    int ctas = c->opt_gemm_ctas > 0 ? c->opt_gemm_ctas : c->sm_count;
    if (ctas > c->sm_count) ctas = c->sm_count;
    if (c->opt_gemm_ctas <= 0 && epi.mode != EPI_DEFER && p.n_tiles < c->sm_count) {
        // Fewer tiles than SMs: every CTA range is shorter than a tile.  With n_tiles * q / (q - 1) CTAs each
        // range is (q-1)/q of a tile and always touches a tile boundary, so no tile is shared by three CTAs
        // and no CTA's only unit sits strictly inside a tile (those finish together and take the slow
        // split-tile path).  Take the largest such count that fits the SMs.
        int best = 0;
        for (int q = 2; q <= 64; ++q)
            if ((p.n_tiles * q) % (q - 1) == 0) {
                const int g = p.n_tiles * q / (q - 1);
                if (g <= c->sm_count && g > best) best = g;
            }
        if (best >= c->sm_count * 3 / 4) ctas = best;
    }
    if (ctas > total) ctas = (int)total;
    p.ctas = ctas;
    plan->smem = smem_bytes_for(p.nb, p.ks, p.stages);
    for (int t = 0; t < p.n_tiles; ++t) {
        const long long t_first = (long long)t * p.kiters;
        const int c_first = (int)(((t_first + 1) * ctas + total - 1) / total) - 1;
        const int c_last = (int)(((t_first + p.kiters) * ctas + total - 1) / total) - 1;
        p.tile_first[t] = (unsigned short)c_first;
        p.tile_count[t] = (unsigned char)(c_last - c_first + 1);
        p.tile_slot[t] = (total * c_first / ctas >= t_first) ? 0 : 1;
    }
    plan->pending.active = 0;
    if (epi.mode == EPI_DEFER) {
        if (total / ctas + 1 > p.kiters) {                // a CTA range must touch at most two tiles
            snprintf(c->err, sizeof(c->err), "tcgen05 GEMM: deferred reduction needs n_tiles <= CTAs");
            return GHD_EUNSUPPORTED;
        }
        PendingPartials& pp = plan->pending;
        pp.active = 1;
        pp.kiters = p.kiters;
        pp.ctas = ctas;
        pp.total = total;
        pp.slot_elems = (size_t)((p.nb + EPI_CHUNK - 1) / EPI_CHUNK * EPI_CHUNK) * TILE_M;
        pp.m = m;
        for (int t = 0; t < p.n_tiles && t < 128; ++t) {
            pp.first_cta[t] = p.tile_first[t];
            pp.n_contrib[t] = p.tile_count[t];
            pp.first_slot[t] = p.tile_slot[t];
        }
    }
    return GHD_OK;
}

ghd_status launch_gemm_tc(ghd_ctx* c, const void* x, const void* w, int n, int k, int m, const EpiArgs& epi) {
    GemmPlan plan;
    const ghd_status s = plan_gemm_tc(c, x, w, n, k, m, epi, &plan);
    if (s != GHD_OK) return s;
    if (!c->attr_gemm) {       // per context: the attribute belongs to the device the context was created on
        if (cudaFuncSetAttribute(k_gemm_tc<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess ||
            cudaFuncSetAttribute(k_gemm_tc<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess) {
            snprintf(c->err, sizeof(c->err), "tcgen05 GEMM: cannot raise dynamic shared memory: %s", cudaGetErrorString(cudaGetLastError()));
            return GHD_ECUDA;
        }
        c->attr_gemm = true;
    }
    if (plan.pending.active) c->pending = plan.pending;
    const bool two = c->opt_gemm_epi ? c->opt_gemm_epi == 2 : plan.p.nb > EPI_CHUNK;
    if (two) launch_k(c, true, k_gemm_tc<true>, plan.p.ctas, THREADS_TC, plan.smem, plan.tm_w, plan.tm_x, plan.p);
    else launch_k(c, true, k_gemm_tc<false>, plan.p.ctas, THREADS, plan.smem, plan.tm_w, plan.tm_x, plan.p);
    return GHD_OK;
}

}  // namespace ghd
