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
// workspace and bumps the tile's arrival counter; the contributor that completes its
// share of the tile last (chosen on the host from the ranges) keeps that share in
// tensor memory, waits - bounded - for the counter, adds the others' partials in CTA
// order (fixed order -> bit-reproducible) and runs the epilogue.  Contributors that
// store never wait.
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
// PAIR: the grid is made of clusters of two CTAs that work on two neighbouring 128-row weight tiles at once
// (tcgen05 cta_group::2, MMA M = 256): each CTA loads its own weight tile but only HALF of the activation rows;
// one thread of the even CTA issues the MMAs, which read both CTAs' shared memory and fill both CTAs' tensor
// memory.  A wide tree's activation slab (up to 32 KB per 64-wide k-step against 16 KB of weights) is then
// fetched once per 256 weight rows instead of once per 128.  Every CTA issues its own plain TMA loads (no
// multicast); the pair shares the ring's "full" barriers in the even CTA.  Work units ("wt") are tile pairs dealt to
// clusters; each CTA runs the epilogue of its own tile exactly as in the single-CTA kernel.
template <bool TWO, bool PAIR>
__global__ void __launch_bounds__(TWO ? THREADS_TC : THREADS, 1)
k_gemm_tc(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_x, const GemmParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t pad = (1024u - (raw_addr & 1023u)) & 1023u;
    uint8_t* tiles = smem_raw + pad;
    const int nb_cta = PAIR ? p.nb / 2 : p.nb;              // activation rows this CTA loads
    const uint32_t a_slab = TILE_M * TILE_K * 2, b_slab = (uint32_t)nb_cta * TILE_K * 2;
    const uint32_t a_bytes = p.ks * a_slab, b_bytes = p.ks * b_slab;
    const uint32_t stage_bytes = a_bytes + b_bytes;
    Smem* sm = reinterpret_cast<Smem*>(tiles + (size_t)p.stages * stage_bytes);
    const uint32_t tiles_addr = smem_u32(tiles);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int cta = blockIdx.x;
    const int rank = PAIR ? (int)cluster_ctarank() : 0;      // 0: the CTA that issues the pair's MMAs
    const int wk = PAIR ? cta >> 1 : cta;                   // this CTA's worker: a CTA, or a pair of CTAs
    const long long it_beg = p.range_beg[wk], it_end = p.range_beg[wk + 1];
    const int my_iters = (int)(it_end - it_beg);
    const int prefill = my_iters < p.stages ? my_iters : p.stages;    // weight stages requested during set-up
    // work unit -> this CTA's 128-row tile, and the row coordinate of that tile in the weight map
    auto tile_of = [&](int wt) { return PAIR ? 2 * wt + rank : wt; };
    auto w_row = [&](int wt) { return p.swiglu_f ? tile_of(wt) * 64 : tile_of(wt) * TILE_M; };
    // barrier (in the even CTA when PAIR) that counts the bytes of ring stage s
    auto full_bar = [&](int s) { return PAIR ? mapa_shared(smem_u32(&sm->full[s]), 0) : smem_u32(&sm->full[s]); };
    auto load_w = [&](uint32_t dst, int wt, int kc, uint32_t bar, uint64_t pol) {
        if constexpr (PAIR) tma_load_4d_pair(dst, &tm_w, 0, w_row(wt), 0, kc * p.ks, bar, pol);
        else tma_load_4d(dst, &tm_w, 0, w_row(wt), 0, kc * p.ks, bar, pol);
    };
    auto load_x = [&](uint32_t dst, int kc, uint32_t bar, uint64_t pol) {
        if constexpr (PAIR) tma_load_4d_pair(dst, &tm_x, 0, rank * nb_cta, 0, kc * p.ks, bar, pol);
        else tma_load_4d(dst, &tm_x, 0, 0, 0, kc * p.ks, bar, pol);
    };
    const uint32_t full_tx = PAIR ? 2 * stage_bytes : stage_bytes;      // both CTAs' loads land on the even CTA's barrier

    // accumulator buffers are EPI_CHUNK-aligned so that a 32-column read never leaves the allocation
    const uint32_t buf_cols = (uint32_t)((p.nb + EPI_CHUNK - 1) / EPI_CHUNK * EPI_CHUNK);
    uint32_t tmem_cols = 32;
    while (tmem_cols < 2u * buf_cols) tmem_cols <<= 1;

    if (threadIdx.x == 32) {        // descriptor fetches overlap the barrier set-up
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_w) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_x) : "memory");
    }
    // Weights never change, so the first ring-full of weight stages is requested during set-up: their latency
    // overlaps the tensor-memory allocation, the CTA barrier and the tail of the preceding kernel; the activations
    // of those stages follow after the dependency wait.
    auto prefill_weights = [&] {
        uint64_t pol_first;
        asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol_first));
        int wt = (int)(it_beg / p.kiters), kc = (int)(it_beg - (long long)wt * p.kiters);
        for (int i = 0; i < prefill; ++i) {
            if (rank == 0) mbar_expect_tx(smem_u32(&sm->full[i]), full_tx);
            load_w(tiles_addr + i * stage_bytes, wt, kc, full_bar(i), pol_first);
            if (++kc == p.kiters) { kc = 0; ++wt; }
        }
    };
    if (threadIdx.x == 0) {
        const uint32_t epi_warps = TWO ? 8 : 4;
        for (int s = 0; s < p.stages; ++s) { mbar_init(smem_u32(&sm->full[s]), 1); mbar_init(smem_u32(&sm->empty[s]), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(smem_u32(&sm->tmem_full[b]), 1); mbar_init(smem_u32(&sm->tmem_empty[b]), PAIR ? 2 * epi_warps : epi_warps); }
        mbar_init(smem_u32(&sm->drain), 1);
        sm->abort_flag = 0;
        sm->last_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if constexpr (!PAIR) prefill_weights();            // this thread is also the TMA producer
    }
    if (warp == 1) {
        if constexpr (PAIR) {       // the same warp of both CTAs: columns are reserved in both tensor memories
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm->tmem_base)), "r"(tmem_cols) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm->tmem_base)), "r"(tmem_cols) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
    }
    tc_fence_before();
    if constexpr (PAIR) cluster_sync_all();     // the other CTA's barriers exist before anything is counted on them
    else __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = sm->tmem_base;
    volatile int* abort_flag = &sm->abort_flag;
    if (threadIdx.x == 0) pdl_trigger();       // this CTA now owns its shared and tensor memory

    if (warp == 0) {
        // ------------------------------------------------ TMA producer
        if (lane == 0) {
            if constexpr (PAIR) prefill_weights();
            uint64_t pol_stream, pol_keep;
            asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol_stream));
            asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol_keep));
            uint32_t stage = 0, phase = 0;
            int issued = 0;
            bool ok = true;
            // (work unit, kc) advance incrementally: a 64-bit division per stage would cost this single thread
            // more cycles than the loads it issues
            int wt = (int)(it_beg / p.kiters), kc = (int)(it_beg - (long long)wt * p.kiters);
            if (prefill > 0) {
                pdl_wait();                                    // the activations belong to the preceding kernel until now
                for (int q = 0; q < prefill; ++q) {            // activations of the stages whose weights went out during set-up
                    load_x(tiles_addr + q * stage_bytes + a_bytes, kc, full_bar(q), pol_keep);
                    if (++kc == p.kiters) { kc = 0; ++wt; }
                }
                issued = prefill;
                if (prefill == p.stages) phase = 1; else stage = (uint32_t)prefill;
            }
            for (int i = prefill; i < my_iters && ok; ++i) {
                ok = mbar_wait(smem_u32(&sm->empty[stage]), phase ^ 1, abort_flag, p.status, DEV_TIMEOUT_TMA);
                if (!ok) break;
                const uint32_t full = full_bar(stage);
                const uint32_t a_dst = tiles_addr + stage * stage_bytes, b_dst = a_dst + a_bytes;
                if (rank == 0) mbar_expect_tx(smem_u32(&sm->full[stage]), full_tx);
                load_w(a_dst, wt, kc, full, pol_stream);
                load_x(b_dst, kc, full, pol_keep);
                ++issued;
                if (++stage == (uint32_t)p.stages) { stage = 0; phase ^= 1; }
                if (++kc == p.kiters) { kc = 0; ++wt; }
            }
            if (!ok) {
                // drain: wait (bounded) until every load issued into the ring has landed (the even CTA sees the
                // pair's byte counts; the odd one relies on the cluster barrier at the end of the kernel)
                const int inflight = issued < p.stages ? issued : p.stages;
                uint32_t s = stage, ph = phase;
                for (int q = 0; q < inflight && rank == 0; ++q) {
                    if (s == 0) { s = p.stages - 1; ph ^= 1; } else --s;
                    for (uint32_t spin = 0; spin < SPIN_LIMIT && !mbar_try(smem_u32(&sm->full[s]), ph); ++spin) __nanosleep(64);
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer (PAIR: in the even CTA only)
        if (lane == 0 && rank == 0) {
            const uint32_t idesc = instr_desc_f16(p.nb, false, PAIR ? 256 : 128);
            uint32_t stage = 0, phase = 0, buf = 0, buf_phase = 0;
            long long units = 0;
            bool ok = true;
            long long it = it_beg;
            int k0 = (int)(it_beg - (it_beg / p.kiters) * p.kiters);   // later units: next work unit, k0 = 0
            auto commit = [&](uint64_t* bar) {                 // PAIR: the barrier at this offset in both CTAs
                if constexpr (PAIR) tc_commit_pair_both(smem_u32(bar));
                else tc_commit(smem_u32(bar));
            };
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
                        for (int j = 0; j < TILE_K / UMMA_K; ++j) {   // +32 bytes along k inside the swizzle row per step
                            const uint32_t acc = (kc > k0 || sl > 0 || j > 0) ? 1u : 0u;
                            if constexpr (PAIR) tc_mma_f16_pair(d_tmem, adesc + (uint64_t)(j * 2), bdesc + (uint64_t)(j * 2), idesc, acc);
                            else tc_mma_f16(d_tmem, adesc + (uint64_t)(j * 2), bdesc + (uint64_t)(j * 2), idesc, acc);
                        }
                    }
                    commit(&sm->empty[stage]);                 // stage is free once these MMAs have read it
                    if (++stage == (uint32_t)p.stages) { stage = 0; phase ^= 1; }
                }
                if (!ok) break;
                commit(&sm->tmem_full[buf]);                    // accumulator complete
                ++units;
                if (++buf == 2) { buf = 0; buf_phase ^= 1; }
                it += (k1 - k0);
                k0 = 0;
            }
            if (!ok) {
                // make sure no MMA is still running before TMEM goes away
                if constexpr (PAIR) tc_commit_pair_local(smem_u32(&sm->drain));
                else tc_commit(smem_u32(&sm->drain));
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
        // partial-tile buffer of worker c's CTA that works on the same tile parity as this one
        auto part_of = [&](int c) { return p.part + (size_t)(PAIR ? 2 * c + rank : c) * 2 * slot_elems; };
        // the accumulator buffer is free again: counted on the MMA issuer's barrier
        const uint32_t tmem_empty0 = PAIR ? mapa_shared(smem_u32(&sm->tmem_empty[0]), 0) : smem_u32(&sm->tmem_empty[0]);
        auto release_acc = [&](uint32_t b) {
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                if constexpr (PAIR) mbar_arrive_cluster(tmem_empty0 + b * (uint32_t)sizeof(uint64_t));
                else mbar_arrive(tmem_empty0 + b * (uint32_t)sizeof(uint64_t));
            }
        };
        // Epilogue of a complete tile.  split = false: the accumulator holds the whole sum.  split = true: this CTA
        // (the tile's first contributor) has its share in tensor memory and adds the other contributors' partial
        // tiles from the workspace in worker order (fixed order -> reproducible); each one's 32 loads go out together.
        auto finish_tile = [&](int wt_, int tile_, uint32_t t_addr_, bool split, int c_first_, int c_last_) {
            for (int c0 = grp * EPI_CHUNK; c0 < p.nb && c0 < p.n; c0 += GROUPS * EPI_CHUNK) {
                float v[32];
                tc_ld32(t_addr_ + c0, v);                  // may run past nb, never past the buffer
                if (split) {
                    for (int c = c_first_; c <= c_last_; ++c) {          // the first contributor's slot varies, later ones use slot 0
                        if (c == wk) continue;                             // this CTA's own share came from tensor memory
                        const float* src = part_of(c) + (size_t)(c == c_first_ ? p.tile_slot[wt_] * slot_elems : 0) + (size_t)c0 * TILE_M + row;
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
        // Projections into the residual stream finish their split tiles in SLICES: every contributor stores its share
        // and counts itself in; when its range is done it waits (bounded) until all contributors of the tile have
        // arrived and finishes its own share of the tile's node columns (sum of the partial tiles in worker order,
        // residual add, gain-weighted copy, sums of squares).  All SMs take part in the reduction, nobody keeps an
        // accumulator waiting, and the epilogue needs no exchange between rows.
        const bool sliced = p.epi.mode == EPI_RESID_NORM || p.epi.mode == EPI_RESID;
        int pend_wt[2], n_pend = 0;
        uint32_t buf = 0, buf_phase = 0;
        bool ok = true;
        long long it = it_beg;
        int wt = (int)(it_beg / p.kiters), k0 = (int)(it_beg - (long long)wt * p.kiters);
        for (; it < it_end && ok; ++wt, k0 = 0) {
            const int tile = tile_of(wt);
            const long long left = it_end - it;
            const int k1 = (p.kiters - k0 < left) ? p.kiters : (int)(k0 + left);
            const bool whole = (k0 == 0 && k1 == p.kiters) && p.epi.mode != EPI_DEFER;
            mbar_wait(smem_u32(&sm->tmem_full[buf]), buf_phase, abort_flag, p.status, DEV_TIMEOUT_EPI);
            epi_all();                                     // all 256 threads take the same decision
            ok = (*abort_flag == 0);
            if (!ok) break;
            tc_fence_after();
            const uint32_t t_addr = tmem_base + buf * buf_cols + ((uint32_t)(quad * 32) << 16);
            // A tile some workers share is finished by the contributor that completes its share of it LAST (the host
            // knows from the ranges: usually the first contributor, for which the tile is the last unit of its range,
            // while every other contributor handles its share as the first unit of its range, stores it and counts
            // itself in without ever waiting).  The finisher keeps its own share in tensor memory and waits (bounded)
            // for the others; they run at the same time on other SMs and depend on nobody, so the wait is short.
            const int c_first = p.tile_first[wt], c_last = c_first + p.tile_count[wt] - 1;
            bool finish = whole;
            if (!whole && sliced) pend_wt[n_pend++] = wt;
            if (!whole && p.epi.mode != EPI_DEFER && !sliced) {
                if (et == 0) {
                    int fl = 0;
                    if (wk == c_first + p.tile_fin[wt]) {
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
                finish_tile(wt, tile, t_addr, !whole, c_first, c_last);
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
            release_acc(buf);
            if (!finish && p.epi.mode != EPI_DEFER) {
                // count this arrival: the barrier orders every thread's stores before thread 0's
                // release, and the release is cumulative over them
                epi_all();
                if (et == 0) atom_add_acq_rel_gpu(p.counters + tile, 1);
            }
            if (++buf == 2) { buf = 0; buf_phase ^= 1; }
            it += (k1 - k0);
        }
        for (int q = 0; q < n_pend && ok; ++q) {
            const int swt = pend_wt[q], tile = tile_of(swt);
            const int c_first = p.tile_first[swt], cnt = p.tile_count[swt], idx = wk - c_first;
            if (et == 0) {
                uint32_t spin = 0;
                while (ld_acquire_gpu(p.counters + tile) != cnt) {
                    if (++spin >= SPIN_LIMIT) { *abort_flag = 1; atomicCAS(p.status, DEV_OK, DEV_TIMEOUT_GRID); break; }
                    __nanosleep(spin > 64 ? 64 : 20);
                }
            }
            epi_all();
            ok = (*abort_flag == 0);
            if (!ok) break;
            constexpr int CB = 8, P = TWO ? 2 : 1;             // columns per batch of a thread; column phases
            const int lo = p.n * idx / cnt, hi = p.n * (idx + 1) / cnt;
            const int phase = et >> 7;                          // row = et & 127 (the thread's feature), quad = its warp
            const int f = tile * TILE_M + row;
            const unsigned m = (unsigned)p.m;
            const bool norm = p.epi.mode == EPI_RESID_NORM;
            const float g = (norm && f < p.m) ? __half2float(__ldg((const __half*)p.epi.gain + f)) : 0.f;
            const int slot0 = p.tile_slot[swt];
            for (int j0 = lo + phase; j0 < hi; j0 += P * CB) {
                float acc[CB], old[CB];
#pragma unroll
                for (int b = 0; b < CB; ++b) {
                    const int col = j0 + b * P;
                    acc[b] = 0.f;
                    old[b] = (col < hi && f < p.m) ? __ldcg(p.epi.out_f32 + (size_t)col * m + f) : 0.f;
                }
                for (int c = 0; c < cnt; c += 4) {               // four contributors' loads in flight together
                    float t[4][CB];
#pragma unroll
                    for (int cc = 0; cc < 4; ++cc) {
                        const float* src = part_of(c_first + c + cc) + (size_t)((c + cc == 0) ? slot0 : 0) * slot_elems + row;
#pragma unroll
                        for (int b = 0; b < CB; ++b) {
                            const int col = j0 + b * P;
                            t[cc][b] = (c + cc < cnt && col < hi) ? __ldcg(src + (size_t)col * TILE_M) : 0.f;
                        }
                    }
#pragma unroll
                    for (int cc = 0; cc < 4; ++cc)
#pragma unroll
                        for (int b = 0; b < CB; ++b) acc[b] += t[cc][b];
                }
#pragma unroll
                for (int b = 0; b < CB; ++b) {
                    const int col = j0 + b * P;
                    const float v = acc[b] + old[b];
                    if (col < hi && f < p.m) {
                        p.epi.out_f32[(size_t)col * m + f] = v;
                        if (norm) ((__half*)p.epi.xg_out)[(size_t)col * m + f] = __float2half_rn(v * g);
                    }
                    if (norm) {
                        float sq = (col < hi && f < p.m) ? v * v : 0.f;
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
                        if (lane == 0 && col < hi) sm->ssq_slice[quad][col - lo] = sq;
                    }
                }
            }
            epi_all();
            if (norm && et < hi - lo)
                p.epi.ssq_out[(size_t)tile * SSQ_PITCH + lo + et] =
                    (sm->ssq_slice[0][et] + sm->ssq_slice[1][et]) + (sm->ssq_slice[2][et] + sm->ssq_slice[3][et]);
            epi_all();
            if (et == 0 && atom_add_acq_rel_gpu(p.counters + DONE_OFF + tile, 1) == cnt - 1) {
                p.counters[tile] = 0;                           // everybody has passed the wait: ready for the next launch
                p.counters[DONE_OFF + tile] = 0;
            }
        }
    }

    tc_fence_before();
    if constexpr (PAIR) {
        // neither CTA may leave while the other's MMAs can still read its shared memory or write its tensor memory
        if (warp == 0 && lane == 0 && rank != 0 && *abort_flag)
            for (int q = 0; q < 64; ++q) __nanosleep(1000);      // gave up: let this CTA's loads in flight land
        cluster_sync_all();
        if (warp == 1) {
            tc_fence_after();
            asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
        }
    } else {
        __syncthreads();
        if (warp == 1) {
            tc_fence_after();
            asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
        }
    }
}

// ---------------------------------------------------------------- host side
size_t smem_bytes_for(int nb_cta, int ks, int stages) {      // nb_cta: activation rows one CTA loads per k-slab
    return 1024 + (size_t)stages * ks * (TILE_M * TILE_K * 2 + (size_t)nb_cta * TILE_K * 2) + sizeof(Smem);
}

int pick_stages(int nb_cta, int ks) {
    int s = MAX_STAGES;
    while (s > 2 && smem_bytes_for(nb_cta, ks, s) > 227 * 1024) --s;
    return s;
}

int tiles_of(int m, int epi_mode) { return (epi_mode == EPI_SWIGLU) ? (m / 2) / 64 : (m + TILE_M - 1) / TILE_M; }

// CTA pairs (one activation half per CTA) pay off once the activation slab outweighs the weight tile.
bool use_pairs(const ghd_ctx* c, int n, int m, int epi_mode) {
    const int nb = ((n + 15) / 16) * 16;
    const int tiles = tiles_of(m, epi_mode);
    if (c->opt_gemm_pair == 1 || tiles % 2 || tiles < 2 || nb < 32 || c->sm_count < 2) return false;
    return c->opt_gemm_pair == 2 || nb > 128;
}

// CTAs of a launch before the clamp to the work there is
int base_ctas(const ghd_ctx* c, bool pair) {
    int ctas = c->opt_gemm_ctas > 0 && c->opt_gemm_ctas < c->sm_count ? c->opt_gemm_ctas : c->sm_count;
    if (pair) ctas &= ~1;
    return ctas < (pair ? 2 : 1) ? (pair ? 2 : 1) : ctas;
}

}  // namespace

bool gemm_tc_supported(const ghd_ctx* c, int n, int k, int m, int epi_mode) {
    if (c->cfg.dtype != GHD_F16 || n < 1 || n > GHD_MAX_NODES || k % TILE_K || k < TILE_K) return false;
    const int n_tiles = tiles_of(m, epi_mode);
    if (n_tiles < 1 || n_tiles > MAX_TILES) return false;
    if (epi_mode == EPI_SWIGLU && (m / 2) % 64) return false;
    if (epi_mode == EPI_ROPE_KV && ((m / 3) % TILE_M || m % 3)) return false;
    if (epi_mode == EPI_RESID_NORM && (m % TILE_M || m / TILE_M > SSQ_MAX_TILES)) return false;
    if (epi_mode == EPI_DEFER) {
        const bool pair = use_pairs(c, n, m, epi_mode);
        int workers = base_ctas(c, pair) / (pair ? 2 : 1);
        const int nb = ((n + 15) / 16) * 16;
        const int ks = c->opt_gemm_burst > 0 ? (c->opt_gemm_burst > 4 ? 4 : c->opt_gemm_burst) : ((pair ? nb / 2 : nb) <= 128 ? 2 : 1);
        const int kch = (k / TILE_K + ks - 1) / ks;
        const long long total = (long long)(n_tiles / (pair ? 2 : 1)) * kch;
        if (workers > total) workers = (int)total;
        if (m % 4 || m > 16384 || total / workers + 1 > kch || total / workers < 1) return false;
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
    p.n_tiles = tiles_of(m, epi.mode);
    p.pair = use_pairs(c, n, m, epi.mode) ? 1 : 0;
    p.n_work = p.pair ? p.n_tiles / 2 : p.n_tiles;
    const int nb_cta = p.pair ? p.nb / 2 : p.nb;
    p.ks = c->opt_gemm_burst > 0 ? c->opt_gemm_burst : (nb_cta <= 128 ? 2 : 1);
    if (p.ks > 4) p.ks = 4;
    p.kslabs = k / TILE_K;
    p.kiters = (p.kslabs + p.ks - 1) / p.ks;
    p.stages = pick_stages(nb_cta, p.ks);
    if (c->opt_gemm_stages >= 2 && c->opt_gemm_stages < p.stages) p.stages = c->opt_gemm_stages;
    p.part = c->gemm_part;
    p.counters = c->counters;
    p.status = c->status;
    p.epi = epi;
    if (!tmap_slabs(c, w, (uint64_t)m, (uint64_t)k, p.swiglu_f ? 2 : 1, p.swiglu_f ? 64 : TILE_M, (uint32_t)p.ks, &plan->tm_w) ||
        !tmap_slabs(c, x, (uint64_t)n, (uint64_t)k, 1, (uint32_t)nb_cta, (uint32_t)p.ks, &plan->tm_x)) {
        snprintf(c->err, sizeof(c->err), "tcgen05 GEMM: tensor map encoding failed");
        return GHD_ECUDA;
    }
    // workers: CTAs, or clusters of two CTAs; they share the flattened (work unit, k-chunk) space
    const int per = p.pair ? 2 : 1;
    const long long total = (long long)p.n_work * p.kiters;
    int workers = base_ctas(c, p.pair != 0) / per;
    if (c->opt_gemm_ctas <= 0 && epi.mode != EPI_DEFER && p.n_work < workers) {
        // Fewer work units than workers: every range is shorter than a unit.  With n_work * q / (q - 1) workers each
        // range is (q-1)/q of a unit and always touches a unit boundary, so no tile is shared by three workers
        // and no worker's only share sits strictly inside a tile (those finish together and take the slow
        // split-tile path).  Take the largest such count that fits the SMs.
        int best = 0;
        for (int q = 2; q <= 64; ++q)
            if ((p.n_work * q) % (q - 1) == 0) {
                const int g = p.n_work * q / (q - 1);
                if (g <= workers && g > best) best = g;
            }
        if (best >= workers * 3 / 4) workers = best;
    }
    if (workers > total) workers = (int)total;
    const int ctas = workers * per;
    p.ctas = ctas;
    plan->smem = smem_bytes_for(nb_cta, p.ks, p.stages);
    if (workers > MAX_WORKERS) {
        snprintf(c->err, sizeof(c->err), "tcgen05 GEMM: more than %d workers", MAX_WORKERS);
        return GHD_EUNSUPPORTED;
    }
    for (int w2 = 0; w2 <= workers; ++w2) p.range_beg[w2] = (int)(total * w2 / workers);
    // Three workers per two work units (every range 2/3 of a unit): the middle worker of a group holds the tail of one
    // unit and the head of the next and would end together with the worker that finishes the second unit, which would
    // then wait for its store.  A few k-chunks less for the middle worker and it is done early; the outer two grow a
    // little and each finishes its own unit without waiting.
    int skew = c->opt_gemm_skew > 0 ? c->opt_gemm_skew - 1 : 1;       // automatic: one k-chunk, as measured
    if (epi.mode != EPI_DEFER && workers % 3 == 0 && (long long)workers * 2 == (long long)p.n_work * 3 && skew > 0 && 3 * skew < p.kiters)
        for (int g = 0; g < workers / 3; ++g) {
            p.range_beg[3 * g + 1] += skew;          // the first worker of the group takes `skew` more
            p.range_beg[3 * g + 2] -= skew;          // so does the third
        }
    for (int t = 0; t < p.n_work; ++t) {
        const long long t_first = (long long)t * p.kiters, t_end = t_first + p.kiters;
        int c_first = 0;
        while (p.range_beg[c_first + 1] <= t_first) ++c_first;
        int c_last = c_first;
        while (c_last + 1 < workers && p.range_beg[c_last + 1] < t_end) ++c_last;
        p.tile_first[t] = (unsigned short)c_first;
        p.tile_count[t] = (unsigned char)(c_last - c_first + 1);
        p.tile_slot[t] = (p.range_beg[c_first] >= t_first) ? 0 : 1;
        // the finisher: the contributor that completes its share of this tile last, counted in k-chunks from the start
        // of its own range (all workers start together); the first contributor on a tie: for it the tile comes last
        auto share_done = [&](int cc) {
            const long long e = p.range_beg[cc + 1] < t_end ? p.range_beg[cc + 1] : t_end;
            return e - p.range_beg[cc];
        };
        int fin = c_first;
        for (int cc = c_first + 1; cc <= c_last; ++cc)
            if (share_done(cc) > share_done(fin)) fin = cc;
        p.tile_fin[t] = (unsigned char)(fin - c_first);
    }
    plan->pending.active = 0;
    if (epi.mode == EPI_DEFER) {
        if (total / workers + 1 > p.kiters) {             // a worker's range must touch at most two work units
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
        pp.stride = per;                                  // CTA pairs: a tile's contributors are every other CTA
        for (int t = 0; t < p.n_tiles && t < 128; ++t) {
            const int wt = t / per;
            pp.first_cta[t] = (unsigned short)(p.tile_first[wt] * per + t % per);
            pp.n_contrib[t] = p.tile_count[wt];
            pp.first_slot[t] = p.tile_slot[wt];
        }
    }
    return GHD_OK;
}

ghd_status launch_gemm_tc(ghd_ctx* c, const void* x, const void* w, int n, int k, int m, const EpiArgs& epi) {
    GemmPlan plan;
    const ghd_status s = plan_gemm_tc(c, x, w, n, k, m, epi, &plan);
    if (s != GHD_OK) return s;
    if (!c->attr_gemm) {       // per context: the attribute belongs to the device the context was created on
        if (cudaFuncSetAttribute(k_gemm_tc<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess ||
            cudaFuncSetAttribute(k_gemm_tc<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess ||
            cudaFuncSetAttribute(k_gemm_tc<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess ||
            cudaFuncSetAttribute(k_gemm_tc<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess) {
            snprintf(c->err, sizeof(c->err), "tcgen05 GEMM: cannot raise dynamic shared memory: %s", cudaGetErrorString(cudaGetLastError()));
            return GHD_ECUDA;
        }
        c->attr_gemm = true;
    }
    if (plan.pending.active) c->pending = plan.pending;
    const bool two = c->opt_gemm_epi ? c->opt_gemm_epi == 2 : plan.p.nb > EPI_CHUNK;
    if (plan.p.pair) {
        c->path_count[GHD_PATH_GEMM_PAIR]++;
        if (two) launch_kc(c, true, 2, k_gemm_tc<true, true>, plan.p.ctas, THREADS_TC, plan.smem, plan.tm_w, plan.tm_x, plan.p);
        else launch_kc(c, true, 2, k_gemm_tc<false, true>, plan.p.ctas, THREADS, plan.smem, plan.tm_w, plan.tm_x, plan.p);
    } else if (two) {
        launch_k(c, true, k_gemm_tc<true, false>, plan.p.ctas, THREADS_TC, plan.smem, plan.tm_w, plan.tm_x, plan.p);
    } else {
        launch_k(c, true, k_gemm_tc<false, false>, plan.p.ctas, THREADS, plan.smem, plan.tm_w, plan.tm_x, plan.p);
    }
    return GHD_OK;
}

}  // namespace ghd
