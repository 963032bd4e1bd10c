// Skinny projection GEMM without any k-split, for few nodes (MMA N <= 64) and many output
// rows: Y[n][m] = X[n][k] * W[m][k]^T on the 5th-generation tensor cores (sm_100a).
//
// k_gemm_tc cuts the flattened (128-row tile, k-chunk) space into equal ranges, which balances
// the weight bytes per SM but leaves most tiles shared by two or more CTAs: partial tiles go
// through memory and a last arriver finishes them, a few microseconds at the end of every launch
// that no weight streams through.  Here the OUTPUT ROWS are cut into equal contiguous ranges, one
// per CTA (m / SMs rows each, not a multiple of anything), and every CTA runs the whole reduction
// for its rows: no partial tiles, no arrival counters, no finishing pass.  The price is a TMA box
// whose height is the ragged range (at most 128 rows): the MMA still computes 128 rows, the rows
// past the box hold whatever the ring held before and their results are dropped (the tensor pipe
// is far from busy at these widths), and the activation tile is re-read by more CTAs (L2 traffic).
//
// Rows come in "planes" so that values that meet in the epilogue sit in the same accumulator:
//   EPI_RAW      1 plane : rows t of W
//   EPI_SWIGLU   2 planes: gate row t, up row t + d_ffn            -> SiLU(gate) * up
//   EPI_ROPE_KV  2 planes: rows t and t + d_head/2 of one head     -> rotary pair (q, k), plain copy (v)
// and in groups (one group = one head of q, k or v; a single group otherwise); a unit never
// crosses a group.  A unit of `len` rows per plane is fetched with a box of h rows per plane whose
// start is chosen so that the rows outside the unit fall outside the group where possible: the
// hardware fills those with zeros without reading memory.
//
// Per CTA: warp 0 = TMA producer, warp 1 = MMA issuer and TMEM owner, warps 2..5 = epilogue.
// All waits are bounded; on expiry the kernel records a status code, drains and returns.
#include <cuda.h>

#include <cstdio>
#include <cstring>

#include "gemm_tc_dev.cuh"

namespace ghd {

using namespace gemmdev;

namespace {

constexpr int EV_MAX_UNITS = 6;

struct EvenParams {
    int n, nb, m;                    // nodes, padded nodes (MMA N), output features
    int kslabs, ks, kiters, stages;  // 64-column slabs per row, slabs per stage, stages per unit, ring depth
    int planes, h;                   // planes per unit, box rows per plane (planes * h <= 128)
    int gs, total;                   // rows per plane in a group, rows per plane in all groups together
    int a_slab_bytes;                // shared-memory bytes reserved per weight slab (whole 8-row groups)
    int ctas;
    int plane_off;                   // distance between the two planes in output terms (d_ffn, or d_head / 2)
    int heads;                       // EPI_ROPE_KV: heads per section
    int* status;
    EpiArgs epi;
};

struct Unit {
    int group, tb, t0, len;          // box starts at row tb of the group (may be negative); rows t0 .. t0+len-1 are the unit's
};

struct EvenSmem {
    uint64_t full[MAX_STAGES];
    uint64_t empty[MAX_STAGES];
    uint64_t tmem_full[2];
    uint64_t tmem_empty[2];
    uint64_t drain;
    uint32_t tmem_base;
    int abort_flag;
    int n_units;
    Unit units[EV_MAX_UNITS];
    float stage_x[EPI_CHUNK][TILE_M + 1];
};

__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, int c3, int c4, uint32_t bar,
                                            uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint"
        " [%0], [%1, {%2, %3, %4, %5, %6}], [%7], %8;"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4), "r"(bar), "l"(policy) : "memory");
}

// ---------------------------------------------------------------- fused epilogue
// Thread `row` holds the sums v[j] of accumulator row `row` for nodes c0 .. c0+31.  Row r < planes * h
// is plane r / h, row t = u.tb + r % h of the group; it belongs to the unit when t0 <= t < t0 + len.
__device__ __forceinline__ void epilogue_even(const EvenParams& p, EvenSmem* sm, const Unit& u, int row, int c0, float (&v)[32]) {
    const EpiArgs& e = p.epi;
    const int pl = row / p.h, tr = row - pl * p.h, t = u.tb + tr;
    const bool mine = pl < p.planes && t >= u.t0 && t < u.t0 + u.len;
    if (e.mode == EPI_RAW) {
        if (mine) {
            float* dst = e.out_f32 + (size_t)c0 * p.m + t;
#pragma unroll
            for (int j = 0; j < 32; ++j)
                if (c0 + j < p.n) dst[(size_t)j * p.m] = v[j];
        }
        return;
    }
    if (e.mode == EPI_SWIGLU) {
        // plane 0 = gate, plane 1 = up.  After the exchange the thread of plane pl finishes nodes
        // 16 * pl .. 16 * pl + 15 of feature t.
#pragma unroll
        for (int j = 0; j < 32; ++j) sm->stage_x[j][row] = v[j];
        epi_bar();
        if (mine) {
            const int jb = pl * 16;
            float g[16], up[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) { g[j] = sm->stage_x[jb + j][tr]; up[j] = sm->stage_x[jb + j][tr + p.h]; }
            __half res[16];
#pragma unroll
            for (int j = 0; j < 16; ++j)
                res[j] = __float2half_rn(__fdividef(g[j] * up[j], 1.f + exp2f(-1.4426950408889634f * g[j])));
            __half* dst = (__half*)e.out_t + (size_t)(c0 + jb) * p.plane_off + t;
#pragma unroll
            for (int j = 0; j < 16; ++j)
                if (c0 + jb + j < p.n) dst[(size_t)j * p.plane_off] = res[j];
        }
        epi_bar();
        return;
    }
    // EPI_ROPE_KV: group = section * heads + head; plane 0 holds element t of the head, plane 1 element t + d_head / 2
    const int d = e.d_model, dh = e.d_head, half = dh >> 1;
    const int section = u.group / p.heads, head = u.group - section * p.heads;
    const int idx = t + pl * half;
    if (section < 2) {
        float2 cs[32];
        const int tt = mine ? t : 0;
        const float2* tab = reinterpret_cast<const float2*>(e.rope + (size_t)c0 * dh + 2 * tt);
#pragma unroll
        for (int j = 0; j < 32; ++j) cs[j] = (mine && c0 + j < p.n) ? __ldg(tab + (size_t)j * half) : make_float2(1.f, 0.f);
#pragma unroll
        for (int j = 0; j < 32; ++j) sm->stage_x[j][row] = v[j];
        epi_bar();
        if (mine) {
            const int prow = pl == 0 ? row + p.h : row - p.h;
            const float sign = pl == 0 ? -1.f : 1.f;
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = fmaf(sign * sm->stage_x[j][prow], cs[j].y, v[j] * cs[j].x);
            __half* dst;
            size_t pitch;
            if (section == 0) { dst = (__half*)e.out_t + (size_t)c0 * d + head * dh + idx; pitch = (size_t)d; }
            else { dst = (__half*)e.k_cache + ((size_t)head * e.max_kv_len + e.kv_len + c0) * dh + idx; pitch = (size_t)dh; }
#pragma unroll
            for (int j = 0; j < 32; ++j)
                if (c0 + j < p.n) dst[(size_t)j * pitch] = __float2half_rn(v[j]);
        }
        epi_bar();
    } else if (mine) {
        __half* dst = (__half*)e.v_cache + ((size_t)head * e.max_kv_len + e.kv_len + c0) * dh + idx;
#pragma unroll
        for (int j = 0; j < 32; ++j)
            if (c0 + j < p.n) dst[(size_t)j * dh] = __float2half_rn(v[j]);
    }
}

// ---------------------------------------------------------------- kernel
__global__ void __launch_bounds__(THREADS, 1)
k_gemm_even(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_x, const EvenParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t pad = (1024u - (raw_addr & 1023u)) & 1023u;
    uint8_t* tiles = smem_raw + pad;
    const uint32_t b_slab = (uint32_t)p.nb * TILE_K * 2;
    const uint32_t a_bytes = p.ks * p.a_slab_bytes, b_bytes = p.ks * b_slab;
    const uint32_t stage_bytes = a_bytes + b_bytes;
    const uint32_t box_bytes = (uint32_t)(p.planes * p.h) * TILE_K * 2;          // one weight box as the TMA counts it
    // the MMA reads 128 rows from every weight slab: keep the rows past the last slab of the ring inside the allocation
    const uint32_t tail_pad = TILE_M * TILE_K * 2;
    EvenSmem* sm = reinterpret_cast<EvenSmem*>(tiles + (size_t)p.stages * stage_bytes + tail_pad);
    const uint32_t tiles_addr = smem_u32(tiles);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int cta = blockIdx.x;

    const uint32_t buf_cols = (uint32_t)((p.nb + EPI_CHUNK - 1) / EPI_CHUNK * EPI_CHUNK);
    uint32_t tmem_cols = 32;
    while (tmem_cols < 2u * buf_cols) tmem_cols <<= 1;

    if (threadIdx.x == 32) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_w) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_x) : "memory");
    }
    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) { mbar_init(smem_u32(&sm->full[s]), 1); mbar_init(smem_u32(&sm->empty[s]), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(smem_u32(&sm->tmem_full[b]), 1); mbar_init(smem_u32(&sm->tmem_empty[b]), 4); }
        mbar_init(smem_u32(&sm->drain), 1);
        sm->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        // this CTA's rows [lo, hi) of the plane, cut at group borders and into pieces of at most h rows
        const int lo = (int)((long long)p.total * cta / p.ctas), hi = (int)((long long)p.total * (cta + 1) / p.ctas);
        int nu = 0;
        for (int cur = lo; cur < hi && nu < EV_MAX_UNITS;) {
            Unit u;
            u.group = cur / p.gs;
            u.t0 = cur - u.group * p.gs;
            int len = hi - cur;
            if (len > p.gs - u.t0) len = p.gs - u.t0;
            if (len > p.h) len = p.h;
            u.len = len;
            // rows of the box outside the unit cost memory traffic only when they lie inside the group
            u.tb = (u.t0 + len == p.gs) ? u.t0 : (u.t0 == 0 ? len - p.h : u.t0);
            sm->units[nu++] = u;
            cur += len;
        }
        sm->n_units = nu;
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
    const int n_units = sm->n_units;
    if (threadIdx.x == 0) pdl_trigger();

    if (warp == 0) {
        // ------------------------------------------------ TMA producer
        if (lane == 0) {
            uint64_t pol_stream, pol_keep;
            asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol_stream));
            asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol_keep));
            uint32_t stage = 0, phase = 0;
            int issued = 0;
            bool ok = true, waited = false;
            // weights never change: the first stages' weight boxes go out before the dependency wait,
            // the activations of those stages follow after it
            const int total_iters = n_units * p.kiters;
            const int prefill = total_iters < p.stages / 2 ? total_iters : p.stages / 2;
            for (int ui = 0; ui < n_units && ok; ++ui) {
                const Unit u = sm->units[ui];
                for (int kc = 0; kc < p.kiters; ++kc) {
                    if (issued >= p.stages) ok = mbar_wait(smem_u32(&sm->empty[stage]), phase ^ 1, abort_flag, p.status, DEV_TIMEOUT_TMA);
                    if (!ok) break;
                    const uint32_t full = smem_u32(&sm->full[stage]);
                    const uint32_t a_dst = tiles_addr + stage * stage_bytes;
                    const int nslab = (p.kslabs - kc * p.ks < p.ks) ? p.kslabs - kc * p.ks : p.ks;
                    mbar_expect_tx(full, (uint32_t)nslab * box_bytes + b_bytes);
                    for (int sl = 0; sl < nslab; ++sl)
                        tma_load_5d(a_dst + sl * p.a_slab_bytes, &tm_w, 0, u.tb, 0, u.group, kc * p.ks + sl, full, pol_stream);
                    if (issued >= prefill) {
                        if (!waited) { pdl_wait(); waited = true; }
                        tma_load_4d(a_dst + a_bytes, &tm_x, 0, 0, 0, kc * p.ks, full, pol_keep);
                    } else if (issued == prefill - 1) {
                        pdl_wait();
                        waited = true;
                        // stages 0 .. prefill-1 hold k-chunks 0 .. prefill-1 of the first units, in order
                        for (int q = 0; q < prefill; ++q)
                            tma_load_4d(tiles_addr + q * stage_bytes + a_bytes, &tm_x, 0, 0, 0, (q % p.kiters) * p.ks, smem_u32(&sm->full[q]), pol_keep);
                    }
                    ++issued;
                    if (++stage == (uint32_t)p.stages) { stage = 0; phase ^= 1; }
                }
            }
            if (!ok) {
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
            bool ok = true;
            for (int ui = 0; ui < n_units && ok; ++ui) {
                if (ui >= 2) ok = mbar_wait(smem_u32(&sm->tmem_empty[buf]), buf_phase ^ 1, abort_flag, p.status, DEV_TIMEOUT_TMEM);
                if (!ok) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * buf_cols;
                for (int kc = 0; kc < p.kiters; ++kc) {
                    ok = mbar_wait(smem_u32(&sm->full[stage]), phase, abort_flag, p.status, DEV_TIMEOUT_MMA);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t a_addr = tiles_addr + stage * stage_bytes, b_addr = a_addr + a_bytes;
                    const int nslab = (p.kslabs - kc * p.ks < p.ks) ? p.kslabs - kc * p.ks : p.ks;
                    for (int sl = 0; sl < nslab; ++sl) {
                        const uint64_t adesc = smem_desc_sw128(a_addr + sl * p.a_slab_bytes), bdesc = smem_desc_sw128(b_addr + sl * b_slab);
#pragma unroll
                        for (int j = 0; j < TILE_K / UMMA_K; ++j)
                            tc_mma_f16(d_tmem, adesc + (uint64_t)(j * 2), bdesc + (uint64_t)(j * 2), idesc, (kc > 0 || sl > 0 || j > 0) ? 1u : 0u);
                    }
                    tc_commit(smem_u32(&sm->empty[stage]));
                    if (++stage == (uint32_t)p.stages) { stage = 0; phase ^= 1; }
                }
                if (!ok) break;
                tc_commit(smem_u32(&sm->tmem_full[buf]));
                if (++buf == 2) { buf = 0; buf_phase ^= 1; }
            }
            if (!ok) {
                tc_commit(smem_u32(&sm->drain));
                for (uint32_t spin = 0; spin < SPIN_LIMIT && !mbar_try(smem_u32(&sm->drain), 0); ++spin) __nanosleep(64);
            }
        }
    } else {
        // ------------------------------------------------ epilogue warps (TMEM lanes 32 * (warp % 4) ..)
        const int quad = warp & 3;
        const int row = quad * 32 + lane;
        pdl_wait();
        uint32_t buf = 0, buf_phase = 0;
        for (int ui = 0; ui < n_units; ++ui) {
            const Unit u = sm->units[ui];
            mbar_wait(smem_u32(&sm->tmem_full[buf]), buf_phase, abort_flag, p.status, DEV_TIMEOUT_EPI);
            epi_bar();
            if (*abort_flag != 0) break;
            tc_fence_after();
            const uint32_t t_addr = tmem_base + buf * buf_cols + ((uint32_t)(quad * 32) << 16);
            for (int c0 = 0; c0 < p.nb; c0 += EPI_CHUNK) {
                float v[32];
                tc_ld32(t_addr + c0, v);
                if (c0 < p.n) epilogue_even(p, sm, u, row, c0, v);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sm->tmem_empty[buf]));
            if (++buf == 2) { buf = 0; buf_phase ^= 1; }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
    }
}

size_t even_smem_bytes(int nb, int ks, int a_slab_bytes, int stages) {
    return 1024 + (size_t)stages * ks * ((size_t)a_slab_bytes + (size_t)nb * TILE_K * 2) + TILE_M * TILE_K * 2 + sizeof(EvenSmem);
}

}  // namespace

// Fills the shape part of the parameters; false when this kernel does not take the problem.
static bool even_shape(const ghd_ctx* c, int n, int k, int m, int epi_mode, EvenParams& p, uint64_t& groups, uint64_t& group_stride,
                       uint64_t& plane_stride) {
    if (c->cfg.dtype != GHD_F16 || n < 1 || n > 64 || k % TILE_K || k < TILE_K) return false;
    if (epi_mode != EPI_RAW && epi_mode != EPI_SWIGLU && epi_mode != EPI_ROPE_KV) return false;
    if (epi_mode == EPI_SWIGLU && m % 2) return false;
    if (epi_mode == EPI_ROPE_KV && (m % 3 || m / 3 != c->cfg.d_model)) return false;
    p.n = n;
    p.nb = ((n + 15) / 16) * 16;
    p.m = m;
    p.kslabs = k / TILE_K;
    p.ks = 2;
    p.kiters = (p.kslabs + p.ks - 1) / p.ks;
    p.planes = epi_mode == EPI_RAW ? 1 : 2;
    p.ctas = c->opt_gemm_ctas > 0 && c->opt_gemm_ctas < c->sm_count ? c->opt_gemm_ctas : c->sm_count;
    groups = 1; group_stride = 0; plane_stride = 0;
    p.heads = 1;
    p.plane_off = 0;
    if (epi_mode == EPI_ROPE_KV) {
        const int half = c->cfg.d_head / 2;
        p.gs = half;
        p.heads = c->cfg.n_heads;
        groups = 3ull * c->cfg.n_heads;
        group_stride = c->cfg.d_head;
        plane_stride = half;
        p.plane_off = half;
    } else if (epi_mode == EPI_SWIGLU) {
        p.gs = m / 2;
        plane_stride = m / 2;
        p.plane_off = m / 2;
    } else {
        p.gs = m;
    }
    p.total = p.gs * (int)groups;
    // worth it only when every CTA gets a decent share of rows, and a short unit list must cover that share
    if (p.total < 8 * p.ctas) return false;
    const int per_cta = (p.total + p.ctas - 1) / p.ctas;
    const int hmax = (TILE_M / p.planes < p.gs) ? TILE_M / p.planes : p.gs;
    const int pieces = (per_cta + hmax - 1) / hmax;
    p.h = (per_cta + pieces - 1) / pieces;
    if ((per_cta + p.h - 1) / p.h + (per_cta + p.gs - 1) / p.gs + 1 > EV_MAX_UNITS) return false;
    p.a_slab_bytes = ((p.planes * p.h + 7) / 8) * 8 * TILE_K * 2;
    int stages = MAX_STAGES;
    while (stages > 2 && even_smem_bytes(p.nb, p.ks, p.a_slab_bytes, stages) > 227 * 1024) --stages;
    p.stages = stages;
    return even_smem_bytes(p.nb, p.ks, p.a_slab_bytes, stages) <= 227 * 1024;
}

bool gemm_even_supported(const ghd_ctx* c, int n, int k, int m, int epi_mode) {
    EvenParams p{};
    uint64_t groups, group_stride, plane_stride;
    return even_shape(c, n, k, m, epi_mode, p, groups, group_stride, plane_stride);
}

ghd_status launch_gemm_even(ghd_ctx* c, const void* x, const void* w, int n, int k, int m, const EpiArgs& epi) {
    if (((uintptr_t)x & 15) || ((uintptr_t)w & 15)) {
        snprintf(c->err, sizeof(c->err), "tcgen05 GEMM: operands must be 16-byte aligned");
        return GHD_EINVAL;
    }
    EvenParams p{};
    uint64_t groups, group_stride, plane_stride;
    if (!even_shape(c, n, k, m, epi.mode, p, groups, group_stride, plane_stride)) {
        snprintf(c->err, sizeof(c->err), "tcgen05 GEMM (even rows): shape not taken");
        return GHD_EUNSUPPORTED;
    }
    p.status = c->status;
    p.epi = epi;
    CUtensorMap tm_w, tm_x;
    if (!tmap_even(c, w, (uint64_t)k, (uint32_t)p.planes, plane_stride, groups, group_stride, (uint64_t)p.gs, (uint32_t)p.h, &tm_w) ||
        !tmap_slabs(c, x, (uint64_t)n, (uint64_t)k, 1, (uint32_t)p.nb, (uint32_t)p.ks, &tm_x)) {
        snprintf(c->err, sizeof(c->err), "tcgen05 GEMM: tensor map encoding failed");
        return GHD_ECUDA;
    }
    static bool attr_set = false;
    if (!attr_set) {
        if (cudaFuncSetAttribute(k_gemm_even, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess) {
            snprintf(c->err, sizeof(c->err), "tcgen05 GEMM: cannot raise dynamic shared memory: %s", cudaGetErrorString(cudaGetLastError()));
            return GHD_ECUDA;
        }
        attr_set = true;
    }
    launch_k(c, true, k_gemm_even, p.ctas, THREADS, even_smem_bytes(p.nb, p.ks, p.a_slab_bytes, p.stages), tm_w, tm_x, p);
    return GHD_OK;
}

}  // namespace ghd
