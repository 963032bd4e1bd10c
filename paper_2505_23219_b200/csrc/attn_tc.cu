// Tree attention on the tensor cores (sm_100a, half in, float softmax/accumulate).
//
// One CTA = one head x one tile of up to 128 query nodes x one KV split.  Keys are
// walked in 64-key units: the cache rows [0, kv_len) first (the dense part: every
// query sees every row), then the new rows in groups of 64 nodes = one word of the
// packed ancestor bitmask per query (the sparse part).  A node group whose mask
// word is zero for every query of the CTA is dropped before anything of it is
// loaded.  The cache tiles are divided evenly among the splits of a head and the
// node groups are dealt to the splits one each.
//
// Per unit:  S = Q K^T   (tcgen05.mma, Q and K tile K-major in swizzled shared memory,
//                         S [128 x 64] float in tensor memory)
//            softmax warps (one thread per query row) read S, apply the mask, keep a
//            running (max, sum), and write P = exp(S - max) as half into shared memory
//            PV = P V     (tcgen05.mma, V tile consumed row-major as an N-major operand)
//            softmax warps fold PV into their float output registers, rescaled by
//            exp(old max - new max)
// S and PV are double-buffered in tensor memory so that S of unit j+1 is computed
// while unit j is in softmax.  Each CTA writes un-normalised (o, max, sum) for its
// split; k_attn_combine merges the splits (paper Sec. III-B-2: per-partition
// softmax aligned by a scaling factor at the end).
//
// Warp 0 = TMA producer, warp 1 = issuer of the S MMAs + tensor-memory owner, warps 2..5 =
// softmax (128 threads = 128 tensor-memory lanes), warp 6 = issuer of the PV MMAs (two issuing
// threads because one thread's MMA issue rate, not the tensor pipe, was the limit).  All waits are bounded.  Cache tiles that
// lie wholly below kv_len cannot be touched by the preceding kernel, so the producer requests
// the first of them before it waits for that kernel to finish.
#include <cstdio>

#include "internal.h"
#include "tc_common.cuh"

namespace ghd {

namespace {

using namespace tc;

constexpr int QM = 128;        // query rows per CTA (MMA M)
constexpr int BN = 64;         // keys per unit (MMA N of S, MMA K of PV)
constexpr int KV_STAGES = 4;
constexpr int THREADS = 224;
constexpr int THREADS_DUO = 352;   // two more softmax warpgroups' worth of threads: see k_attn_tc, DUO
constexpr int MAX_UNITS_WORDS = GHD_MAX_NODES / 64;

struct AttnParams {
    int n, heads, kv_len, max_nodes, splits, n_words;
    const int* kv_len_dev;     // non-null: the cache length comes from this device word
    int max_kv_len;
    int cache_only;            // 1: the new rows are somebody else's (the coordinate-index kernel): no node groups here
    const uint64_t* mask;
    float* part_o;
    float* part_ml;
    int* status;
    float scale;               // 1 / sqrt(d_head)
};

struct AttnSmem {
    uint64_t q_full;
    uint64_t kv_full[KV_STAGES], kv_empty[KV_STAGES];
    uint64_t s_full[2], s_empty[2], p_full[2], p_empty[2], pv_full[2], pv_empty[2];
    uint64_t drain, drain_pv;
    uint64_t mask_ready;          // all 128 row threads have merged their mask words into word_or
    unsigned long long word_or[MAX_UNITS_WORDS];
    uint32_t tmem_base;
    int abort_flag;
    float xmax[2][2 * QM];        // two threads per row: they exchange their partial maxima
    float xl[2 * QM];             // ... and, at the end, their partial sums
};

template <int THREADS_IN> __device__ __forceinline__ void pair_bar() { asm volatile("bar.sync 2, %0;" ::"n"(THREADS_IN) : "memory"); }

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// PAIR: at most 64 query rows.  The queries are loaded twice (tile rows r and r + 64 hold the same
// query), so S, P and PV come out duplicated and two threads share a row: thread r takes the
// first 32 keys of a unit and the first half of d_head, thread r + 64 the rest.  This halves the
// per-unit softmax time, which is what bounds the kernel at small trees.
// DUO: more than 64 query rows, so nothing can be duplicated; instead a second group of four softmax warps
// (warps 7..10) shares the tensor-memory lanes of the first (a warp may touch lanes 32 (w mod 4) ..): again two
// threads per row, the first group's thread taking the first 32 keys of a unit and the first half of d_head.
template <int DH, bool PAIR, bool DUO = false>
__global__ void __launch_bounds__(DUO ? THREADS_DUO : THREADS, 1)
k_attn_tc(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
          const __grid_constant__ CUtensorMap tm_v, const AttnParams p) {
    constexpr int SLABS = DH / 64;                       // 64-wide (128-byte) column slabs of a d_head row
    constexpr uint32_t Q_SLAB = QM * 128;                // bytes of one [128 x 64] half slab
    constexpr uint32_t KV_SLAB = BN * 128;               // bytes of one [64 x 64] half slab
    constexpr uint32_t Q_BYTES = SLABS * Q_SLAB;
    constexpr uint32_t STAGE_BYTES = 2 * SLABS * KV_SLAB;   // K slabs then V slabs
    constexpr uint32_t P_BYTES = QM * 128;               // [128 x 64] half
    constexpr uint32_t TMEM_S = 0, TMEM_PV = 2 * BN;     // columns: S[2] then PV[2]

    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t pad = (1024u - (raw_addr & 1023u)) & 1023u;
    uint8_t* base = smem_raw + pad;
    const uint32_t q_addr = smem_u32(base);
    const uint32_t kv_addr = q_addr + Q_BYTES;
    const uint32_t p_addr = kv_addr + KV_STAGES * STAGE_BYTES;
    uint8_t* p_ptr = base + Q_BYTES + KV_STAGES * STAGE_BYTES;
    AttnSmem* sm = reinterpret_cast<AttnSmem*>(p_ptr + 2 * P_BYTES);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int split = blockIdx.x, h = blockIdx.y, mtile = blockIdx.z;
    const int row0 = mtile * QM;

    if (threadIdx.x == 32) {        // descriptor fetches overlap the barrier set-up
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_q) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_k) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_v) : "memory");
    }
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&sm->q_full), 1);
        for (int s = 0; s < KV_STAGES; ++s) { mbar_init(smem_u32(&sm->kv_full[s]), 1); mbar_init(smem_u32(&sm->kv_empty[s]), 1); }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&sm->s_full[b]), 1);
            mbar_init(smem_u32(&sm->s_empty[b]), DUO ? 256 : 128);
            mbar_init(smem_u32(&sm->p_full[b]), DUO ? 256 : 128);
            mbar_init(smem_u32(&sm->p_empty[b]), 1);
            mbar_init(smem_u32(&sm->pv_full[b]), 1);
            mbar_init(smem_u32(&sm->pv_empty[b]), DUO ? 256 : 128);
        }
        mbar_init(smem_u32(&sm->drain), 1);
        mbar_init(smem_u32(&sm->drain_pv), 1);
        mbar_init(smem_u32(&sm->mask_ready), DUO ? 256 : 128);
        for (int w = 0; w < MAX_UNITS_WORDS; ++w) sm->word_or[w] = 0ull;
        sm->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm->tmem_base)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (threadIdx.x == 0) pdl_trigger();
    const uint32_t tmem_base = sm->tmem_base;
    volatile int* abort_flag = &sm->abort_flag;

    // Units of this CTA: its share of the cache tiles first (known at once), then the node groups
    // dealt to this split - group w goes to split (splits - 1 - w mod splits) - that some query
    // row of the CTA can see.  Which groups are visible is known only after the mask rows have
    // arrived; every role waits for that (mask_ready) when it reaches the first node group, so
    // the mask's load latency hides behind the cache tiles.
    // (a length kept on the device was written at least two kernels ago: it may be read ahead of the dependency wait)
    const int kv_len = resolve_kv_len(p.kv_len, p.kv_len_dev, p.max_kv_len, p.n);
    const int n_cache = (kv_len + BN - 1) / BN;
    const int c_beg = n_cache * split / p.splits, c_end = n_cache * (split + 1) / p.splits;
    uint32_t cand = 0;
#pragma unroll
    for (int w = 0; w < MAX_UNITS_WORDS; ++w)
        if (!p.cache_only && w < p.n_words && p.splits - 1 - (w % p.splits) == split) cand |= 1u << w;
    // body(i, key0, w): unit number, first key row, node group (-1 for a cache tile); false stops the walk
    auto walk = [&](auto&& body) -> int {
        int i = 0;
        for (int c = c_beg; c < c_end; ++c) {
            if (!body(i, c * BN, -1)) return i;
            ++i;
        }
        if (cand) {
            mbar_wait(smem_u32(&sm->mask_ready), 0, abort_flag, p.status, DEV_TIMEOUT_EPI);
#pragma unroll
            for (int w = 0; w < MAX_UNITS_WORDS; ++w)
                if (((cand >> w) & 1u) && sm->word_or[w] != 0ull) {
                    if (!body(i, kv_len + 64 * w, w)) return i;
                    ++i;
                }
        }
        return i;
    };

    if (warp == 0) {
        // ------------------------------------------------ TMA producer
        if (lane == 0) {
            uint64_t pol_q, pol_kv;
            asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol_q));
            if (gridDim.z > 1) asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol_kv));
            else asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol_kv));
            auto load_kv = [&](uint32_t st, int key0) {
                const uint32_t full = smem_u32(&sm->kv_full[st]);
                const uint32_t k_dst = kv_addr + st * STAGE_BYTES, v_dst = k_dst + SLABS * KV_SLAB;
                mbar_expect_tx(full, STAGE_BYTES);
                // one request per operand: all 64-column slabs of the 64 rows
                tma_load_4d(k_dst, &tm_k, 0, key0, 0, h, full, pol_kv);
                tma_load_4d(v_dst, &tm_v, 0, key0, 0, h, full, pol_kv);
            };
            // cache tiles wholly below kv_len are not written by the preceding kernel: request the
            // first ring-full of them before waiting for that kernel to finish
            int pre = 0;
            for (int c = c_beg; c < c_end && pre < KV_STAGES && (c + 1) * BN <= kv_len; ++c, ++pre) load_kv(pre, c * BN);
            pdl_wait();
            uint32_t stage = 0, phase = 0;
            int issued = 0;
            bool ok = true;
            walk([&](int i, int key0, int) -> bool {
                if (i == 0) {
                    mbar_expect_tx(smem_u32(&sm->q_full), Q_BYTES);
#pragma unroll
                    for (int s = 0; s < SLABS; ++s) {
                        if constexpr (PAIR) {      // 64-row box, twice: rows 64..127 repeat rows 0..63
                            tma_load_2d(q_addr + s * Q_SLAB, &tm_q, h * DH + s * 64, 0, smem_u32(&sm->q_full), pol_q);
                            tma_load_2d(q_addr + s * Q_SLAB + 64 * 128, &tm_q, h * DH + s * 64, 0, smem_u32(&sm->q_full), pol_q);
                        } else {
                            tma_load_2d(q_addr + s * Q_SLAB, &tm_q, h * DH + s * 64, row0, smem_u32(&sm->q_full), pol_q);
                        }
                    }
                }
                if (i >= pre) {
                    if (issued >= KV_STAGES) ok = mbar_wait(smem_u32(&sm->kv_empty[stage]), phase ^ 1, abort_flag, p.status, DEV_TIMEOUT_TMA);
                    if (!ok) return false;
                    load_kv(stage, key0);
                }
                ++issued;
                if (++stage == KV_STAGES) { stage = 0; phase ^= 1; }
                return true;
            });
            if (!ok) {
                // drain: wait (bounded) for every load still in flight, and for Q
                const int outstanding = issued > pre ? issued : pre;
                const int inflight = outstanding < KV_STAGES ? outstanding : KV_STAGES;
                for (int q = 0; q < inflight; ++q) {
                    const int idx = outstanding - 1 - q;
                    for (uint32_t spin = 0; spin < SPIN_LIMIT && !mbar_try(smem_u32(&sm->kv_full[idx % KV_STAGES]), (idx / KV_STAGES) & 1); ++spin)
                        __nanosleep(64);
                }
                if (issued > 0)
                    for (uint32_t spin = 0; spin < SPIN_LIMIT && !mbar_try(smem_u32(&sm->q_full), 0); ++spin) __nanosleep(64);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ issuer of S = Q K^T
        if (lane == 0) {
            const uint32_t idesc_s = instr_desc_f16(BN, false);          // S: N = 64 keys, K tile K-major
            // operand descriptors are built once; per MMA only the 16-byte-unit address field moves
            const uint64_t q_desc = smem_desc_sw128(q_addr), k_desc = smem_desc_sw128(kv_addr);
            bool ok = true, have_q = false;
            walk([&](int i, int, int) -> bool {
                if (!have_q) {
                    ok = mbar_wait(smem_u32(&sm->q_full), 0, abort_flag, p.status, DEV_TIMEOUT_MMA);
                    have_q = true;
                }
                const int b = i & 1, stage = i % KV_STAGES;
                if (ok) ok = mbar_wait(smem_u32(&sm->kv_full[stage]), (i / KV_STAGES) & 1, abort_flag, p.status, DEV_TIMEOUT_MMA);
                if (ok && i >= 2) ok = mbar_wait(smem_u32(&sm->s_empty[b]), ((i >> 1) - 1) & 1, abort_flag, p.status, DEV_TIMEOUT_TMEM);
                if (!ok) return false;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + TMEM_S + b * BN;
                const uint64_t kd = k_desc + (uint64_t)((stage * STAGE_BYTES) >> 4);
#pragma unroll
                for (int s = 0; s < SLABS; ++s)
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks)
                        tc_mma_f16(d_tmem, q_desc + (uint64_t)(((s * Q_SLAB) >> 4) + ks * 2), kd + (uint64_t)(((s * KV_SLAB) >> 4) + ks * 2),
                                   idesc_s, (s > 0 || ks > 0) ? 1u : 0u);
                tc_commit(smem_u32(&sm->s_full[b]));
                return true;
            });
            if (!ok) {
                tc_commit(smem_u32(&sm->drain));
                for (uint32_t spin = 0; spin < SPIN_LIMIT && !mbar_try(smem_u32(&sm->drain), 0); ++spin) __nanosleep(64);
            }
        }
    } else if (warp == 6) {
        // ------------------------------------------------ issuer of PV = P V
        if (lane == 0) {
            const uint32_t idesc_pv = instr_desc_f16(DH, true);          // PV: N = d_head, V is N-major
            const uint64_t p_desc = smem_desc_sw128(p_addr);
            // V: rows = keys (the MMA K dimension), 64 d_head columns per 128-byte row, the next 64
            // columns one slab (KV_SLAB bytes) further: that distance is the leading-dimension offset
            const uint64_t v_desc = smem_desc_sw128(kv_addr + SLABS * KV_SLAB, KV_SLAB);
            bool ok = true;
            walk([&](int i, int, int) -> bool {
                const int b = i & 1, stage = i % KV_STAGES;
                ok = mbar_wait(smem_u32(&sm->p_full[b]), (i >> 1) & 1, abort_flag, p.status, DEV_TIMEOUT_MMA);
                if (ok && i >= 2) ok = mbar_wait(smem_u32(&sm->pv_empty[b]), ((i >> 1) - 1) & 1, abort_flag, p.status, DEV_TIMEOUT_TMEM);
                if (!ok) return false;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + TMEM_PV + b * DH;
                const uint64_t pd = p_desc + (uint64_t)((b * P_BYTES) >> 4);
                const uint64_t vd = v_desc + (uint64_t)((stage * STAGE_BYTES) >> 4);
#pragma unroll
                for (int ks = 0; ks < BN / 16; ++ks)     // 16 keys per MMA: +32 B along P's rows, +16 rows of V
                    tc_mma_f16(d_tmem, pd + (uint64_t)(ks * 2), vd + (uint64_t)((ks * 16 * 128) >> 4), idesc_pv, ks > 0 ? 1u : 0u);
                tc_commit(smem_u32(&sm->pv_full[b]));
                tc_commit(smem_u32(&sm->kv_empty[stage]));   // P V is the last reader of the stage (S of the same unit came first)
                tc_commit(smem_u32(&sm->p_empty[b]));
                return true;
            });
            if (!ok) {
                tc_commit(smem_u32(&sm->drain_pv));
                for (uint32_t spin = 0; spin < SPIN_LIMIT && !mbar_try(smem_u32(&sm->drain_pv), 0); ++spin) __nanosleep(64);
            }
        }
    } else if constexpr (PAIR || DUO) {
        // ------------------------------------------------ softmax warps, two threads per query row
        constexpr int HC = BN / 2;                             // keys of a unit per thread
        constexpr int HD = DH / 2;                             // d_head columns per thread
        constexpr int NT = DUO ? 256 : 128;                    // softmax threads
        const int quad = warp & 3;
        const int r = quad * 32 + lane;                        // tensor-memory lane
        // which half of the row's work; the row of the P tile this thread writes; its query row; its exchange slots
        const int half = DUO ? (warp >= 7 ? 1 : 0) : r >> 6;
        const int prow_i = DUO ? r : r & 63;
        const int row = DUO ? row0 + r : r & 63;
        const int xi = DUO ? half * QM + r : r, xpartner = DUO ? (half ^ 1) * QM + r : r ^ 64;
        const bool live = row < p.n;
        const bool warp_live = DUO ? row0 + quad * 32 < p.n : (quad & 1) * 32 < p.n;   // warps whose 32 rows are all padding skip the math
        const uint32_t lane_off = (uint32_t)(quad * 32) << 16;
        const float sl2 = p.scale * 1.4426950408889634f;       // scores are kept in the log2 domain
        pdl_wait();                                            // the mask comes from an earlier kernel
        unsigned long long myw[MAX_UNITS_WORDS];
#pragma unroll
        for (int w = 0; w < MAX_UNITS_WORDS; ++w) {
            myw[w] = (live && w < p.n_words) ? p.mask[(size_t)row * p.n_words + w] : 0ull;
            if (myw[w] && half == 0) atomicOr(&sm->word_or[w], myw[w]);
        }
        mbar_arrive(smem_u32(&sm->mask_ready));
        float m = -INFINITY, l = 0.f, corr_prev = 1.f;         // l: sum over this thread's keys only
        float o[HD];
#pragma unroll
        for (int c = 0; c < HD; ++c) o[c] = 0.f;
        if (!warp_live) {                                      // padding rows contribute zero rows of P, written once
#pragma unroll
            for (int bb = 0; bb < 2; ++bb)
#pragma unroll
                for (int ch = 0; ch < 8; ++ch) *reinterpret_cast<uint4*>(p_ptr + bb * P_BYTES + r * 128 + (ch << 4)) = make_uint4(0, 0, 0, 0);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        }

        auto fold_pv = [&](int i, float corr) {
            const int b = i & 1;
            mbar_wait(smem_u32(&sm->pv_full[b]), (i >> 1) & 1, abort_flag, p.status, DEV_TIMEOUT_EPI);
            if (warp_live) {
                tc_fence_after();
                if constexpr (HD == 64) {                      // both 32-column reads in flight, one wait
                    float v[64];
                    const uint32_t a0 = tmem_base + TMEM_PV + b * DH + half * HD + lane_off;
                    tc_ld32x2(a0, a0 + 32, v);
#pragma unroll
                    for (int j = 0; j < 64; ++j) o[j] = fmaf(o[j], corr, v[j]);
                } else {
#pragma unroll
                    for (int c0 = 0; c0 < HD; c0 += 32) {
                        float v[32];
                        tc_ld32(tmem_base + TMEM_PV + b * DH + half * HD + c0 + lane_off, v);
#pragma unroll
                        for (int j = 0; j < 32; ++j) o[c0 + j] = fmaf(o[c0 + j], corr, v[j]);
                    }
                }
                tc_fence_before();
            }
            mbar_arrive(smem_u32(&sm->pv_empty[b]));
        };

        const int cnt = walk([&](int i, int key0, int w) -> bool {
            const int b = i & 1;
            // visibility of this thread's 32 keys
            uint32_t bits = 0u;
            if (w < 0) {
                const int valid = kv_len - key0 - half * HC;
                if (live) bits = valid >= HC ? 0xffffffffu : (valid > 0 ? ((1u << valid) - 1u) : 0u);
            } else {
#pragma unroll
                for (int a = 0; a < MAX_UNITS_WORDS; ++a) if (a == w) bits = (uint32_t)(myw[a] >> (half * HC));
            }
            mbar_wait(smem_u32(&sm->s_full[b]), (i >> 1) & 1, abort_flag, p.status, DEV_TIMEOUT_EPI);
            if (!warp_live) {
                mbar_arrive(smem_u32(&sm->s_empty[b]));
                pair_bar<NT>();                                // every softmax thread takes part in the exchange barrier
                if (i >= 2) mbar_wait(smem_u32(&sm->p_empty[b]), ((i >> 1) - 1) & 1, abort_flag, p.status, DEV_TIMEOUT_EPI);
                mbar_arrive(smem_u32(&sm->p_full[b]));
                if (i >= 1) fold_pv(i - 1, 1.f);
                return true;
            }
            tc_fence_after();
            float s[HC];
            tc_ld32(tmem_base + TMEM_S + b * BN + half * HC + lane_off, s);
            tc_fence_before();
            mbar_arrive(smem_u32(&sm->s_empty[b]));
            if (bits != 0xffffffffu) {
#pragma unroll
                for (int j = 0; j < HC; ++j) s[j] = ((bits >> j) & 1u) ? s[j] : -INFINITY;
            }
            float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
            for (int j = 0; j < HC; j += 4) {
                mx[0] = fmaxf(mx[0], s[j]); mx[1] = fmaxf(mx[1], s[j + 1]);
                mx[2] = fmaxf(mx[2], s[j + 2]); mx[3] = fmaxf(mx[3], s[j + 3]);
            }
            const float mine = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
            sm->xmax[b][xi] = mine;                            // the partner thread holds the other 32 keys
            pair_bar<NT>();
            const float tmax = fmaxf(mine, sm->xmax[b][xpartner]) * sl2;
            const float m_new = fmaxf(m, tmax);
            const float neg = (m_new == -INFINITY) ? 0.f : -m_new;
            const float corr = (m_new == -INFINITY) ? 1.f : ex2_approx(m + neg);
            if (i >= 2) mbar_wait(smem_u32(&sm->p_empty[b]), ((i >> 1) - 1) & 1, abort_flag, p.status, DEV_TIMEOUT_EPI);
            // this thread's 32 probabilities go into the row (PAIR: into both copies, tile rows row and row + 64)
            uint8_t* prow = p_ptr + b * P_BYTES + prow_i * 128;
            float ps[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                uint32_t packed[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int j = q * 8 + 2 * e;
                    const float p0 = ex2_approx(fmaf(s[j], sl2, neg));
                    const float p1 = ex2_approx(fmaf(s[j + 1], sl2, neg));
                    ps[e] += p0 + p1;
                    const __half2 hh = __floats2half2_rn(p0, p1);
                    packed[e] = *reinterpret_cast<const uint32_t*>(&hh);
                }
                const uint32_t off = (uint32_t)(((half * 4 + q) ^ (prow_i & 7)) << 4);
                const uint4 val = make_uint4(packed[0], packed[1], packed[2], packed[3]);
                *reinterpret_cast<uint4*>(prow + off) = val;
                if constexpr (!DUO) *reinterpret_cast<uint4*>(prow + 64 * 128 + off) = val;
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            mbar_arrive(smem_u32(&sm->p_full[b]));
            l = l * corr + ((ps[0] + ps[1]) + (ps[2] + ps[3]));
            m = m_new;
            if (i >= 1) fold_pv(i - 1, corr_prev);
            corr_prev = corr;
            return true;
        });
        if (cnt > 0) fold_pv(cnt - 1, corr_prev);
        sm->xl[xi] = l;
        pair_bar<NT>();
        if (live) {
            float* po = p.part_o + ((size_t)split * p.max_nodes + row) * (size_t)(p.heads * DH) + h * DH + half * HD;
#pragma unroll
            for (int c = 0; c < HD; c += 4) *reinterpret_cast<float4*>(po + c) = make_float4(o[c], o[c + 1], o[c + 2], o[c + 3]);
            if (half == 0) {
                float* pm = p.part_ml + (((size_t)split * p.max_nodes + row) * p.heads + h) * 2;
                pm[0] = m * 0.6931471805599453f;               // back to the natural-log domain the merge kernel uses
                pm[1] = l + sm->xl[xpartner];
            }
        }
    } else {
        // ------------------------------------------------ softmax warps: thread = query row
        const int quad = warp & 3;
        const int r = quad * 32 + lane;                        // row inside the tile = tensor-memory lane
        const int row = row0 + r;
        const bool live = row < p.n;
        const bool warp_live = row0 + quad * 32 < p.n;         // warps whose 32 rows are all padding skip the math
        const uint32_t lane_off = (uint32_t)(quad * 32) << 16;
        const float sl2 = p.scale * 1.4426950408889634f;       // scores are kept in the log2 domain: s * scale * log2(e)
        pdl_wait();                                            // the mask comes from an earlier kernel
        // this row's mask words stay in registers; their OR over the CTA's rows tells every role
        // which node groups exist for this CTA
        unsigned long long myw[MAX_UNITS_WORDS];
#pragma unroll
        for (int w = 0; w < MAX_UNITS_WORDS; ++w) {
            myw[w] = (live && w < p.n_words) ? p.mask[(size_t)row * p.n_words + w] : 0ull;
            if (myw[w]) atomicOr(&sm->word_or[w], myw[w]);
        }
        mbar_arrive(smem_u32(&sm->mask_ready));
        float m = -INFINITY, l = 0.f, corr_prev = 1.f;
        float o[DH];
#pragma unroll
        for (int c = 0; c < DH; ++c) o[c] = 0.f;
        if (!warp_live) {                                      // padding rows contribute zero rows of P, written once
#pragma unroll
            for (int bb = 0; bb < 2; ++bb)
#pragma unroll
                for (int ch = 0; ch < 8; ++ch) *reinterpret_cast<uint4*>(p_ptr + bb * P_BYTES + r * 128 + (ch << 4)) = make_uint4(0, 0, 0, 0);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        }

        auto fold_pv = [&](int i, float corr) {
            const int b = i & 1;
            mbar_wait(smem_u32(&sm->pv_full[b]), (i >> 1) & 1, abort_flag, p.status, DEV_TIMEOUT_EPI);
            if (warp_live) {
                tc_fence_after();
#pragma unroll
                for (int c0 = 0; c0 < DH; c0 += 64) {          // two 32-column reads in flight per wait
                    float v[64];
                    const uint32_t a0 = tmem_base + TMEM_PV + b * DH + c0 + lane_off;
                    tc_ld32x2(a0, a0 + 32, v);
#pragma unroll
                    for (int j = 0; j < 64; ++j) o[c0 + j] = fmaf(o[c0 + j], corr, v[j]);
                }
                tc_fence_before();
            }
            mbar_arrive(smem_u32(&sm->pv_empty[b]));
        };

        const int cnt = walk([&](int i, int key0, int w) -> bool {
            const int b = i & 1;
            // visibility of the 64 keys of this unit for this row
            unsigned long long vis = 0ull;
            if (w < 0) {
                const int valid = kv_len - key0;
                if (live) vis = valid >= 64 ? ~0ull : ((1ull << valid) - 1ull);
            } else {
#pragma unroll
                for (int a = 0; a < MAX_UNITS_WORDS; ++a) if (a == w) vis = myw[a];
            }
            mbar_wait(smem_u32(&sm->s_full[b]), (i >> 1) & 1, abort_flag, p.status, DEV_TIMEOUT_EPI);
            if (!warp_live) {
                mbar_arrive(smem_u32(&sm->s_empty[b]));
                if (i >= 2) mbar_wait(smem_u32(&sm->p_empty[b]), ((i >> 1) - 1) & 1, abort_flag, p.status, DEV_TIMEOUT_EPI);
                mbar_arrive(smem_u32(&sm->p_full[b]));
                if (i >= 1) fold_pv(i - 1, 1.f);
                return true;
            }
            tc_fence_after();
            float s[BN];
            tc_ld32x2(tmem_base + TMEM_S + b * BN + lane_off, tmem_base + TMEM_S + b * BN + 32 + lane_off, s);
            tc_fence_before();
            mbar_arrive(smem_u32(&sm->s_empty[b]));
            // hidden keys become -inf once; exp2(-inf) = 0 then needs no further selects
            if (vis != ~0ull) {
#pragma unroll
                for (int j = 0; j < BN; ++j) s[j] = ((vis >> j) & 1ull) ? s[j] : -INFINITY;
            }
            float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
            for (int j = 0; j < BN; j += 4) {
                mx[0] = fmaxf(mx[0], s[j]); mx[1] = fmaxf(mx[1], s[j + 1]);
                mx[2] = fmaxf(mx[2], s[j + 2]); mx[3] = fmaxf(mx[3], s[j + 3]);
            }
            const float tmax = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) * sl2;
            const float m_new = fmaxf(m, tmax);
            const float neg = (m_new == -INFINITY) ? 0.f : -m_new;
            const float corr = (m_new == -INFINITY) ? 1.f : ex2_approx(m + neg);      // m = -inf gives 0
            // P row -> shared memory, K-major with the 128-byte swizzle the MMA descriptor expects
            if (i >= 2) mbar_wait(smem_u32(&sm->p_empty[b]), ((i >> 1) - 1) & 1, abort_flag, p.status, DEV_TIMEOUT_EPI);
            uint8_t* prow = p_ptr + b * P_BYTES + r * 128;
            float ps[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int ch = 0; ch < 8; ++ch) {
                uint32_t packed[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int j = ch * 8 + 2 * e;
                    const float p0 = ex2_approx(fmaf(s[j], sl2, neg));
                    const float p1 = ex2_approx(fmaf(s[j + 1], sl2, neg));
                    ps[e] += p0 + p1;
                    const __half2 hh = __floats2half2_rn(p0, p1);
                    packed[e] = *reinterpret_cast<const uint32_t*>(&hh);
                }
                *reinterpret_cast<uint4*>(prow + ((ch ^ (r & 7)) << 4)) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            mbar_arrive(smem_u32(&sm->p_full[b]));
            l = l * corr + ((ps[0] + ps[1]) + (ps[2] + ps[3]));
            m = m_new;
            if (i >= 1) fold_pv(i - 1, corr_prev);
            corr_prev = corr;
            return true;
        });
        if (cnt > 0) fold_pv(cnt - 1, corr_prev);
        if (live) {
            float* po = p.part_o + ((size_t)split * p.max_nodes + row) * (size_t)(p.heads * DH) + h * DH;
#pragma unroll
            for (int c = 0; c < DH; c += 4) *reinterpret_cast<float4*>(po + c) = make_float4(o[c], o[c + 1], o[c + 2], o[c + 3]);
            float* pm = p.part_ml + (((size_t)split * p.max_nodes + row) * p.heads + h) * 2;
            pm[0] = m * 0.6931471805599453f;                   // back to the natural-log domain the merge kernel uses
            pm[1] = l;
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    }
}

template <int DH>
size_t attn_smem_bytes() {
    return 1024 + (size_t)(DH / 64) * QM * 128 + (size_t)KV_STAGES * 2 * (DH / 64) * BN * 128 + 2 * QM * 128 + sizeof(AttnSmem);
}

}  // namespace

bool attn_tc_supported(const ghd_ctx* c, const ghd_tree* t) {
    return c->cfg.dtype == GHD_F16 && (c->cfg.d_head == 64 || c->cfg.d_head == 128) && t->n >= 1;
}

ghd_status launch_attn_tc(ghd_ctx* c, const void* q, const ghd_kv_layer* kv, const ghd_tree* t, void* out, bool coo) {
    const ghd_model_cfg& m = c->cfg;
    const int n = t->n, H = m.n_heads, dh = m.d_head, d = m.d_model;
    // rows the K/V maps cover: past them a load returns zeros.  With the length on the device the maps cover the
    // whole cache and rows past kv_len + n (weight exactly zero) must hold finite numbers.
    const int kt = t->kv_len < 0 ? m.max_kv_len : t->kv_len + n;
    if (((uintptr_t)q & 15) || ((uintptr_t)kv->k & 15) || ((uintptr_t)kv->v & 15)) {
        snprintf(c->err, sizeof(c->err), "tcgen05 attention: operands must be 16-byte aligned");
        return GHD_EINVAL;
    }
    // The kernel with 128-key units, four softmax threads per row and the accumulator resident in tensor memory
    // (attn_tc_small.cu): as measured it wins from about 1024 cache rows on (attention + merge, 64 nodes: 19.8 -> 16.8 us
    // at KV 2048, 27.5 -> 22.5 us at KV 4096; 256 nodes: 43.1 -> 36.5 us and 62.0 -> 50.7 us) and is level or up to
    // 1.5 us behind on caches of 256-512 rows.
    const bool small = c->opt_attn_small == 1 || (c->opt_attn_small == 0 && kv_len_host_of(c, t) >= 1024);
    if (small) {
        ghd_status st;
        const int s = launch_attn_tc_small(c, q, kv, t, coo, &st);
        if (s <= 0) return st;
        if (coo) launch_attn_coo(c, q, kv, t, s);
        launch_attn_combine(c, out, s + (coo ? 1 : 0), n);
        return GHD_OK;
    }
    CUtensorMap tm_q, tm_k, tm_v;
    const bool pair = n <= 64;                           // two threads per query row (queries loaded twice)
    if (!tmap_rows_x_k(c, q, (uint64_t)n, (uint64_t)d, pair ? 64 : QM, &tm_q) ||
        !tmap_planes_slabs(c, kv->k, (uint64_t)H, (uint64_t)m.max_kv_len, (uint64_t)kt, (uint64_t)dh, BN, &tm_k) ||
        !tmap_planes_slabs(c, kv->v, (uint64_t)H, (uint64_t)m.max_kv_len, (uint64_t)kt, (uint64_t)dh, BN, &tm_v)) {
        snprintf(c->err, sizeof(c->err), "tcgen05 attention: tensor map encoding failed");
        return GHD_ECUDA;
    }
    const int mtiles = (n + QM - 1) / QM;
    const int units = (kv_len_host_of(c, t) + BN - 1) / BN + (coo ? 0 : t->n_words);
    int splits = c->opt_attn_splits;
    if (splits <= 0) {
        splits = c->sm_count / (H * mtiles);
        const int by_len = (units + 1) / 2;              // at least two units per split
        if (splits > by_len) splits = by_len;
    }
    if (splits > c->max_splits - (coo ? 1 : 0)) splits = c->max_splits - (coo ? 1 : 0);    // the index kernel's partial takes a slot
    if (splits < 1) splits = 1;
    AttnParams p{};
    p.cache_only = coo ? 1 : 0;
    p.n = n; p.heads = H; p.kv_len = t->kv_len; p.kv_len_dev = kv_len_dev_of(c, t); p.max_kv_len = m.max_kv_len; p.max_nodes = m.max_nodes; p.splits = splits; p.n_words = t->n_words;
    p.mask = t->mask; p.part_o = c->att_o; p.part_ml = c->att_ml; p.status = c->status;
    p.scale = 1.0f / sqrtf((float)dh);
    dim3 grid(splits, H, mtiles);
    if (!c->attr_attn) {       // per context: the attribute belongs to the device the context was created on
        const int b64 = (int)attn_smem_bytes<64>(), b128 = (int)attn_smem_bytes<128>();
        if (cudaFuncSetAttribute(k_attn_tc<64, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, b64) != cudaSuccess ||
            cudaFuncSetAttribute(k_attn_tc<64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, b64) != cudaSuccess ||
            cudaFuncSetAttribute(k_attn_tc<128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, b128) != cudaSuccess ||
            cudaFuncSetAttribute(k_attn_tc<128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, b128) != cudaSuccess ||
            cudaFuncSetAttribute(k_attn_tc<64, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, b64) != cudaSuccess ||
            cudaFuncSetAttribute(k_attn_tc<128, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, b128) != cudaSuccess) {
            snprintf(c->err, sizeof(c->err), "tcgen05 attention: cannot raise dynamic shared memory");
            cudaGetLastError();
            return GHD_ECUDA;
        }
        c->attr_attn = true;
    }
    const bool duo = !pair && c->opt_attn_rows != 1;     // more than 64 rows: two softmax warpgroups share the rows
    if (dh == 64) {
        if (pair) launch_k(c, true, k_attn_tc<64, true>, grid, THREADS, attn_smem_bytes<64>(), tm_q, tm_k, tm_v, p);
        else if (duo) launch_k(c, true, k_attn_tc<64, false, true>, grid, THREADS_DUO, attn_smem_bytes<64>(), tm_q, tm_k, tm_v, p);
        else launch_k(c, true, k_attn_tc<64, false>, grid, THREADS, attn_smem_bytes<64>(), tm_q, tm_k, tm_v, p);
    } else {
        if (pair) launch_k(c, true, k_attn_tc<128, true>, grid, THREADS, attn_smem_bytes<128>(), tm_q, tm_k, tm_v, p);
        else if (duo) launch_k(c, true, k_attn_tc<128, false, true>, grid, THREADS_DUO, attn_smem_bytes<128>(), tm_q, tm_k, tm_v, p);
        else launch_k(c, true, k_attn_tc<128, false>, grid, THREADS, attn_smem_bytes<128>(), tm_q, tm_k, tm_v, p);
    }
    if (coo) launch_attn_coo(c, q, kv, t, splits);       // the sparse part as one more partial, slot `splits`
    launch_attn_combine(c, out, splits + (coo ? 1 : 0), n);
    return GHD_OK;
}

}  // namespace ghd
