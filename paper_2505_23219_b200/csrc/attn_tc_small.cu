// Tree attention on the tensor cores (sm_100a, half in, float softmax/accumulate) with 128-key units, four softmax
// threads per query row and the output accumulator kept in tensor memory: the kernel for long caches.
//
// One CTA = one head x one tile of query rows x one KV split.  FOUR threads share a query row.  Up to 64 nodes
// (k_attn_small): the queries are loaded twice (tile rows r and r + 64 hold the same query; the copy picks a 64-key
// half of a unit and a half of d_head) and two groups of four softmax warps work on the same tensor-memory lanes (the
// group picks 32 of those 64 keys).  More nodes (k_attn_wide): 128 distinct rows per CTA and four such groups.
// The per-unit softmax work of a thread - one 32-column read of S, 32 exponentials, four 16-byte stores of P - is
// what the unit chain waits for, so spreading it over 256 threads shortens every unit.
// Keys are walked in 128-key units: the cache rows [0, kv_len) first (the dense part), then the new rows as one
// group of up to 128 nodes (the sparse part, masked by the packed ancestor bitmask; dropped when no query of the
// CTA sees any of them).  Every unit costs a fixed chain of hand-overs between the asynchronous units
// (TMA -> S MMA -> softmax threads -> PV MMA), about as long as the arithmetic of 64 keys, hence the large units;
// and the accumulator [128 x d_head] stays in tensor memory over all units: the probabilities are taken against a
// reference maximum that is raised only when a unit's maximum exceeds it by more than 2^8 (raising it rescales the
// accumulator in place, rare after the first unit), so no unit reads the accumulator back.
// K and V tiles of a unit travel separately (K is free again after S, V after PV).
//
// The un-normalised (o, max, sum) of a split go to the workspace; k_attn_combine_rows merges the splits
// (paper Sec. III-B-2).  Warp 0 = TMA producer, warp 1 = issuer of the S MMAs + tensor-memory owner, warps 2..5 and
// 7..10 = softmax (a warp may touch the tensor-memory lanes 32 (w mod 4) ..), warp 6 = issuer of the PV MMAs.  All
// waits are bounded.  Cache
// tiles that lie wholly below kv_len cannot be touched by the preceding kernel, so the producer requests the first
// of them, and asks the L2 for the rest, before it waits for that kernel to finish.
#include <cstdio>

#include "internal.h"
#include "tc_common.cuh"

namespace ghd {

namespace {

using namespace tc;

constexpr int QM = 128;        // query rows per CTA (MMA M)
constexpr int THREADS_DUP = 352;   // producer, S issuer, four softmax warps, PV issuer, four more softmax warps
constexpr int THREADS_WIDE = 608;  // ... and eight more: four groups of four softmax warps
constexpr int MAX_UNITS_WORDS = GHD_MAX_NODES / 64;
constexpr int NODE_WEIGHT = 2;     // cost of a node-group unit in cache-tile units, for the split of a head
constexpr int CTRL_BYTES = 1536;   // control block behind the tiles

struct AttnParams {
    int n, heads, kv_len, max_nodes, splits, n_words;
    const int* kv_len_dev;     // non-null: the cache length comes from this device word
    int max_kv_len;
    int cache_only;            // 1: the new rows are somebody else's (the coordinate-index kernel): no node group here
    const uint64_t* mask;
    float* part_o;             // [splits][max_nodes][heads * d_head] un-normalised numerators
    float* part_ml;            // [splits][max_nodes][heads][2] running max (natural log domain), running sum
    int* status;
    float scale;               // 1 / sqrt(d_head)
};

template <int DH>
struct Shape {
    // Keys per unit (MMA N of S, MMA K of PV).  Every unit costs a fixed chain of hand-overs between the
    // asynchronous units (TMA -> S MMA -> softmax threads -> PV MMA -> softmax threads), about as long as the
    // arithmetic of 64 keys, so the small-tree shape, whose threads hold half a row each, takes 128 keys a unit.
    static constexpr int BN = 128;
    static constexpr int KSL = BN / 64;                         // 64-key slabs of a P row
    static constexpr int SLABS = DH / 64;                       // 64-wide (128-byte) column slabs of a d_head row
    static constexpr uint32_t Q_SLAB = QM * 128;                // bytes of one [128 x 64] half slab
    static constexpr uint32_t KV_SLAB = BN * 128;               // bytes of one [BN x 64] half slab
    static constexpr uint32_t Q_BYTES = SLABS * Q_SLAB;
    static constexpr uint32_t STAGE_BYTES = 2 * SLABS * KV_SLAB;   // K slabs then V slabs
    static constexpr uint32_t P_BYTES = KSL * QM * 128;         // [128 x BN] half as KSL slabs of [128 x 64]
    static constexpr int KV_STAGES = DH == 128 ? 2 : 4;
    static constexpr int P_BUFS = 2;
    static constexpr int PV_BUFS = 1;                           // one output accumulator that stays in tensor memory
    static constexpr uint32_t TMEM_S = 0, TMEM_PV = 2 * BN;     // columns: S[2] then PV[PV_BUFS]
    static constexpr uint32_t TMEM_COLS = (2 * BN + PV_BUFS * DH) <= 256 ? 256 : 512;
    static constexpr uint32_t TILE_BYTES = Q_BYTES + KV_STAGES * STAGE_BYTES + P_BUFS * P_BYTES;
    // dynamic shared memory asked for: the tiles need a 1024-byte-aligned base, which a kernel without static
    // shared memory gets; the kernel checks and refuses to run otherwise
    static constexpr uint32_t SMEM_BYTES = TILE_BYTES + CTRL_BYTES + 1024;     // + room to align the base
};

struct AttnSmem {
    uint64_t q_full;
    uint64_t k_full[4], k_empty[4], v_full[4], v_empty[4];   // K and V tiles of a unit travel separately: K is free again after S, V after PV
    uint64_t s_full[2], s_empty[2], p_full[2], p_empty[2], pv_full[2], pv_empty[2];
    uint64_t drain, drain_pv;
    uint64_t mask_ready;          // all softmax threads have merged their mask words into word_or
    unsigned long long word_or[MAX_UNITS_WORDS];
    uint32_t tmem_base;
    int abort_flag;
    float xch[2][QM];             // the four threads of a row exchange their partial maxima: float [2][128] when the rows are
                                  // duplicated, bfloat16 [4][128] (as uint16) when four warp groups share 128 distinct rows
};
static_assert(sizeof(AttnSmem) <= CTRL_BYTES, "control block too large");

template <int NT> __device__ __forceinline__ void pair_bar() { asm volatile("bar.sync 2, %0;" ::"n"(NT) : "memory"); }     // all softmax threads

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// End of a split, run by a softmax thread that holds COLS un-normalised output columns [col0, col0 + COLS) of query
// row `row` (m in the log2 domain, l = the row's sum over this split): the partial goes to the workspace.
template <int DH, int COLS>
__device__ __forceinline__ void leave_partial(const AttnParams& p, int split, int h, int row, int col0, bool live, bool writes_ml,
                                              const float (&o)[COLS], float m, float l) {
    if (!live) return;
    float* po = p.part_o + ((size_t)split * p.max_nodes + row) * (size_t)(p.heads * DH) + h * DH + col0;
#pragma unroll
    for (int c = 0; c < COLS; c += 4) *reinterpret_cast<float4*>(po + c) = make_float4(o[c], o[c + 1], o[c + 2], o[c + 3]);
    if (writes_ml) {
        float* pm = p.part_ml + (((size_t)split * p.max_nodes + row) * p.heads + h) * 2;
        pm[0] = m * 0.6931471805599453f;                   // back to the natural-log domain the merge kernel uses
        pm[1] = l;
    }
}

// At most 64 query rows.  The queries are loaded twice (tile rows r and r + 64 hold the same query), so S, P and
// PV come out duplicated and two threads share a row: thread r takes the first 64 keys of a unit and the first
// half of d_head, thread r + 64 the rest.
template <int DH, bool DUP>
__device__ __forceinline__ void attn_body(const CUtensorMap& tm_q, const CUtensorMap& tm_k, const CUtensorMap& tm_v, const AttnParams& p) {
    using SH = Shape<DH>;
    constexpr int SLABS = SH::SLABS;
    constexpr uint32_t Q_SLAB = SH::Q_SLAB, KV_SLAB = SH::KV_SLAB, Q_BYTES = SH::Q_BYTES, STAGE_BYTES = SH::STAGE_BYTES, P_BYTES = SH::P_BYTES;
    constexpr int KV_STAGES = SH::KV_STAGES, P_BUFS = SH::P_BUFS, PV_BUFS = SH::PV_BUFS, BN = SH::BN, KSL = SH::KSL;
    constexpr uint32_t TMEM_S = SH::TMEM_S, TMEM_PV = SH::TMEM_PV, TMEM_COLS = SH::TMEM_COLS;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t pad = (1024u - (raw_addr & 1023u)) & 1023u;      // the swizzled tiles need a 1024-byte-aligned base
    uint8_t* base = smem_raw + pad;
    AttnSmem* sm = reinterpret_cast<AttnSmem*>(base + SH::TILE_BYTES);
    const uint32_t q_addr = smem_u32(base);
    const uint32_t kv_addr = q_addr + Q_BYTES;
    const uint32_t p_addr = kv_addr + KV_STAGES * STAGE_BYTES;
    uint8_t* p_ptr = base + Q_BYTES + KV_STAGES * STAGE_BYTES;
    constexpr bool runnable = true;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int split = blockIdx.x, h = blockIdx.y;
    const int row0 = DUP ? 0 : (int)blockIdx.z * QM;        // first query row of this CTA's tile
    constexpr int NT = DUP ? 256 : 512;                    // softmax threads

    if (threadIdx.x == 32) {        // descriptor fetches overlap the barrier set-up
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_q) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_k) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_v) : "memory");
    }
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&sm->q_full), 1);
        for (int s = 0; s < KV_STAGES; ++s) {
            mbar_init(smem_u32(&sm->k_full[s]), 1); mbar_init(smem_u32(&sm->k_empty[s]), 1);
            mbar_init(smem_u32(&sm->v_full[s]), 1); mbar_init(smem_u32(&sm->v_empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&sm->s_full[b]), 1);
            mbar_init(smem_u32(&sm->s_empty[b]), NT);
            mbar_init(smem_u32(&sm->p_full[b]), NT);
            mbar_init(smem_u32(&sm->p_empty[b]), 1);
            mbar_init(smem_u32(&sm->pv_full[b]), 1);
            mbar_init(smem_u32(&sm->pv_empty[b]), NT);
        }
        mbar_init(smem_u32(&sm->drain), 1);
        mbar_init(smem_u32(&sm->drain_pv), 1);
        mbar_init(smem_u32(&sm->mask_ready), NT);
        for (int w = 0; w < MAX_UNITS_WORDS; ++w) sm->word_or[w] = 0ull;
        sm->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm->tmem_base)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (threadIdx.x == 0) pdl_trigger();
    const uint32_t tmem_base = sm->tmem_base;
    volatile int* abort_flag = &sm->abort_flag;

    // Units of this CTA: the head's units - cache tiles first, then the node groups - are numbered
    // 0 .. n_cache + n_words - 1 and split s takes an even contiguous share.  Which node groups are
    // visible to some query row of the CTA is known only after the mask rows have arrived; every
    // role waits for that (mask_ready) when it reaches the first node group, so the mask's load
    // latency hides behind the cache tiles.  An invisible group is skipped by every role alike.
    // (a length kept on the device was written at least two kernels ago: it may be read ahead of the dependency wait)
    const int kv_len = resolve_kv_len(p.kv_len, p.kv_len_dev, p.max_kv_len, p.n);
    const int n_cache = (kv_len + BN - 1) / BN;
    const int n_groups = p.cache_only ? 0 : (p.n_words + KSL - 1) / KSL;      // node groups of BN nodes = KSL mask words each
    const int n_units = n_cache + n_groups;
    // Even shares by cost: a node group weighs NODE_WEIGHT cache tiles (its rows exist only once the preceding
    // kernel has finished, so its load cannot be requested ahead like a cache tile's).  Unit u sits at
    // position u (cache tile) or n_cache + NODE_WEIGHT * g (node group g) and goes to the split whose share
    // [W * s / splits, W * (s + 1) / splits) of the total weight W holds that position.
    const int wtot = n_cache + NODE_WEIGHT * n_groups;
    auto first_unit_of = [&](int s_) -> int {
        const int pos = (wtot * s_ + p.splits - 1) / p.splits;        // first position of split s_ (ceiling)
        if (pos <= n_cache) return pos;
        const int g = (pos - n_cache + NODE_WEIGHT - 1) / NODE_WEIGHT;
        return n_cache + (g < n_groups ? g : n_groups);
    };
    const int u_beg = first_unit_of(split), u_end = (split + 1 == p.splits) ? n_units : first_unit_of(split + 1);
    // body(i, key0, g): unit number within the CTA, first key row, node group (-1 for a cache tile); false stops the walk
    auto walk = [&](auto&& body) -> int {
        int i = 0;
        bool have_mask = false;
        for (int u = u_beg; u < u_end; ++u) {
            if (u < n_cache) {
                if (!body(i, u * BN, -1)) return i;
                ++i;
                continue;
            }
            if (!have_mask) {
                mbar_wait(smem_u32(&sm->mask_ready), 0, abort_flag, p.status, DEV_TIMEOUT_EPI);
                have_mask = true;
            }
            const int g = u - n_cache;
            unsigned long long any = 0ull;
#pragma unroll
            for (int k = 0; k < KSL; ++k)
                if (g * KSL + k < MAX_UNITS_WORDS) any |= sm->word_or[g * KSL + k];
            if (any != 0ull) {
                if (!body(i, kv_len + BN * g, g)) return i;
                ++i;
            }
        }
        return i;
    };

    // The same enumeration, one unit per call (the producer keeps two cursors): u is the cursor, key0 the
    // unit's first key row; false at the end.
    auto next_unit = [&](int& u, int& key0, bool& have_mask) -> bool {
        for (; u < u_end; ++u) {
            if (u < n_cache) { key0 = u * BN; ++u; return true; }
            if (!have_mask) {
                mbar_wait(smem_u32(&sm->mask_ready), 0, abort_flag, p.status, DEV_TIMEOUT_EPI);
                have_mask = true;
            }
            const int g = u - n_cache;
            unsigned long long any = 0ull;
#pragma unroll
            for (int k = 0; k < KSL; ++k)
                if (g * KSL + k < MAX_UNITS_WORDS) any |= sm->word_or[g * KSL + k];
            if (any != 0ull) { key0 = kv_len + BN * g; ++u; return true; }
        }
        return false;
    };

    if (!runnable) {
        // nothing: fall through to the common exit
    } else if (warp == 0) {
        // ------------------------------------------------ TMA producer
        if (lane == 0) {
            uint64_t pol_q, pol_kv;
            asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol_q));
            if (gridDim.z > 1) asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol_kv));
            else asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol_kv));
            constexpr uint32_t OPERAND_BYTES = SLABS * KV_SLAB;      // one K or one V tile: all 64-column slabs of BN rows
            // one request per operand tile
            auto load_k = [&](int i, int key0) {
                const uint32_t st = (uint32_t)(i % KV_STAGES), full = smem_u32(&sm->k_full[st]);
                mbar_expect_tx(full, OPERAND_BYTES);
                tma_load_4d(kv_addr + st * STAGE_BYTES, &tm_k, 0, key0, 0, h, full, pol_kv);
            };
            auto load_v = [&](int i, int key0) {
                const uint32_t st = (uint32_t)(i % KV_STAGES), full = smem_u32(&sm->v_full[st]);
                mbar_expect_tx(full, OPERAND_BYTES);
                tma_load_4d(kv_addr + st * STAGE_BYTES + OPERAND_BYTES, &tm_v, 0, key0, 0, h, full, pol_kv);
            };
            // cache tiles wholly below kv_len are not written by the preceding kernel: request the
            // first ring-full of them before waiting for that kernel to finish
            int pre = 0;
            for (int u = u_beg; u < u_end && u < n_cache && pre < KV_STAGES && (u + 1) * BN <= kv_len; ++u, ++pre) { load_k(pre, u * BN); load_v(pre, u * BN); }
            // ... and pull the rest of this CTA's cache tiles into L2 right away: a tile requested when its slot
            // frees up would otherwise pay the full HBM latency inside the unit chain
            for (int u = u_beg + pre; u < u_end && u < n_cache; ++u) {
                tma_prefetch_4d(&tm_k, 0, u * BN, 0, h);
                tma_prefetch_4d(&tm_v, 0, u * BN, 0, h);
            }
            pdl_wait();
            // Two cursors over this CTA's units: K tiles run one unit ahead of V tiles (order K0 K1 V0 K2 V1 ...).
            // A K slot is free as soon as the S product of two units back has completed, a V slot only after that
            // unit's PV product: waiting for the V slot first would hold the next K back for no reason.
            int uk = u_beg, uv = u_beg, ik = 0, iv = 0, key_k = 0, key_v = 0;
            bool mask_k = false, mask_v = false, ok = true;
            bool more_k = next_unit(uk, key_k, mask_k), more_v = next_unit(uv, key_v, mask_v);
            if (more_k) {
                mbar_expect_tx(smem_u32(&sm->q_full), Q_BYTES);
#pragma unroll
                for (int s = 0; s < SLABS; ++s) {
                    if constexpr (DUP) {       // 64-row box, twice: rows 64..127 repeat rows 0..63
                        tma_load_2d(q_addr + s * Q_SLAB, &tm_q, h * DH + s * 64, 0, smem_u32(&sm->q_full), pol_q);
                        tma_load_2d(q_addr + s * Q_SLAB + 64 * 128, &tm_q, h * DH + s * 64, 0, smem_u32(&sm->q_full), pol_q);
                    } else {
                        tma_load_2d(q_addr + s * Q_SLAB, &tm_q, h * DH + s * 64, row0, smem_u32(&sm->q_full), pol_q);
                    }
                }
            }
            while (ok && (more_k || more_v)) {
                if (more_k) {
                    if (ik >= pre) {
                        if (ik >= KV_STAGES) ok = mbar_wait(smem_u32(&sm->k_empty[ik % KV_STAGES]), ((ik / KV_STAGES) - 1) & 1, abort_flag, p.status, DEV_TIMEOUT_TMA);
                        if (!ok) break;
                        load_k(ik, key_k);
                    }
                    ++ik;
                    more_k = next_unit(uk, key_k, mask_k);
                }
                if (more_v && (iv + 1 < ik || !more_k)) {
                    if (iv >= pre) {
                        if (iv >= KV_STAGES) ok = mbar_wait(smem_u32(&sm->v_empty[iv % KV_STAGES]), ((iv / KV_STAGES) - 1) & 1, abort_flag, p.status, DEV_TIMEOUT_TMA);
                        if (!ok) break;
                        load_v(iv, key_v);
                    }
                    ++iv;
                    more_v = next_unit(uv, key_v, mask_v);
                }
            }
            if (!ok) {
                // drain: wait (bounded) for every load still in flight, and for Q
                const int nk = ik > pre ? ik : pre, nv = iv > pre ? iv : pre;
                for (int idx = (nk > KV_STAGES ? nk - KV_STAGES : 0); idx < nk; ++idx)
                    for (uint32_t spin = 0; spin < SPIN_LIMIT && !mbar_try(smem_u32(&sm->k_full[idx % KV_STAGES]), (idx / KV_STAGES) & 1); ++spin) __nanosleep(64);
                for (int idx = (nv > KV_STAGES ? nv - KV_STAGES : 0); idx < nv; ++idx)
                    for (uint32_t spin = 0; spin < SPIN_LIMIT && !mbar_try(smem_u32(&sm->v_full[idx % KV_STAGES]), (idx / KV_STAGES) & 1); ++spin) __nanosleep(64);
                if (ik > 0 || iv > 0)
                    for (uint32_t spin = 0; spin < SPIN_LIMIT && !mbar_try(smem_u32(&sm->q_full), 0); ++spin) __nanosleep(64);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ issuer of S = Q K^T
        if (lane == 0) {
            const uint32_t idesc_s = instr_desc_f16(BN, false);          // S: N = BN keys, K tile K-major
            // operand descriptors are built once; per MMA only the 16-byte-unit address field moves
            const uint64_t q_desc = smem_desc_sw128(q_addr), k_desc = smem_desc_sw128(kv_addr);
            bool ok = true, have_q = false;
            walk([&](int i, int, int) -> bool {
                if (!have_q) {
                    ok = mbar_wait(smem_u32(&sm->q_full), 0, abort_flag, p.status, DEV_TIMEOUT_MMA);
                    have_q = true;
                }
                const int b = i & 1, stage = i % KV_STAGES;
                if (ok) ok = mbar_wait(smem_u32(&sm->k_full[stage]), (i / KV_STAGES) & 1, abort_flag, p.status, DEV_TIMEOUT_MMA);
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
                tc_commit(smem_u32(&sm->k_empty[stage]));    // the K tile is free once this product has read it
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
                const int pb = i % P_BUFS, vb = i % PV_BUFS, stage = i % KV_STAGES;
                ok = mbar_wait(smem_u32(&sm->v_full[stage]), (i / KV_STAGES) & 1, abort_flag, p.status, DEV_TIMEOUT_MMA);
                if (ok) ok = mbar_wait(smem_u32(&sm->p_full[pb]), (i / P_BUFS) & 1, abort_flag, p.status, DEV_TIMEOUT_MMA);
                // the accumulator is never handed back, every unit adds to it (the softmax threads rescale it in place,
                // before they publish the P that needs the new scale)
                if (!ok) return false;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + TMEM_PV + vb * DH;
                const uint64_t pd = p_desc + (uint64_t)((pb * P_BYTES) >> 4);
                const uint64_t vd = v_desc + (uint64_t)((stage * STAGE_BYTES) >> 4);
#pragma unroll
                for (int ks = 0; ks < BN / 16; ++ks)     // 16 keys per MMA: +32 B along P's rows (next slab after 64 keys), +16 rows of V
                    tc_mma_f16(d_tmem, pd + (uint64_t)((((ks >> 2) * (QM * 128)) >> 4) + (ks & 3) * 2), vd + (uint64_t)((ks * 16 * 128) >> 4),
                               idesc_pv, (ks > 0 || i > 0) ? 1u : 0u);
                tc_commit(smem_u32(&sm->pv_full[vb]));
                tc_commit(smem_u32(&sm->v_empty[stage]));    // the V tile is free once this product has read it
                tc_commit(smem_u32(&sm->p_empty[pb]));
                return true;
            });
            if (!ok) {
                tc_commit(smem_u32(&sm->drain_pv));
                for (uint32_t spin = 0; spin < SPIN_LIMIT && !mbar_try(smem_u32(&sm->drain_pv), 0); ++spin) __nanosleep(64);
            }
        }
    } else if ((warp >= 2 && warp <= 5) || warp >= 7) {
        // ------------------------------------------------ softmax warps
        // FOUR threads per query row, each with 32 of a unit's 128 keys (key block kb).  DUP: the tile rows r and
        // r + 64 hold the same query and two groups of four warps (warps 2..5 and 7..10) work on the same tensor-memory
        // lanes: kb = 2 (r / 64) + group.  Otherwise 128 distinct rows and four groups (warps 2..5, 7..10, 11..14,
        // 15..18): kb = group.  A thread also owns a share of the row's accumulator columns (for the rare rescale and
        // for carrying the result home): columns [32 cb, 32 cb + 32), cb = its index among the threads of its lane.
        constexpr int HC = 32;                                 // keys of a unit per thread: a quarter of the unit's 128
        static_assert(BN / 4 == HC, "a thread takes 32 keys of a unit");
        constexpr int NG = DUP ? 2 : 4;                        // warp groups
        const int grp = warp < 7 ? 0 : 1 + (warp - 7) / 4;
        const int quad = warp & 3;
        const int r = quad * 32 + lane;                        // tensor-memory lane
        const int kb = DUP ? 2 * (r >> 6) + grp : grp;         // key block
        const int row = DUP ? (r & 63) : row0 + r;             // query row
        const int prow_i = DUP ? (r & 63) : r;                 // row of the P tile this thread writes (DUP: and that row + 64)
        // accumulator columns: DUP - each row copy holds all DH columns, the copy takes a half and the group half of that
        // (d_head 64: the first group all 32 of the half); otherwise the four groups take DH / 4 each (d_head 64: two groups 32 each)
        constexpr int CBN = DH / 32;                           // 32-column blocks of a row
        const int cb = DUP ? (r >> 6) * (CBN / 2) + (CBN >= 4 ? grp : 0) : grp;
        const bool carries = DUP ? (CBN >= 4 || grp == 0) : grp < CBN;
        const bool live = row < p.n;
        const bool warp_live = DUP ? (quad & 1) * 32 < p.n : row0 + quad * 32 < p.n;   // warps whose 32 rows are all padding skip the math
        const uint32_t lane_off = (uint32_t)(quad * 32) << 16;
        const float sl2 = p.scale * 1.4426950408889634f;       // scores are kept in the log2 domain: s * scale * log2(e)
        pdl_wait();                                            // the mask comes from an earlier kernel
        // this row's mask words stay in registers; their OR over the CTA's rows tells every role
        // which node groups exist for this CTA
        constexpr int MW = DUP ? 1 : MAX_UNITS_WORDS;          // up to 64 nodes: one mask word (a word that does not exist reads as 0)
        unsigned long long myw[MW];
#pragma unroll
        for (int w = 0; w < MW; ++w) {
            myw[w] = (live && w < p.n_words) ? p.mask[(size_t)row * p.n_words + w] : 0ull;
            if (myw[w] && kb == 0) atomicOr(&sm->word_or[w], myw[w]);
        }
        mbar_arrive(smem_u32(&sm->mask_ready));
        {
            // ---- the output accumulator [128 x DH] stays in tensor memory over all units.  The
            // probabilities are taken against a reference maximum m that is raised only when a unit's maximum
            // exceeds it by more than 2^8 (the probabilities then stay below 256, exact enough in half and far
            // from overflow in the float sums); raising it rescales the row's accumulator in place, which is
            // rare after the first unit.  Any reference gives the same o / l, so the result is unchanged.
            constexpr float RAISE = 8.f;
            float m = -INFINITY, l = 0.f;                      // l: sum over this thread's keys only
            if (!warp_live) {                                  // padding rows contribute zero rows of P, written once
#pragma unroll
                for (int bb = 0; bb < P_BUFS * KSL; ++bb)
#pragma unroll
                    for (int ch = 0; ch < 8; ++ch) *reinterpret_cast<uint4*>(p_ptr + bb * (QM * 128) + r * 128 + (ch << 4)) = make_uint4(0, 0, 0, 0);
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            }
            const int cnt = walk([&](int i, int key0, int g) -> bool {
                const int b = i & 1, pb = i % P_BUFS;
                uint32_t vis = 0u;                             // visibility of this thread's 32 keys of the unit
                if (g < 0) {
                    const int valid = kv_len - key0 - kb * HC;
                    if (live) vis = valid >= HC ? 0xffffffffu : (valid > 0 ? ((1u << valid) - 1u) : 0u);
                } else {
                    const int word = g * KSL + (kb >> 1);      // this thread's 32 nodes of the group: half of a mask word
#pragma unroll
                    for (int a = 0; a < MW; ++a) if (a == word) vis = (uint32_t)(myw[a] >> ((kb & 1) * HC));
                }
                mbar_wait(smem_u32(&sm->s_full[b]), (i >> 1) & 1, abort_flag, p.status, DEV_TIMEOUT_EPI);
                if (!warp_live) {
                    mbar_arrive(smem_u32(&sm->s_empty[b]));
                    pair_bar<NT>();                                // every softmax thread takes part in the exchange barriers
                    pair_bar<NT>();
                    if (i >= P_BUFS) mbar_wait(smem_u32(&sm->p_empty[pb]), ((i / P_BUFS) - 1) & 1, abort_flag, p.status, DEV_TIMEOUT_EPI);
                    mbar_arrive(smem_u32(&sm->p_full[pb]));
                    return true;
                }
                tc_fence_after();
                float s[HC];
                tc_ld32(tmem_base + TMEM_S + b * BN + kb * HC + lane_off, s);
                tc_fence_before();
                mbar_arrive(smem_u32(&sm->s_empty[b]));
                if (vis != 0xffffffffu) {
#pragma unroll
                    for (int j = 0; j < HC; ++j) s[j] = ((vis >> j) & 1u) ? s[j] : -INFINITY;
                }
                float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
                for (int j = 0; j < HC; j += 4) {
                    mx[0] = fmaxf(mx[0], s[j]); mx[1] = fmaxf(mx[1], s[j + 1]);
                    mx[2] = fmaxf(mx[2], s[j + 2]); mx[3] = fmaxf(mx[3], s[j + 3]);
                }
                float tmax = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
                // the three partner threads hold the other 96 keys of the row
                if constexpr (DUP) {
                    sm->xch[grp][r] = tmax;
                    pair_bar<NT>();
                    tmax = fmaxf(fmaxf(tmax, sm->xch[grp ^ 1][r]), fmaxf(sm->xch[grp][r ^ 64], sm->xch[grp ^ 1][r ^ 64])) * sl2;
                } else {
                    // Four groups: the maxima travel as bfloat16 (the exchange block holds 1 KB).  Every thread, the owner
                    // included, uses the ROUNDED values, so all four agree; the reference maximum only has to be common to
                    // the row and close to the true one (a rounding of 2^-8 relative moves the probabilities by a factor
                    // near 1, far from the 2^8 head-room).
                    uint16_t* x16 = reinterpret_cast<uint16_t*>(&sm->xch[0][0]);
                    x16[grp * QM + r] = (uint16_t)(__float_as_uint(tmax) >> 16);       // truncation: never above the true value...
                    pair_bar<NT>();
                    float t4 = -INFINITY;
#pragma unroll
                    for (int a = 0; a < NG; ++a) t4 = fmaxf(t4, __uint_as_float((uint32_t)x16[a * QM + r] << 16));
                    // ... for positive values; a negative one is truncated towards zero, i.e. upwards: both are within 2^-7 relative
                    tmax = t4 * sl2;
                }
                pair_bar<NT>();                                    // everybody has read: the slots may be written again
                const bool raise = tmax > m + RAISE || (m == -INFINITY && tmax != -INFINITY);
                if (__any_sync(0xffffffffu, raise)) {
                    const float f = raise ? ex2_approx(m - tmax) : 1.f;      // m = -inf gives 0
                    if (i > 0) {
                        // The accumulator holds the products of units 0 .. i-1 once the last of them has completed, which
                        // is also what frees that unit's P buffer.  (A parity wait only tells "the phase after the one
                        // I saw last is over", so it must be a barrier whose phases this thread sees one by one: the P
                        // buffers' are, each is waited for two units later anyway; a barrier that completes once per
                        // unit and is looked at only now and then is not.)
                        mbar_wait(smem_u32(&sm->p_empty[(i - 1) % P_BUFS]), ((i - 1) / P_BUFS) & 1, abort_flag, p.status, DEV_TIMEOUT_EPI);
                        tc_fence_after();
                        if (carries) {                         // this thread's own block of the row's columns
                            float v[32];
                            tc_ld32(tmem_base + TMEM_PV + cb * 32 + lane_off, v);
#pragma unroll
                            for (int j = 0; j < 32; ++j) v[j] *= f;
                            tc_st32(tmem_base + TMEM_PV + cb * 32 + lane_off, v);
                        }
                        tc_fence_before();
                    }
                    if (raise) { l *= f; m = tmax; }
                }
                const float neg = (m == -INFINITY) ? 0.f : -m;
                if (i >= P_BUFS) mbar_wait(smem_u32(&sm->p_empty[pb]), ((i / P_BUFS) - 1) & 1, abort_flag, p.status, DEV_TIMEOUT_EPI);
                // this thread's 32 probabilities are half of a 128-byte row of key slab `half`; they go into both
                // copies of the row (tile rows row and row + 64)
                uint8_t* prow = p_ptr + pb * P_BYTES + (kb >> 1) * (QM * 128) + prow_i * 128;
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
                    const uint32_t off = (uint32_t)((((kb & 1) * 4 + q) ^ (prow_i & 7)) << 4);
                    const uint4 val = make_uint4(packed[0], packed[1], packed[2], packed[3]);
                    *reinterpret_cast<uint4*>(prow + off) = val;
                    if constexpr (DUP) *reinterpret_cast<uint4*>(prow + 64 * 128 + off) = val;
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                mbar_arrive(smem_u32(&sm->p_full[pb]));
                l += (ps[0] + ps[1]) + (ps[2] + ps[3]);
                return true;
            });
            float o[32];
#pragma unroll
            for (int c = 0; c < 32; ++c) o[c] = 0.f;
            if (cnt > 0) {
                // the last product is complete when its P buffer has been released (see the rescale above)
                mbar_wait(smem_u32(&sm->p_empty[(cnt - 1) % P_BUFS]), ((cnt - 1) / P_BUFS) & 1, abort_flag, p.status, DEV_TIMEOUT_EPI);
                if (warp_live && carries) {
                    tc_fence_after();
                    tc_ld32(tmem_base + TMEM_PV + cb * 32 + lane_off, o);
                    tc_fence_before();
                }
            }
            // the four partial sums of a row meet in the P buffers, which nobody reads any more
            float* lx = reinterpret_cast<float*>(p_ptr);
            lx[kb * QM + prow_i] = l;
            pair_bar<NT>();
            l = (lx[prow_i] + lx[QM + prow_i]) + (lx[2 * QM + prow_i] + lx[3 * QM + prow_i]);
            leave_partial<DH, 32>(p, split, h, row, cb * 32, live && carries, kb == 0, o, m, l);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

template <int DH>
__global__ void __launch_bounds__(THREADS_DUP, 1) k_attn_small(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                                                               const __grid_constant__ CUtensorMap tm_v, const AttnParams p) {
    attn_body<DH, true>(tm_q, tm_k, tm_v, p);
}

// The same kernel for trees of more than 64 nodes: 128 distinct query rows per CTA, four groups of softmax warps.
template <int DH>
__global__ void __launch_bounds__(THREADS_WIDE, 1) k_attn_wide(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                                                               const __grid_constant__ CUtensorMap tm_v, const AttnParams p) {
    attn_body<DH, false>(tm_q, tm_k, tm_v, p);
}

}  // namespace

// Launches the split kernel only (partials to att_o / att_ml); -> number of splits written, or 0 after an error.
int launch_attn_tc_small(ghd_ctx* c, const void* q, const ghd_kv_layer* kv, const ghd_tree* t, bool coo, ghd_status* st) {
    const ghd_model_cfg& m = c->cfg;
    const int n = t->n, H = m.n_heads, dh = m.d_head, d = m.d_model;
    constexpr int BN = 128;                              // keys per unit
    const int kt = t->kv_len < 0 ? m.max_kv_len : t->kv_len + n;      // rows the K/V maps cover (see launch_attn_tc)
    *st = GHD_OK;
    CUtensorMap tm_q, tm_k, tm_v;
    const bool dup = n <= 64;                            // duplicated rows (two warp groups) or 128 distinct rows (four)
    const int mtiles = (n + QM - 1) / QM;
    if (!tmap_rows_x_k(c, q, (uint64_t)n, (uint64_t)d, dup ? 64 : QM, &tm_q) ||
        !tmap_planes_slabs(c, kv->k, (uint64_t)H, (uint64_t)m.max_kv_len, (uint64_t)kt, (uint64_t)dh, (uint32_t)BN, &tm_k) ||
        !tmap_planes_slabs(c, kv->v, (uint64_t)H, (uint64_t)m.max_kv_len, (uint64_t)kt, (uint64_t)dh, (uint32_t)BN, &tm_v)) {
        snprintf(c->err, sizeof(c->err), "tcgen05 attention: tensor map encoding failed");
        *st = GHD_ECUDA;
        return 0;
    }
    const int units = (kv_len_host_of(c, t) + BN - 1) / BN + (coo ? 0 : (n + BN - 1) / BN);
    int splits = c->opt_attn_splits;
    if (splits <= 0) {
        splits = c->sm_count / (H * mtiles);             // one CTA per SM
        const int by_len = units;                        // at least one unit per split
        if (splits > by_len) splits = by_len;
    }
    if (splits > c->max_splits - (coo ? 1 : 0)) splits = c->max_splits - (coo ? 1 : 0);
    if (splits < 1) splits = 1;
    AttnParams p{};
    p.n = n; p.heads = H; p.kv_len = t->kv_len; p.kv_len_dev = kv_len_dev_of(c, t); p.max_kv_len = m.max_kv_len;
    p.max_nodes = m.max_nodes; p.splits = splits; p.n_words = t->n_words; p.cache_only = coo ? 1 : 0;
    p.mask = t->mask; p.status = c->status; p.part_o = c->att_o; p.part_ml = c->att_ml;
    p.scale = 1.0f / sqrtf((float)dh);
    dim3 grid(splits, H, mtiles);
    if (!c->attr_attn_small) {       // per context: the attribute belongs to the device the context was created on
        if (cudaFuncSetAttribute(k_attn_small<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Shape<64>::SMEM_BYTES) != cudaSuccess ||
            cudaFuncSetAttribute(k_attn_small<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Shape<128>::SMEM_BYTES) != cudaSuccess ||
            cudaFuncSetAttribute(k_attn_wide<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Shape<64>::SMEM_BYTES) != cudaSuccess ||
            cudaFuncSetAttribute(k_attn_wide<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Shape<128>::SMEM_BYTES) != cudaSuccess) {
            snprintf(c->err, sizeof(c->err), "tcgen05 attention: cannot raise dynamic shared memory");
            cudaGetLastError();
            *st = GHD_ECUDA;
            return 0;
        }
        c->attr_attn_small = true;
    }
    if (dup) {
        if (dh == 64) launch_k(c, true, k_attn_small<64>, grid, THREADS_DUP, Shape<64>::SMEM_BYTES, tm_q, tm_k, tm_v, p);
        else launch_k(c, true, k_attn_small<128>, grid, THREADS_DUP, Shape<128>::SMEM_BYTES, tm_q, tm_k, tm_v, p);
    } else {
        if (dh == 64) launch_k(c, true, k_attn_wide<64>, grid, THREADS_WIDE, Shape<64>::SMEM_BYTES, tm_q, tm_k, tm_v, p);
        else launch_k(c, true, k_attn_wide<128>, grid, THREADS_WIDE, Shape<128>::SMEM_BYTES, tm_q, tm_k, tm_v, p);
    }
    return splits;
}

}  // namespace ghd
