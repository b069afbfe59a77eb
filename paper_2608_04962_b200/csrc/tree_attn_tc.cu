// Tree-verification attention on the 5th-generation tensor cores (tcgen05 + TMEM), one layer.
//
// Decomposition: for one (sequence, KV head) the N*G query rows form the M dimension; a work unit
// is up to 128 of them (whole nodes) times one chunk of the cache (split-KV), streamed as 64-token
// K/V tiles.  The kernel is persistent: one CTA per SM takes work units from a global counter, in an
// order prepared on the device (longest chunks first), and its pipeline runs across unit boundaries.
// Warp roles (320 threads):
//   warp 0     scheduler + TMA producer: fetches the next unit, publishes its descriptor in a
//              two-slot ring, loads the Q block (3-D box over [node, head, D]) and the K and V tiles
//              (3-D boxes over [token, kv head, D], 128-byte swizzle, six stages)
//   warp 1     allocates TMEM, issues  S = Q K^T  (M=128, N=64, operands from shared memory) and
//              O += P V  (M=128, N=D, A = P from TMEM, B = V tile read MN-major from shared memory);
//              S runs four tiles ahead of P V
//   warps 2-5  softmax group 0: even tiles      } thread = query row = TMEM lane, so row max and
//   warps 6-9  softmax group 1: odd tiles       } row sum need no shuffles
// The two softmax groups are independent: each keeps its own running (reference max, sum) per row
// and its own output accumulator in TMEM, exactly like two KV splits, and they are merged at the
// end of the unit.  Each group has two S buffers, so its next S tile is ready when it finishes
// the current one.  P overwrites the first half of its S buffer in place (packed bf16).  An output
// accumulator is rescaled only when a row's maximum grows by more than 2^8 (rare), by the thread
// that owns the row.  Chunks of a split sequence leave fp32 partials in the workspace; the CTA that
// finishes a sequence's last chunk (atomic ticket, nobody waits) merges them.
// TMEM columns: O0 [0,128)  O1 [128,256)  S/P of group g, buffer h: [256 + 128 g + 64 h, +64).
#include <math.h>

#include "tc05.cuh"
#include "tree_attn.cuh"

namespace specroll {

namespace attc {
constexpr int BN = 64;        // KV tokens per tile
constexpr int AHEAD = 4;      // S tiles in flight ahead of P V (two per softmax group)
constexpr int THREADS = 320;
constexpr int STAGES = 6;
constexpr int TMEM_COLS = 512;
constexpr uint32_t O_COL = 0, S_COL = 256;  // O_COL + 128*group ; S_COL + 128*group + 64*buffer
constexpr float RESCALE_LOG2 = 8.0f;
constexpr int Q_BOX_BYTES = 128 * 128;  // 128 query rows x 128 bytes (64 bf16)
constexpr int KV_BOX_BYTES = BN * 128;  // 64 tokens x 128 bytes
constexpr int N_BARS = 3 * STAGES + 21;

struct UnitDesc {
    int32_t valid, b, hkv, rb, n_splits, kv0, L, t_lo, n_it, has_tree, item, item0;
};

template <int D>
struct Cfg {
    static constexpr int NBOX = D / 64;
    static constexpr int Q_BYTES = NBOX * Q_BOX_BYTES;
    static constexpr int KV_BYTES = NBOX * KV_BOX_BYTES;  // one K tile or one V tile
    static constexpr int STAGE_BYTES = 2 * KV_BYTES;
    static constexpr int BAR_BYTES = (8 * N_BARS + 15) / 16 * 16;
    static constexpr int EXTRA = BAR_BYTES + 16 + 128 * 8 + 2 * 64;  // barriers, slot/abort/ticket, merge, ring
    static constexpr int USED = Q_BYTES + STAGES * STAGE_BYTES + 1024 + EXTRA;
    // at least ~118 KB so that two CTAs can never share an SM (each allocates all of TMEM)
    static constexpr int SMEM = USED > 120832 ? USED : 120832;
    static_assert(sizeof(UnitDesc) <= 64, "ring slot");
    static_assert(USED <= 232448, "shared memory budget");
};

// Group rendezvous on an mbarrier (count = number of participants) with the same bounded wait as every
// other wait here: a hardware named barrier would hang if a participant had left through the abort path.
__device__ __forceinline__ bool group_sync(uint32_t bar, uint32_t &uses, volatile int *abort_flag) {
    mbar_arrive(bar);
    const bool ok = mbar_wait(bar, uses & 1u, abort_flag);
    ++uses;
    return ok;
}
}  // namespace attc

template <int D>
__global__ void __launch_bounds__(attc::THREADS, 1)
tree_attn_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                    const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmKt,
                    const __grid_constant__ CUtensorMap tmVt, AttnArgs a, TopoMask mask,
                    int32_t *__restrict__ status) {
    using namespace attc;
    using C = Cfg<D>;
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    unsigned char *aligned = smem_raw + (base - raw);
    const uint32_t q_s = base;
    const uint32_t kv_s = base + C::Q_BYTES;
    const uint32_t bar0 = kv_s + STAGES * C::STAGE_BYTES;
    auto k_full = [&](int s) { return bar0 + 8u * s; };
    auto v_full = [&](int s) { return bar0 + 8u * (STAGES + s); };
    auto kv_empty = [&](int s) { return bar0 + 8u * (2 * STAGES + s); };
    constexpr int B1 = 3 * STAGES;
    auto s_full = [&](int g, int h) { return bar0 + 8u * (B1 + 2 * g + h); };
    // one P barrier per S buffer: a group may finish two tiles before the MMA thread looks, and a
    // single barrier would then have flipped twice and hide the first completion
    auto p_ready = [&](int g, int h) { return bar0 + 8u * (B1 + 4 + 2 * g + h); };
    // likewise one "P V done" barrier per S buffer: two P V of a group can be pending at once, and on a
    // single barrier the completion of the older one would pass for the completion of the newer one
    auto pv_done = [&](int g, int h) { return bar0 + 8u * (B1 + 8 + 2 * g + h); };
    const uint32_t q_full = bar0 + 8u * (B1 + 12), q_free = bar0 + 8u * (B1 + 13);
    auto unit_full = [&](int s) { return bar0 + 8u * (B1 + 14 + s); };
    auto unit_empty = [&](int s) { return bar0 + 8u * (B1 + 16 + s); };
    const uint32_t sync_a = bar0 + 8u * (B1 + 18), sync_b = bar0 + 8u * (B1 + 19), sync_g0 = bar0 + 8u * (B1 + 20);
    unsigned char *extra = aligned + C::Q_BYTES + STAGES * C::STAGE_BYTES + C::BAR_BYTES;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(extra);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(extra + 4);
    volatile int *ticket = reinterpret_cast<volatile int *>(extra + 8);
    float2 *merge_ml = reinterpret_cast<float2 *>(extra + 16);  // group 1's (max, sum) per row
    volatile UnitDesc *ring = reinterpret_cast<volatile UnitDesc *>(extra + 16 + 128 * 8);  // 2 slots of 64 bytes

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int N = a.N, G = a.G;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(k_full(s), 1);
            mbar_init(v_full(s), 1);
            mbar_init(kv_empty(s), 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(s_full(i, 0), 1);
            mbar_init(s_full(i, 1), 1);
            mbar_init(p_ready(i, 0), 128);
            mbar_init(p_ready(i, 1), 128);
            mbar_init(pv_done(i, 0), 1);
            mbar_init(pv_done(i, 1), 1);
            mbar_init(unit_full(i), 1);
            mbar_init(unit_empty(i), 257);  // the MMA thread and the 256 softmax threads
        }
        mbar_init(q_full, 1);
        mbar_init(q_free, 1);
        mbar_init(sync_a, 256);
        mbar_init(sync_b, 256);
        mbar_init(sync_g0, 128);
        *abort_flag = 0;
        fence_mbar_init();
        prefetch_tmap(&tmQ);
        prefetch_tmap(&tmK);
        prefetch_tmap(&tmV);
        prefetch_tmap(&tmKt);
        prefetch_tmap(&tmVt);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), TMEM_COLS);
        tmem_relinquish();
    }
    // The Q block's TMA box covers rows_per_block rows; the rest of the 128-row operand stays zero.
    for (int c = threadIdx.x; c < C::Q_BYTES / 16; c += THREADS)
        reinterpret_cast<uint4 *>(aligned)[c] = make_uint4(0u, 0u, 0u, 0u);
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------------ scheduler + TMA producer
        if (lane == 0) {
            int issued[STAGES];
#pragma unroll
            for (int s = 0; s < STAGES; ++s) issued[s] = -1;
            bool ok = true, q_inflight = false;
            uint32_t gt = 0;  // K/V tiles loaded so far (all units)
            for (uint32_t u = 0; ok; ++u) {
                const int slot = (int)(u & 1u);
                if (!mbar_wait(unit_empty(slot), ((u >> 1) & 1u) ^ 1u, abort_flag)) {
                    ok = false;
                    break;
                }
                const int w = atomicAdd(a.work_counter, 1);
                volatile UnitDesc *d = ring + slot;
                if (w >= a.total_work) {
                    d->valid = 0;
                    mbar_arrive(unit_full(slot));
                    break;
                }
                // ---- decode: w = (position in work order * Hkv + hkv) * n_rb + rb
                int t = w;
                const int rb = t % a.n_rb;
                t /= a.n_rb;
                const int hkv = t % a.Hkv;
                const int si = t / a.Hkv;
                int lo = 0, hi = a.B;  // largest rank r with sorted_start[r] <= si
                while (hi - lo > 1) {
                    const int mid = (lo + hi) >> 1;
                    if (a.sorted_start[mid] <= si) lo = mid; else hi = mid;
                }
                const int b = a.seq_at_rank[lo];
                const int split = si - a.sorted_start[lo];
                const int n_splits = a.sorted_start[lo + 1] - a.sorted_start[lo];
                const int kv0 = a.kv_indptr[b];
                const int L = a.kv_indptr[b + 1] - kv0;
                const int tiles_b = (L + BN - 1) / BN;
                const int tps = (tiles_b + n_splits - 1) / n_splits;
                const int t_lo = min(tiles_b, split * tps), t_hi = min(tiles_b, t_lo + tps);
                const int has_tree = (split == n_splits - 1) ? 1 : 0;
                const int n_it = (t_hi - t_lo) + has_tree;
                const int item0 = a.item_start[b];
                d->valid = 1;
                d->b = b;
                d->hkv = hkv;
                d->rb = rb;
                d->n_splits = n_splits;
                d->kv0 = kv0;
                d->L = L;
                d->t_lo = t_lo;
                d->n_it = n_it;
                d->has_tree = has_tree;
                d->item = item0 + split;
                d->item0 = item0;
                mbar_arrive(unit_full(slot));  // release: the descriptor is visible to whoever acquires
                // ---- Q block of this unit, once every S of the previous unit has been computed
                if (u > 0 && !mbar_wait(q_free, (u - 1u) & 1u, abort_flag)) {
                    ok = false;
                    break;
                }
                mbar_arrive_expect_tx(q_full, (uint32_t)(C::NBOX * 128 * a.rows_per_block));
#pragma unroll
                for (int bx = 0; bx < C::NBOX; ++bx)
                    tma_load_3d(q_s + bx * Q_BOX_BYTES, &tmQ, bx * 64, hkv * G, b * N + rb * a.nodes_per_block, q_full);
                q_inflight = true;
                // ---- K/V tiles
                for (int it = 0; it < n_it; ++it, ++gt) {
                    const int s = (int)(gt % STAGES);
                    const uint32_t ph = (gt / STAGES) & 1u;
                    if (!mbar_wait(kv_empty(s), ph ^ 1u, abort_flag)) {
                        ok = false;
                        break;
                    }
                    const bool tree = has_tree && (it == n_it - 1);
                    const int tok = tree ? b * N : kv0 + (t_lo + it) * BN;
                    const CUtensorMap *mk = tree ? &tmKt : &tmK;
                    const CUtensorMap *mv = tree ? &tmVt : &tmV;
                    const uint32_t ks = kv_s + s * C::STAGE_BYTES, vs = ks + C::KV_BYTES;
                    mbar_arrive_expect_tx(k_full(s), C::KV_BYTES);
#pragma unroll
                    for (int bx = 0; bx < C::NBOX; ++bx)
                        tma_load_3d(ks + bx * KV_BOX_BYTES, mk, bx * 64, hkv, tok, k_full(s));
                    mbar_arrive_expect_tx(v_full(s), C::KV_BYTES);
#pragma unroll
                    for (int bx = 0; bx < C::NBOX; ++bx)
                        tma_load_3d(vs + bx * KV_BOX_BYTES, mv, bx * 64, hkv, tok, v_full(s));
                    issued[s] = (int)ph;
                }
                if (ok) q_inflight = false;  // the MMA thread has consumed q_full before its first S
            }
            if (!ok) {
                // aborting: give the copies already in flight time to land before the CTA goes away
                const unsigned long long t0 = globaltimer_ns();
                bool pending = true;
                while (pending && globaltimer_ns() - t0 < 100000000ull) {
                    pending = false;
#pragma unroll
                    for (int s = 0; s < STAGES; ++s)
                        if (issued[s] >= 0 && !(mbar_try_wait(k_full(s), (uint32_t)issued[s]) &&
                                                mbar_try_wait(v_full(s), (uint32_t)issued[s])))
                            pending = true;
                }
                if (q_inflight) {
                    const unsigned long long t1 = globaltimer_ns();
                    while (!mbar_try_wait(q_full, 0u) && !mbar_try_wait(q_full, 1u) && globaltimer_ns() - t1 < 100000000ull) {
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        // tcgen05.mma operations of one thread execute in issue order, which is what lets an S tile
        // overwrite the buffer whose P the previously issued P V has read.
        if (lane == 0) {
            constexpr uint32_t idesc_s = idesc_bf16(128, BN, false, false);
            constexpr uint32_t idesc_pv = idesc_bf16(128, D, false, true);  // V is read MN-major
            uint32_t gt = 0;            // K/V tiles consumed so far (all units)
            uint32_t cnt[2] = {0u, 0u};  // tiles handed to each softmax group so far
            bool ok = true;
            for (uint32_t u = 0; ok; ++u) {
                const int slot = (int)(u & 1u);
                if (!mbar_wait(unit_full(slot), (u >> 1) & 1u, abort_flag)) break;
                const int valid = ring[slot].valid, n_it = ring[slot].n_it;
                mbar_arrive(unit_empty(slot));
                if (!valid) break;
                if (!mbar_wait(q_full, u & 1u, abort_flag)) break;
                tc_fence_after();
                if (n_it == 0) {
                    umma_commit(q_free);
                    continue;
                }
                // S of tile j -> buffer (group j&1, parity of that group's tile count); waits for the K tile
                auto issue_s = [&](int j) -> bool {
                    const uint32_t gj = gt + (uint32_t)j;
                    const int s = (int)(gj % STAGES);
                    if (!mbar_wait(k_full(s), (gj / STAGES) & 1u, abort_flag)) return false;
                    tc_fence_after();
                    const int g = j & 1;
                    const uint32_t c = cnt[g] + (uint32_t)(j >> 1);
                    const int h = (int)(c & 1u);
                    const uint32_t ks = kv_s + s * C::STAGE_BYTES;
                    const uint32_t d_t = tmem_base + S_COL + 128u * (uint32_t)g + 64u * (uint32_t)h;
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk) {
                        const uint32_t qoff = (uint32_t)(kk >> 2) * Q_BOX_BYTES + (uint32_t)(kk & 3) * 32u;
                        const uint32_t koff = (uint32_t)(kk >> 2) * KV_BOX_BYTES + (uint32_t)(kk & 3) * 32u;
                        umma_ss(d_t, smem_desc_sw128(q_s + qoff, 1024, 0), smem_desc_sw128(ks + koff, 1024, 0), idesc_s,
                                kk > 0 ? 1u : 0u);
                    }
                    umma_commit(s_full(g, h));
                    if (j == n_it - 1) umma_commit(q_free);  // last S of the unit: Q may be replaced after it
                    return true;
                };
                for (int j = 0; j < AHEAD && j < n_it && ok; ++j) ok = issue_s(j);
                for (int j = 0; j < n_it && ok; ++j) {
                    const int g = j & 1;
                    const uint32_t c = cnt[g] + (uint32_t)(j >> 1);
                    if (!mbar_wait(p_ready(g, (int)(c & 1u)), (c >> 1) & 1u, abort_flag)) {
                        ok = false;
                        break;
                    }
                    const uint32_t gj = gt + (uint32_t)j;
                    const int s = (int)(gj % STAGES);
                    if (!mbar_wait(v_full(s), (gj / STAGES) & 1u, abort_flag)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t vs = kv_s + s * C::STAGE_BYTES + C::KV_BYTES;
                    const uint32_t p_t = tmem_base + S_COL + 128u * (uint32_t)g + 64u * (c & 1u);
                    const uint32_t o_t = tmem_base + O_COL + 128u * (uint32_t)g;
#pragma unroll
                    for (int kk = 0; kk < BN / 16; ++kk) {
                        // 16 tokens per step: 2048 bytes down the V tile, 8 packed columns along P
                        umma_ts(o_t, p_t + 8u * kk, smem_desc_sw128(vs + kk * 2048, 1024, KV_BOX_BYTES), idesc_pv,
                                (j > 1 || kk > 0) ? 1u : 0u);
                    }
                    umma_commit(kv_empty(s));
                    umma_commit(pv_done(g, (int)(c & 1u)));
                    if (j + AHEAD < n_it) ok = issue_s(j + AHEAD);  // reuses the buffer this P V has just read
                }
                gt += (uint32_t)n_it;
                cnt[0] += (uint32_t)((n_it + 1) >> 1);
                cnt[1] += (uint32_t)(n_it >> 1);
            }
        }
    } else {
        // ------------------------------------------------------------------ softmax groups (warps 2..9)
        const int grp = (warp - 2) >> 2;  // 0: even tiles, 1: odd tiles
        const int lg = warp & 3;          // TMEM lane group of this warp
        const int row = lg * 32 + lane;
        const uint32_t t_lane = tmem_base + ((uint32_t)(lg * 32) << 16);
        const uint32_t o_t = t_lane + O_COL + 128u * (uint32_t)grp;
        const float sc = a.scale_log2;
        uint32_t cnt = 0;  // tiles this group has processed so far (all units)
        uint32_t use_a = 0, use_b = 0, use_g0 = 0;
        bool ok = true;
        for (uint32_t u = 0; ok; ++u) {
            const int slot = (int)(u & 1u);
            ok = mbar_wait(unit_full(slot), (u >> 1) & 1u, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            const int valid = ring[slot].valid, b = ring[slot].b, hkv = ring[slot].hkv, rb = ring[slot].rb;
            const int n_splits = ring[slot].n_splits, L = ring[slot].L, t_lo = ring[slot].t_lo;
            const int n_it = ring[slot].n_it, has_tree = ring[slot].has_tree, item = ring[slot].item;
            const int item0 = ring[slot].item0;
            mbar_arrive(unit_empty(slot));
            if (!valid) break;
            const int gr = rb * a.rows_per_block + row;
            const bool row_ok = row < a.rows_per_block && gr < a.rows;
            const uint64_t anc = row_ok ? mask.anc[gr / G] : 0ull;
            float m_used = -INFINITY, l = 0.f;
            int n_mine = 0;
            for (int j = grp; j < n_it; j += 2, ++n_mine) {
                const uint32_t c_idx = cnt + (uint32_t)n_mine;
                const int h = (int)(c_idx & 1u);
                ok = mbar_wait(s_full(grp, h), (c_idx >> 1) & 1u, abort_flag);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
                const uint32_t s_t = t_lane + S_COL + 128u * (uint32_t)grp + 64u * (uint32_t)h;
                const bool tree = has_tree && (j == n_it - 1);
                const int limit = tree ? BN : (L - (t_lo + j) * BN);  // columns >= limit are outside the sequence
                const bool full = !tree && limit >= BN;
                uint32_t r0[32], r1[32];
                tmem_ld32(s_t, r0);
                tmem_ld32(s_t + 32u, r1);
                tmem_ld_wait();
                uint32_t bits0, bits1;  // admissible columns 0..31 and 32..63
                if (full) {
                    bits0 = bits1 = 0xffffffffu;
                } else if (tree) {
                    bits0 = (uint32_t)anc;
                    bits1 = (uint32_t)(anc >> 32);
                } else {
                    bits0 = limit >= 32 ? 0xffffffffu : ((1u << limit) - 1u);
                    bits1 = limit >= 64 ? 0xffffffffu : (limit <= 32 ? 0u : ((1u << (limit - 32)) - 1u));
                }
                float mx0 = -INFINITY, mx1 = -INFINITY;
                if (full) {
#pragma unroll
                    for (int i2 = 0; i2 < 32; ++i2) {
                        mx0 = fmaxf(mx0, __uint_as_float(r0[i2]));
                        mx1 = fmaxf(mx1, __uint_as_float(r1[i2]));
                    }
                } else {
#pragma unroll
                    for (int i2 = 0; i2 < 32; ++i2) {
                        if ((bits0 >> i2) & 1u) mx0 = fmaxf(mx0, __uint_as_float(r0[i2]));
                        if ((bits1 >> i2) & 1u) mx1 = fmaxf(mx1, __uint_as_float(r1[i2]));
                    }
                }
                const float mt = fmaxf(mx0, mx1) * sc;  // scale > 0; -inf stays -inf
                float alpha = 1.f;
                const bool need = mt > m_used + RESCALE_LOG2;  // also true on the first admissible tile
                if (need) {
                    alpha = (m_used == -INFINITY) ? 0.f : ex2_approx(m_used - mt);
                    m_used = mt;
                    l *= alpha;
                }
                if (__any_sync(0xffffffffu, need) && n_mine > 0) {
                    // rows of this warp change their reference maximum: rescale their running outputs
                    // in TMEM.  This group's previous P V must have landed first.
                    ok = mbar_wait(pv_done(grp, (int)((c_idx - 1u) & 1u)), ((c_idx - 1u) >> 1) & 1u, abort_flag);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    tc_fence_after();
#pragma unroll 1
                    for (int c = 0; c < D; c += 32) {
                        uint32_t o[32];
                        tmem_ld32(o_t + (uint32_t)c, o);
                        tmem_ld_wait();
#pragma unroll
                        for (int i2 = 0; i2 < 32; ++i2) o[i2] = __float_as_uint(__uint_as_float(o[i2]) * alpha);
                        tmem_st32(o_t + (uint32_t)c, o);
                    }
                    tmem_st_wait();
                }
                const float mref = (m_used == -INFINITY) ? 0.f : m_used;
                // p = 2^(s*scale - m), packed bf16 pairs written over the first 32 columns of the S buffer
                float ls0 = 0.f, ls1 = 0.f;
                uint32_t pk0[16], pk1[16];
#pragma unroll
                for (int i2 = 0; i2 < 32; i2 += 2) {
                    float p0 = ex2_approx(fmaf(__uint_as_float(r0[i2]), sc, -mref));
                    float p1 = ex2_approx(fmaf(__uint_as_float(r0[i2 + 1]), sc, -mref));
                    float p2 = ex2_approx(fmaf(__uint_as_float(r1[i2]), sc, -mref));
                    float p3 = ex2_approx(fmaf(__uint_as_float(r1[i2 + 1]), sc, -mref));
                    if (!full) {
                        p0 = ((bits0 >> i2) & 1u) ? p0 : 0.f;
                        p1 = ((bits0 >> (i2 + 1)) & 1u) ? p1 : 0.f;
                        p2 = ((bits1 >> i2) & 1u) ? p2 : 0.f;
                        p3 = ((bits1 >> (i2 + 1)) & 1u) ? p3 : 0.f;
                    }
                    ls0 += p0 + p1;
                    ls1 += p2 + p3;
                    pk0[i2 >> 1] = pack_bf16x2(p0, p1);
                    pk1[i2 >> 1] = pack_bf16x2(p2, p3);
                }
                tmem_st16(s_t, pk0);
                tmem_st16(s_t + 16u, pk1);
                tmem_st_wait();
                l += ls0 + ls1;
                tc_fence_before();
                mbar_arrive(p_ready(grp, h));
            }
            // ---- wait for this group's last P V of the unit
            if (ok && n_mine > 0) {
                // (operations complete in issue order, so the last P V covers the one before it)
                const uint32_t c_last = cnt + (uint32_t)n_mine - 1u;
                ok = mbar_wait(pv_done(grp, (int)(c_last & 1u)), (c_last >> 1) & 1u, abort_flag);
                ok = __all_sync(0xffffffffu, ok);
            }
            cnt += (uint32_t)n_mine;
            if (grp == 1) merge_ml[row] = make_float2(m_used, (ok && n_mine > 0) ? l : 0.f);
            tc_fence_before();
            if (!group_sync(sync_a, use_a, abort_flag)) ok = false;
            ok = __all_sync(0xffffffffu, ok);
            tc_fence_after();
            if (grp == 0 && ok) {
                // ---- merge the two groups; write the output, or this chunk's partial
                const float2 other = merge_ml[row];
                const float m1 = other.x, l1 = other.y;
                const bool have0 = n_mine > 0 && l > 0.f, have1 = l1 > 0.f;
                const float M = fmaxf(have0 ? m_used : -INFINITY, have1 ? m1 : -INFINITY);
                const float w0 = have0 ? ex2_approx(m_used - M) : 0.f, w1 = have1 ? ex2_approx(m1 - M) : 0.f;
                const float lt = w0 * l + w1 * l1;
                const int n = row_ok ? gr / G : 0, g = row_ok ? gr % G : 0;
                const bool direct = (n_splits == 1);
                const float inv = direct ? (lt > 0.f ? 1.0f / lt : 0.f) : 1.0f;
                const float f0 = w0 * inv, f1 = w1 * inv;
                __nv_bfloat16 *dst_o = a.O + (((size_t)b * N + n) * a.Hq + hkv * G + g) * D;
                const size_t prow = ((size_t)item * a.Hkv + hkv) * a.rows_pad + (row_ok ? gr : 0);
                float *dst_p = a.part_o + prow * D;
                const bool any0 = __any_sync(0xffffffffu, have0), any1 = __any_sync(0xffffffffu, have1);
#pragma unroll 1
                for (int c = 0; c < D; c += 32) {
                    uint32_t o0[32], o1[32];
                    if (any0) tmem_ld32(t_lane + O_COL + (uint32_t)c, o0);
                    if (any1) tmem_ld32(t_lane + O_COL + 128u + (uint32_t)c, o1);
                    tmem_ld_wait();
                    float v[32];
#pragma unroll
                    for (int i2 = 0; i2 < 32; ++i2)
                        v[i2] = (have0 ? __uint_as_float(o0[i2]) * f0 : 0.f) + (have1 ? __uint_as_float(o1[i2]) * f1 : 0.f);
                    if (!row_ok) continue;
                    if (direct) {
#pragma unroll
                        for (int i2 = 0; i2 < 32; i2 += 8) {
                            uint4 q4;
                            q4.x = pack_bf16x2(v[i2], v[i2 + 1]);
                            q4.y = pack_bf16x2(v[i2 + 2], v[i2 + 3]);
                            q4.z = pack_bf16x2(v[i2 + 4], v[i2 + 5]);
                            q4.w = pack_bf16x2(v[i2 + 6], v[i2 + 7]);
                            *reinterpret_cast<uint4 *>(dst_o + c + i2) = q4;
                        }
                    } else {
#pragma unroll
                        for (int i2 = 0; i2 < 32; i2 += 4)
                            *reinterpret_cast<float4 *>(dst_p + c + i2) = make_float4(v[i2], v[i2 + 1], v[i2 + 2], v[i2 + 3]);
                    }
                }
                if (row_ok) {
                    if (direct) {
                        if (a.lse) a.lse[((size_t)b * N + n) * a.Hq + hkv * G + g] = (M + log2f(lt)) * 0.6931471805599453f;
                    } else {
                        a.part_ml[prow * 2] = M;
                        a.part_ml[prow * 2 + 1] = lt;
                    }
                }
                if (!direct) {
                    // ---- the chunk that arrives last merges all chunks of this (sequence, kv head, row block)
                    __threadfence();
                    bool ok3 = group_sync(sync_g0, use_g0, abort_flag);
                    if (row == 0) *ticket = atomicAdd(a.split_counters + ((size_t)b * a.Hkv + hkv) * a.n_rb + rb, 1);
                    ok3 = group_sync(sync_g0, use_g0, abort_flag) && ok3;
                    if (ok3 && *ticket == n_splits - 1 && row_ok) {
                        __threadfence();
                        float Mx = -INFINITY;
                        for (int s = 0; s < n_splits; ++s) {
                            const size_t pr = ((size_t)(item0 + s) * a.Hkv + hkv) * a.rows_pad + gr;
                            Mx = fmaxf(Mx, __ldcg(a.part_ml + pr * 2));
                        }
                        float lsum = 0.f;
                        for (int s = 0; s < n_splits; ++s) {
                            const size_t pr = ((size_t)(item0 + s) * a.Hkv + hkv) * a.rows_pad + gr;
                            const float ms = __ldcg(a.part_ml + pr * 2);
                            lsum += ((ms == -INFINITY) ? 0.f : ex2_approx(ms - Mx)) * __ldcg(a.part_ml + pr * 2 + 1);
                        }
                        const float invl = lsum > 0.f ? 1.0f / lsum : 0.f;
#pragma unroll 1
                        for (int c = 0; c < D; c += 32) {
                            float acc[32];
#pragma unroll
                            for (int i2 = 0; i2 < 32; ++i2) acc[i2] = 0.f;
                            for (int s = 0; s < n_splits; ++s) {
                                const size_t pr = ((size_t)(item0 + s) * a.Hkv + hkv) * a.rows_pad + gr;
                                const float ms = __ldcg(a.part_ml + pr * 2);
                                const float ws = (ms == -INFINITY) ? 0.f : ex2_approx(ms - Mx) * invl;
                                const float4 *src = reinterpret_cast<const float4 *>(a.part_o + pr * D + c);
#pragma unroll
                                for (int i2 = 0; i2 < 8; ++i2) {
                                    const float4 x = __ldcg(src + i2);
                                    acc[4 * i2] += ws * x.x;
                                    acc[4 * i2 + 1] += ws * x.y;
                                    acc[4 * i2 + 2] += ws * x.z;
                                    acc[4 * i2 + 3] += ws * x.w;
                                }
                            }
#pragma unroll
                            for (int i2 = 0; i2 < 32; i2 += 8) {
                                uint4 q4;
                                q4.x = pack_bf16x2(acc[i2], acc[i2 + 1]);
                                q4.y = pack_bf16x2(acc[i2 + 2], acc[i2 + 3]);
                                q4.z = pack_bf16x2(acc[i2 + 4], acc[i2 + 5]);
                                q4.w = pack_bf16x2(acc[i2 + 6], acc[i2 + 7]);
                                *reinterpret_cast<uint4 *>(dst_o + c + i2) = q4;
                            }
                        }
                        if (a.lse) a.lse[((size_t)b * N + n) * a.Hq + hkv * G + g] = (Mx + log2f(lsum)) * 0.6931471805599453f;
                    }
                }
            }
            // group 1 must not start the next unit's tiles (its P V overwrites O1) before group 0 has read O1
            tc_fence_before();
            if (!group_sync(sync_b, use_b, abort_flag)) ok = false;
            ok = __all_sync(0xffffffffu, ok);
            tc_fence_after();
        }
    }

    // ------------------------------------------------------------------ teardown
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag) atomicExch(status, SPECROLL_ETIMEOUT);
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

template <int D>
static int launch_tc(const AttnArgs &a, const TopoMask &mask, long long T_kv, int32_t *status, cudaStream_t st) {
    using C = attc::Cfg<D>;
    CUtensorMap tmQ, tmK, tmV, tmKt, tmVt;
    int rc;
    const uint64_t tree_rows = (uint64_t)a.B * a.N;
    // an empty cache still needs well-formed maps; they are never used for a load then
    const void *kc = T_kv > 0 ? (const void *)a.Kc : (const void *)a.Kt;
    const void *vc = T_kv > 0 ? (const void *)a.Vc : (const void *)a.Vt;
    const uint64_t cache_rows = T_kv > 0 ? (uint64_t)T_kv : tree_rows;
    if ((rc = make_tmap_3d_bf16(&tmQ, a.Q, D, a.Hq, tree_rows, (uint32_t)a.G, (uint32_t)a.nodes_per_block)) != SPECROLL_OK)
        return rc;
    if ((rc = make_tmap_3d_bf16(&tmK, kc, D, a.Hkv, cache_rows, 1, attc::BN)) != SPECROLL_OK) return rc;
    if ((rc = make_tmap_3d_bf16(&tmV, vc, D, a.Hkv, cache_rows, 1, attc::BN)) != SPECROLL_OK) return rc;
    if ((rc = make_tmap_3d_bf16(&tmKt, a.Kt, D, a.Hkv, tree_rows, 1, attc::BN)) != SPECROLL_OK) return rc;
    if ((rc = make_tmap_3d_bf16(&tmVt, a.Vt, D, a.Hkv, tree_rows, 1, attc::BN)) != SPECROLL_OK) return rc;
    static int n_sm = 0;
    if (n_sm == 0) {
        int dev = 0;
        SR_CUDA_TRY(cudaGetDevice(&dev));
        SR_CUDA_TRY(cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev));
        SR_CUDA_TRY(cudaFuncSetAttribute(tree_attn_tc_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM));
    }
    const unsigned grid = (unsigned)(a.total_work < n_sm ? a.total_work : n_sm);
    tree_attn_tc_kernel<D><<<grid, attc::THREADS, C::SMEM, st>>>(tmQ, tmK, tmV, tmKt, tmVt, a, mask, status);
    SR_LAUNCH_CHECK();
    return SPECROLL_OK;
}

int launch_attn_tc(const AttnArgs &a, const TopoMask &mask, int D, long long T_kv, int32_t *status, cudaStream_t st) {
    if (D == 128) return launch_tc<128>(a, mask, T_kv, status, st);
    return launch_tc<64>(a, mask, T_kv, status, st);
}

}  // namespace specroll
