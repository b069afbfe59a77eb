// Tree-verification attention on the 5th-generation tensor cores (tcgen05 + TMEM), one layer.
//
// Decomposition: for one (sequence, KV head) the N*G query rows form the M dimension, cut into row
// blocks of up to 128 rows (whole nodes).  A work unit is NRB row blocks (1 when all rows fit one
// block, else 2) times one chunk of the cache (split-KV), streamed as 128-token K/V tiles that all
// row blocks of the unit share.  The kernel is persistent: one CTA per SM takes work units from a
// global counter, in an order prepared on the device (longest chunks first), and its pipeline runs
// across unit boundaries.  Warp roles (64 + 256*NRB threads):
//   warp 0     scheduler + TMA producer: fetches the next unit, publishes its descriptor in a
//              two-slot ring, loads the Q blocks (3-D box over [node, head, D]) and the K and V tiles
//              (3-D boxes over [token, kv head, D], 128-byte swizzle).  K and V have separate rings:
//              K is needed early and is released as soon as its S is computed; V is needed late.
//   warp 1     allocates TMEM, issues  S = Q K^T  (M=128, N=128, operands from shared memory) and
//              O += P V  (M=128, N=D, A = P from TMEM, B = V tile read MN-major from shared memory).
//              NRB=1: three S buffers, S runs three tiles ahead.  NRB=2: one S buffer per row block;
//              the two blocks alternate on the tensor pipe, each one's softmax hiding under the
//              other's MMAs.
//   8 warps per row block: softmax with TWO threads per query row (warps w and w+4 own the same 32
//              TMEM lanes and take columns 0-63 / 64-127 of each S tile).  The pair exchanges its
//              two partial row maxima through shared memory once per tile.
// P is written back to TMEM over parts of S that its writer has already read (columns [0,32) by
// the first thread of a pair, [96,128) by the second), as packed bf16.  An output accumulator is
// rescaled only when a row's reference maximum grows by more than 2^8 (rare).  Chunks of a split
// sequence leave fp32 partials in the workspace; the CTA that finishes a sequence's last chunk
// (atomic ticket, nobody waits) merges them.
// TMEM columns: O of block b: [128 b, +128);  S/P buffer i of block b: [128 NRB + 128 (b SB + i), +128).
#include <math.h>

#include "tc05.cuh"
#include "tree_attn.cuh"

namespace specroll {

// Optional instrumentation, off in normal builds.
//   -DSPECROLL_TRACE: one thread per role adds up the SM cycles it spends in each kind of barrier wait (all CTAs).
//   -DSPECROLL_TRACE_EVENTS (with the above): CTA 0 also records (event, index, SM clock) per role; each record
//   costs a round trip to global memory, so the timeline it gives is stretched.
#ifdef SPECROLL_TRACE
__device__ unsigned long long g_trace[4][8192];
__device__ unsigned int g_trace_n[4];
__device__ unsigned long long g_prof[5][12];
__device__ unsigned long long g_cta_ns[8][2][160];  // per launch (mod 8): start and end of each CTA (global timer)
__device__ unsigned int g_launch_n;
#endif
#if defined(SPECROLL_TRACE) && defined(SPECROLL_TRACE_EVENTS)
#define SR_TRACE(role, ev, idx)                                                                       \
    do {                                                                                              \
        if (blockIdx.x == 0) {                                                                        \
            const unsigned n_ = g_trace_n[role]++;                                                    \
            if (n_ < 4096) {                                                                          \
                g_trace[role][2 * n_] = ((unsigned long long)(ev) << 32) | (unsigned)(idx);           \
                g_trace[role][2 * n_ + 1] = (unsigned long long)clock64();                            \
            }                                                                                         \
        }                                                                                             \
    } while (0)
#else
#define SR_TRACE(role, ev, idx)
#endif

namespace attc {
constexpr int BN = 128;  // KV tokens per tile
constexpr int TMEM_COLS = 512;
constexpr float RESCALE_LOG2 = 8.0f;
constexpr int BOX_BYTES = BN * 128;  // 128 rows x 128 bytes (64 bf16)

struct UnitDesc {
    int32_t valid, b, hkv, rb, n_splits, kv0, L, t_lo, n_it, has_tree, item, item0;
};

template <int D, int NRB>
struct Cfg {
    static constexpr int NBOX = D / 64;
    // One row block per unit: the output of a finished unit is written by four warps of their own while the
    // softmax warps go on with the next unit, which takes two output accumulators and two Q buffers.
    static constexpr bool EPI = NRB == 1;
    static constexpr int SB = NRB == 1 ? 3 : 1;  // S buffers per row block
    // Two row blocks: a K ring and a V ring.  One row block: K and V tiles share ONE ring, filled in the order
    // they are consumed (K0 K1 K2 V0 K3 V1 K4 V2 ...: S runs three tiles ahead of P V), so every load has the
    // whole ring's depth to land; a V ring of its own would have to be three deep for that, which does not fit.
    static constexpr int KS = EPI ? 5 : 3;       // K stages (EPI: stages of the shared ring)
    static constexpr int VS = EPI ? 0 : 2;       // V stages
    static constexpr int QS = EPI ? 2 : 1;       // Q buffers (units)
    static constexpr int OB = 1;                 // output accumulators per row block
    static constexpr int EPI_THREADS = EPI ? 128 : 0;
    static constexpr int MMA_WARPS = 2;          // issuing threads (one lane of each)
    static constexpr int THREADS = 32 * (1 + MMA_WARPS) + 256 * NRB + EPI_THREADS;
    static constexpr int QB_BYTES = NBOX * BOX_BYTES;  // one Q block
    static constexpr int Q_BYTES = NRB * QB_BYTES;     // the Q blocks of one unit
    static constexpr int KV_BYTES = NBOX * BOX_BYTES;  // one K tile or one V tile
    // barrier slots
    static constexpr int B_KFULL = 0, B_KEMPTY = B_KFULL + KS, B_VFULL = B_KEMPTY + KS, B_VEMPTY = B_VFULL + VS,
                         B_SFULL = B_VEMPTY + VS, B_PREADY = B_SFULL + NRB * SB, B_PVDONE = B_PREADY + NRB * SB,
                         B_QFULL = B_PVDONE + NRB * SB, B_QFREE = B_QFULL + QS, B_UFULL = B_QFREE + QS,
                         B_UEMPTY = B_UFULL + 2, B_PAIR = B_UEMPTY + 2, B_ALL = B_PAIR + 4 * NRB,
                         B_OFULL = B_ALL + NRB, B_OFREE = B_OFULL + OB, B_HFULL = B_OFREE + OB, B_HFREE = B_HFULL + 1,
                         N_BARS = B_HFREE + 1;
    static constexpr int BAR_BYTES = (8 * N_BARS + 15) / 16 * 16;
    static constexpr int XCH_BYTES = NRB * 1024;  // per (block, lane group) 256 bytes: maxima as bf16 or row sums as fp32
    // hand-over from the softmax warps to the output warps: two shares of the row sum and the reference maximum
    static constexpr int HAND_BYTES = EPI ? 3 * 128 * 4 : 0;
    static constexpr int EXTRA = BAR_BYTES + 16 + XCH_BYTES + 2 * 64 + HAND_BYTES;  // barriers, slot/abort/tickets, exchange, ring
    // The operand tiles need 1024-byte alignment.  The dynamic shared window starts 1024-aligned on this
    // architecture (checked at run time: the kernel reports an error instead of running misaligned).
    static constexpr int SLACK = EPI ? 0 : 256;
    static constexpr int USED = (QS * Q_BYTES) + (KS + VS) * KV_BYTES + SLACK + EXTRA;
    // at least ~118 KB so that two CTAs can never share an SM (each allocates all of TMEM)
    static constexpr int SMEM = USED > 120832 ? USED : 120832;
    static constexpr uint32_t O_COL = 0, S_COL = 128 * NRB * OB;
    static_assert(sizeof(UnitDesc) <= 64, "ring slot");
    static_assert(USED <= 232448, "shared memory budget");
    static_assert(S_COL + 128 * NRB * SB <= 512, "tensor memory columns");
};

// Rendezvous on an mbarrier (count = number of participants) with the same bounded wait as every other
// wait here: a hardware named barrier would hang if a participant had left through the abort path.
__device__ __forceinline__ bool group_sync(uint32_t bar, uint32_t &uses, volatile int *abort_flag) {
    mbar_arrive(bar);
    const bool ok = mbar_wait(bar, uses & 1u, abort_flag);
    ++uses;
    return ok;
}

__device__ __forceinline__ unsigned short bf16_bits_rn(float x) {
    return __bfloat16_as_ushort(__float2bfloat16_rn(x));
}
__device__ __forceinline__ float bf16_bits_to_float(unsigned short b) { return __uint_as_float((uint32_t)b << 16); }
}  // namespace attc

template <int D, int NRB>
__global__ void __launch_bounds__(attc::Cfg<D, NRB>::THREADS, 1)
tree_attn_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                    const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmKt,
                    const __grid_constant__ CUtensorMap tmVt, AttnArgs a, TopoMask mask,
                    int32_t *__restrict__ status) {
    using namespace attc;
    using C = Cfg<D, NRB>;
    constexpr int DH = D / 2;  // output columns per thread of a pair
    constexpr int SB = C::SB, KS = C::KS, VS = C::VS, QS = C::QS, OB = C::OB, THREADS = C::THREADS;
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    unsigned char *aligned = smem_raw + (base - raw);
    const uint32_t q_s = base;
    const uint32_t k_s = base + QS * C::Q_BYTES;
    const uint32_t v_s = k_s + KS * C::KV_BYTES;
    const uint32_t bar0 = v_s + VS * C::KV_BYTES;
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };
    unsigned char *extra = aligned + QS * C::Q_BYTES + (KS + VS) * C::KV_BYTES + C::BAR_BYTES;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(extra);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(extra + 4);
    volatile int *tickets = reinterpret_cast<volatile int *>(extra + 8);  // one per row block
    unsigned char *xch_base = extra + 16;
    volatile UnitDesc *ring = reinterpret_cast<volatile UnitDesc *>(extra + 16 + C::XCH_BYTES);  // 2 slots of 64 bytes
    volatile float *hand = reinterpret_cast<volatile float *>(extra + 16 + C::XCH_BYTES + 128);  // [l share 0 | l share 1 | m][128 rows]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int N = a.N, G = a.G;
#ifdef SPECROLL_TRACE
    unsigned long long prof[12] = {0ull, 0ull, 0ull, 0ull, 0ull, 0ull, 0ull, 0ull, 0ull, 0ull, 0ull, 0ull};
    const long long prof_t0 = clock64();
    const unsigned launch_slot = *(volatile unsigned int *)&g_launch_n & 7u;
    if (threadIdx.x == 0 && blockIdx.x < 160) g_cta_ns[launch_slot][0][blockIdx.x] = globaltimer_ns();
    auto twait = [&](int slot, uint32_t b_, uint32_t par_) {
        const long long t_ = clock64();
        const bool r_ = mbar_wait(b_, par_, abort_flag);
        prof[slot] += (unsigned long long)(clock64() - t_);
        return r_;
    };
#else
    auto twait = [&](int, uint32_t b_, uint32_t par_) { return mbar_wait(b_, par_, abort_flag); };
#endif
    // Stage and phase of tile t's K and V (t counts tiles over all units of this CTA) and their barriers.
    auto k_slot = [&](uint32_t t, int &st, uint32_t &ph) {
        const uint32_t pos = C::EPI ? (t < 2u ? t : 2u * t - 2u) : t;
        st = (int)(pos % KS);
        ph = (pos / KS) & 1u;
    };
    auto v_slot = [&](uint32_t t, int &st, uint32_t &ph) {
        if constexpr (C::EPI) {
            const uint32_t pos = 2u * t + 3u;
            st = (int)(pos % KS);
            ph = (pos / KS) & 1u;
        } else {
            st = (int)(t % VS);
            ph = (t / VS) & 1u;
        }
    };
    auto v_addr = [&](int st) { return (C::EPI ? k_s : v_s) + (uint32_t)st * C::KV_BYTES; };
    auto v_full = [&](int st) { return bar((C::EPI ? C::B_KFULL : C::B_VFULL) + st); };
    auto v_empty = [&](int st) { return bar((C::EPI ? C::B_KEMPTY : C::B_VEMPTY) + st); };
    if (base - raw > (uint32_t)C::SLACK) {  // uniform: the whole CTA leaves before touching anything
        if (threadIdx.x == 0) atomicExch(status, SPECROLL_ECUDA);
        return;
    }

    if (threadIdx.x == 0) {
        for (int i = 0; i < C::N_BARS; ++i) {
            uint32_t count = 1;
            if (i >= C::B_PREADY && i < C::B_PREADY + NRB * SB) count = 256;
            // a unit's descriptor is read by the MMA threads, the softmax threads and the output threads
            if (i >= C::B_UEMPTY && i < C::B_UEMPTY + 2) count = C::MMA_WARPS + 256 * NRB + C::EPI_THREADS;
            // two row blocks: each block's thread releases the K and V stages and the Q buffer
            if (!C::EPI && ((i >= C::B_KEMPTY && i < C::B_KEMPTY + KS) || (i >= C::B_VEMPTY && i < C::B_VEMPTY + VS) ||
                            i == C::B_QFREE))
                count = NRB;
            if (i >= C::B_PAIR && i < C::B_PAIR + 4 * NRB) count = 64;
            if (i >= C::B_ALL && i < C::B_ALL + NRB) count = C::EPI ? 128 : 256;
            if (i >= C::B_OFREE && i < C::B_OFREE + OB) count = 128;
            if (i == C::B_HFULL) count = 256;
            if (i == C::B_HFREE) count = 128;
            mbar_init(bar(i), count);
        }
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
    // A Q block's TMA box covers rows_per_block rows; the rest of each 128-row operand stays zero.
    for (int c = threadIdx.x; c < QS * C::Q_BYTES / 16; c += THREADS)
        reinterpret_cast<uint4 *>(aligned)[c] = make_uint4(0u, 0u, 0u, 0u);
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const int units_per_chunk = a.n_rb / NRB;  // row-block groups per (chunk, kv head)

    // Sums the partials of all chunks of one (sequence, kv head, row block) for columns [col0, col0 + ncols) of one row;
    // run by the threads that own the row block, after the tickets showed that every chunk has been written.
    auto merge_rows = [&](int b, int hkv, int rb, int n_splits, int item0, int row, int col0, int ncols) {
        const int gr = rb * a.rows_per_block + row;
        if (!(row < a.rows_per_block && gr < a.rows)) return;
        const int n = gr / G, g = gr % G;
        __nv_bfloat16 *dst_o = a.O + (((size_t)b * N + n) * a.Hq + hkv * G + g) * D + col0;
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
        for (int c = 0; c < ncols; c += 32) {
            float acc[32];
#pragma unroll
            for (int i2 = 0; i2 < 32; ++i2) acc[i2] = 0.f;
            for (int s = 0; s < n_splits; ++s) {
                const size_t pr = ((size_t)(item0 + s) * a.Hkv + hkv) * a.rows_pad + gr;
                const float ms = __ldcg(a.part_ml + pr * 2);
                const float wgt = (ms == -INFINITY) ? 0.f : ex2_approx(ms - Mx) * invl;
                const float4 *src = reinterpret_cast<const float4 *>(a.part_o) +
                                    ((size_t)(item0 + s) * a.Hkv + hkv) * (size_t)(D / 4) * a.rows_pad +
                                    (size_t)((col0 + c) / 4) * a.rows_pad + gr;
#pragma unroll
                for (int i2 = 0; i2 < 8; ++i2) {
                    const float4 x = __ldcg(src + (size_t)i2 * a.rows_pad);
                    acc[4 * i2] += wgt * x.x;
                    acc[4 * i2 + 1] += wgt * x.y;
                    acc[4 * i2 + 2] += wgt * x.z;
                    acc[4 * i2 + 3] += wgt * x.w;
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
        if (a.lse && col0 == 0)
            a.lse[((size_t)b * N + n) * a.Hq + hkv * G + g] = (Mx + log2f(lsum)) * 0.6931471805599453f;
    };

    if (warp == 0) {
        // ------------------------------------------------------------------ scheduler + TMA producer
        if (lane == 0) {
            bool ok = true;
            uint32_t kt = 0, vt = 0;  // K and V tiles loaded so far (all units)
            // V loads trail K loads by two tiles, carried over unit boundaries: (map, kv head, token) of pending V tiles
            const CUtensorMap *pv_map[2];
            int pv_h[2], pv_tok[2];
            int n_pend = 0;
            auto load_v = [&](const CUtensorMap *mv, int hkv, int tok) -> bool {
                int s;
                uint32_t ph;
                v_slot(vt, s, ph);
                if (!twait(0, v_empty(s), ph ^ 1u)) return false;
                const uint32_t dst = v_addr(s);
                mbar_arrive_expect_tx(v_full(s), C::KV_BYTES);
#pragma unroll
                for (int bx = 0; bx < C::NBOX; ++bx)
                    tma_load_3d(dst + bx * BOX_BYTES, mv, bx * 64, hkv, tok, v_full(s));
                ++vt;
                return true;
            };
            for (uint32_t u = 0; ok; ++u) {
                const int slot = (int)(u & 1u);
                if (!twait(1, bar(C::B_UEMPTY + slot), ((u >> 1) & 1u) ^ 1u)) {
                    ok = false;
                    break;
                }
                // the first unit of a CTA is its own index (no round trip before the first loads); the counter
                // hands out the units after those
                const int w = u == 0 ? (int)blockIdx.x : (int)gridDim.x + atomicAdd(a.work_counter, 1);
                volatile UnitDesc *d = ring + slot;
                if (w >= a.total_work) {
                    d->valid = 0;
                    mbar_arrive(bar(C::B_UFULL + slot));
                    break;
                }
                // ---- decode: w = (chunk position in work order * Hkv + hkv) * units_per_chunk + row-block group
                int t = w;
                const int rb = (t % units_per_chunk) * NRB;
                t /= units_per_chunk;
                const int hkv = t % a.Hkv;
                const int si = t / a.Hkv;
                const int4 e0 = __ldg(reinterpret_cast<const int4 *>(a.unit_tab) + 2 * (size_t)si);
                const int4 e1 = __ldg(reinterpret_cast<const int4 *>(a.unit_tab) + 2 * (size_t)si + 1);
                const int b = e0.x, split = e0.y, n_splits = e0.z, item0 = e0.w, kv0 = e1.x, L = e1.y;
                const int tiles_b = (L + BN - 1) / BN;
                const int tps = (tiles_b + n_splits - 1) / n_splits;
                const int t_lo = min(tiles_b, split * tps), t_hi = min(tiles_b, t_lo + tps);
                const int has_tree = (split == n_splits - 1) ? 1 : 0;
                const int n_it = (t_hi - t_lo) + has_tree;
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
                mbar_arrive(bar(C::B_UFULL + slot));  // release: the descriptor is visible to whoever acquires
                SR_TRACE(0, 0, u);
                // ---- Q blocks of this unit, once every S of the previous unit has been computed
                const int qb = (int)(u % QS);
                if (u >= (uint32_t)QS && !twait(2, bar(C::B_QFREE + qb), (u / QS - 1u) & 1u)) {
                    ok = false;
                    break;
                }
                mbar_arrive_expect_tx(bar(C::B_QFULL + qb), (uint32_t)(NRB * C::NBOX * 128 * a.rows_per_block));
#pragma unroll
                for (int blk = 0; blk < NRB; ++blk)
#pragma unroll
                    for (int bx = 0; bx < C::NBOX; ++bx)
                        tma_load_3d(q_s + qb * C::Q_BYTES + blk * C::QB_BYTES + bx * BOX_BYTES, &tmQ, bx * 64, hkv * G,
                                    b * N + (rb + blk) * a.nodes_per_block, bar(C::B_QFULL + qb));
                // ---- K tiles, each followed by the V tile from two tiles back.  Paged cache: kv0 is the sequence's
                //      first slot in the page table and a tile is one pool page; page numbers are fetched two
                //      tiles ahead of their use, under the wait for a free stage.
                const int n_kv = t_hi - t_lo;
                const int32_t *pt = a.page_table ? a.page_table + kv0 + t_lo : nullptr;
                int pg0 = (pt && n_kv > 0) ? __ldg(pt) : 0, pg1 = (pt && n_kv > 1) ? __ldg(pt + 1) : 0;
                for (int it = 0; it < n_it && ok; ++it) {
                    const int pg2 = (pt && it + 2 < n_kv) ? __ldg(pt + it + 2) : 0;
                    int s;
                    uint32_t kph;
                    k_slot(kt, s, kph);
                    if (!twait(3, bar(C::B_KEMPTY + s), kph ^ 1u)) {
                        ok = false;
                        break;
                    }
                    const bool tree = has_tree && (it == n_it - 1);
                    const int tok = tree ? b * N : (pt ? pg0 * BN : kv0 + (t_lo + it) * BN);
                    pg0 = pg1;
                    pg1 = pg2;
                    const CUtensorMap *mk = tree ? &tmKt : &tmK;
                    const uint32_t dst = k_s + s * C::KV_BYTES;
                    mbar_arrive_expect_tx(bar(C::B_KFULL + s), C::KV_BYTES);
#pragma unroll
                    for (int bx = 0; bx < C::NBOX; ++bx)
                        tma_load_3d(dst + bx * BOX_BYTES, mk, bx * 64, hkv, tok, bar(C::B_KFULL + s));
                    ++kt;
                    SR_TRACE(0, 1, kt);
                    if (n_pend == 2) {
                        ok = load_v(pv_map[0], pv_h[0], pv_tok[0]);
                        pv_map[0] = pv_map[1];
                        pv_h[0] = pv_h[1];
                        pv_tok[0] = pv_tok[1];
                        n_pend = 1;
                    }
                    pv_map[n_pend] = tree ? &tmVt : &tmV;
                    pv_h[n_pend] = hkv;
                    pv_tok[n_pend] = tok;
                    ++n_pend;
                }
                // The next unit's Q waits for this unit's last S, which is issued after the P V of the tile SB
                // before it: with a single S buffer that P V needs the second-to-last V tile, so it must go
                // out now (its stage depends on earlier tiles only).
                if (SB == 1 && ok && n_pend == 2) {
                    ok = load_v(pv_map[0], pv_h[0], pv_tok[0]);
                    pv_map[0] = pv_map[1];
                    pv_h[0] = pv_h[1];
                    pv_tok[0] = pv_tok[1];
                    n_pend = 1;
                }
                // the unit's last V tiles go out now if their stages are already free; otherwise they wait
                // behind the next unit's Q and first K tiles (never block here)
                auto v_stage_free = [&]() {
                    int s;
                    uint32_t ph;
                    v_slot(vt, s, ph);
                    return mbar_test_wait(v_empty(s), ph ^ 1u);
                };
                while (ok && n_pend > 0 && v_stage_free()) {
                    ok = load_v(pv_map[0], pv_h[0], pv_tok[0]);
                    pv_map[0] = pv_map[1];
                    pv_h[0] = pv_h[1];
                    pv_tok[0] = pv_tok[1];
                    --n_pend;
                }
            }
            // flush the V tiles still pending (the last two tiles of the last unit)
            for (int i = 0; i < n_pend && ok; ++i) ok = load_v(pv_map[i], pv_h[i], pv_tok[i]);
            if (!ok) {
                // aborting: give copies in flight time to land before the CTA goes away
                const unsigned long long t0 = globaltimer_ns();
                while (globaltimer_ns() - t0 < 20000000ull) {
                }
            }
        }
    } else if (warp <= C::MMA_WARPS) {
        // ------------------------------------------------------------------ MMA issuers (one thread each of two warps)
        // The tensor pipe is fed by two threads, so that one can be queueing operations while the other sits
        // in a barrier wait: with one issuing thread the pipe idled more than half of the time.
        //   one row block per unit: warp 1 issues every S = Q K^T, warp 2 every O += P V;
        //   two row blocks: warp 1 + b issues both products of block b, in the order that lets an S tile
        //   overwrite the buffer whose P the previously issued P V has read (operations of one thread
        //   execute in issue order).
        if (lane == 0) {
            constexpr uint32_t idesc_s = idesc_bf16(128, BN, false, false);
            constexpr uint32_t idesc_pv = idesc_bf16(128, D, false, true);  // V is read MN-major
            // Descriptors are assembled from precomputed halves: the high word is constant, the low word is
            // the operand's shared-memory address / 16 (14 bits) plus, for V, LBO / 16 << 16.
            constexpr uint32_t DESC_HI = (1024u >> 4) | (1u << 14) | (2u << 29);  // SBO 1024, version, 128B swizzle
            constexpr uint32_t V_LBO = ((uint32_t)BOX_BYTES >> 4) << 16;
            constexpr uint32_t BOXU = (uint32_t)BOX_BYTES >> 4;
            auto desc = [](uint32_t lo) -> uint64_t { return ((uint64_t)DESC_HI << 32) | (uint64_t)lo; };
            // S of one tile: D/16 operations into S buffer sb
            auto mma_s = [&](uint32_t q_lo, uint32_t k_lo, int sb) {
                const uint32_t d_t = tmem_base + C::S_COL + 128u * (uint32_t)sb;
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint32_t off = (uint32_t)(kk >> 2) * BOXU + (uint32_t)(kk & 3) * 2u;
                    umma_ss(d_t, desc(q_lo + off), desc(k_lo + off), idesc_s, kk > 0 ? 1u : 0u);
                }
            };
            // O += P V of one tile: 16 tokens per operation, 2048 bytes (128 address units) down the V tile; P of
            // tokens 0-63 sits in columns [0,32) of the S buffer, of tokens 64-127 in columns [96,128), 8 packed
            // columns per operation
            auto mma_pv = [&](uint32_t o_t, int sb, uint32_t v_lo, uint32_t acc0) {
                const uint32_t p_t = tmem_base + C::S_COL + 128u * (uint32_t)sb;
#pragma unroll
                for (int kk = 0; kk < BN / 16; ++kk) {
                    const uint32_t pcol = kk < 4 ? 8u * kk : 64u + 8u * kk;
                    umma_ts(o_t, p_t + pcol, desc(v_lo + 128u * kk), idesc_pv, kk > 0 ? 1u : acc0);
                }
            };
            if constexpr (C::EPI) {
                if (warp == 1) {
                    // ---- S issuer: runs up to SB tiles ahead of the P V issuer, also across a unit boundary (the
                    //      next unit's Q has its own buffer)
                    uint32_t ts = 0;
                    bool ok = true;
                    for (uint32_t u = 0; ok; ++u) {
                        const int slot = (int)(u & 1u);
                        if (!twait(0, bar(C::B_UFULL + slot), (u >> 1) & 1u)) break;
                        const int valid = ring[slot].valid, n_it = ring[slot].n_it;
                        mbar_arrive(bar(C::B_UEMPTY + slot));
                        if (!valid) break;
                        const int qb = (int)(u % QS);
                        if (!twait(1, bar(C::B_QFULL + qb), (u / QS) & 1u)) break;
                        const uint32_t q_lo = (q_s + qb * C::Q_BYTES) >> 4;
                        for (int j = 0; j < n_it; ++j, ++ts) {
                            const int sb = (int)(ts % SB);
                            int ks;
                            uint32_t kph;
                            k_slot(ts, ks, kph);
                            // the P V that read P from this buffer must be complete
                            if (ts >= (uint32_t)SB && !twait(3, bar(C::B_PVDONE + sb), (ts / SB - 1u) & 1u)) {
                                ok = false;
                                break;
                            }
                            if (!twait(2, bar(C::B_KFULL + ks), kph)) {
                                ok = false;
                                break;
                            }
                            tc_fence_after();
                            mma_s(q_lo, (k_s + ks * C::KV_BYTES) >> 4, sb);
                            umma_commit(bar(C::B_SFULL + sb));
                            umma_commit(bar(C::B_KEMPTY + ks));  // the stage is free once this S has been computed
                            SR_TRACE(1, 1, ts);
                        }
                        umma_commit(bar(C::B_QFREE + qb));  // every S of the unit computed: its Q buffer may be replaced
                    }
                } else {
                    // ---- P V issuer
                    uint32_t tp = 0;
                    bool ok = true;
                    for (uint32_t u = 0; ok; ++u) {
                        const int slot = (int)(u & 1u);
                        if (!twait(0, bar(C::B_UFULL + slot), (u >> 1) & 1u)) break;
                        const int valid = ring[slot].valid, n_it = ring[slot].n_it;
                        mbar_arrive(bar(C::B_UEMPTY + slot));
                        if (!valid) break;
                        // the output threads have read the accumulator of the unit before
                        if (!twait(3, bar(C::B_OFREE), (u & 1u) ^ 1u)) break;
                        const uint32_t o_t = tmem_base + C::O_COL;
                        for (int j = 0; j < n_it; ++j, ++tp) {
                            const int sb = (int)(tp % SB);
                            int vs;
                            uint32_t vph;
                            v_slot(tp, vs, vph);
                            if (!twait(4, bar(C::B_PREADY + sb), (tp / SB) & 1u) || !twait(5, v_full(vs), vph)) {
                                ok = false;
                                break;
                            }
                            tc_fence_after();
                            mma_pv(o_t, sb, (v_addr(vs) >> 4) | V_LBO, j > 0 ? 1u : 0u);
                            umma_commit(v_empty(vs));
                            umma_commit(bar(C::B_PVDONE + sb));
                            SR_TRACE(1, 3, tp);
                        }
                        if (ok) umma_commit(bar(C::B_OFULL));  // the unit's accumulator is complete when this arrives
                    }
                }
            } else {
                const int blk = warp - 1;  // this thread's row block
                uint32_t gt = 0;           // tiles issued so far (all units)
                bool ok = true;
                for (uint32_t u = 0; ok; ++u) {
                    const int slot = (int)(u & 1u);
                    if (!twait(0, bar(C::B_UFULL + slot), (u >> 1) & 1u)) break;
                    const int valid = ring[slot].valid, n_it = ring[slot].n_it;
                    mbar_arrive(bar(C::B_UEMPTY + slot));
                    if (!valid) break;
                    if (!twait(1, bar(C::B_QFULL), u & 1u)) break;
                    tc_fence_after();
                    if (n_it == 0) {
                        umma_commit(bar(C::B_QFREE));
                        continue;
                    }
                    const uint32_t q_lo = (q_s + blk * C::QB_BYTES) >> 4;
                    const uint32_t o_t = tmem_base + C::O_COL + 128u * (uint32_t)blk;
                    // S of tile j; every block's thread waits for the K tile and releases it (the barrier counts them)
                    auto issue_s = [&](int j) -> bool {
                        const uint32_t t = gt + (uint32_t)j;
                        const int ks = (int)(t % KS);
                        if (!twait(2, bar(C::B_KFULL + ks), (t / KS) & 1u)) return false;
                        tc_fence_after();
                        const int sb = blk * SB + (int)(t % SB);
                        mma_s(q_lo, (k_s + ks * C::KV_BYTES) >> 4, sb);
                        umma_commit(bar(C::B_SFULL + sb));
                        SR_TRACE(1, 1, t);
                        umma_commit(bar(C::B_KEMPTY + ks));  // the K tile is free once every block's S has been computed
                        if (j == n_it - 1) umma_commit(bar(C::B_QFREE));  // last S of the unit: Q may be replaced
                        return true;
                    };
                    for (int j = 0; j < SB && j < n_it && ok; ++j) ok = issue_s(j);
                    for (int j = 0; j < n_it && ok; ++j) {
                        const uint32_t t = gt + (uint32_t)j;
                        const int vs = (int)(t % VS);
                        const int sb = blk * SB + (int)(t % SB);
                        if (!twait(4, bar(C::B_PREADY + sb), (t / SB) & 1u) || !twait(5, bar(C::B_VFULL + vs), (t / VS) & 1u)) {
                            ok = false;
                            break;
                        }
                        SR_TRACE(1, 2, t);
                        tc_fence_after();
                        mma_pv(o_t, sb, ((v_s + vs * C::KV_BYTES) >> 4) | V_LBO, j > 0 ? 1u : 0u);
                        umma_commit(bar(C::B_VEMPTY + vs));
                        umma_commit(bar(C::B_PVDONE + sb));
                        SR_TRACE(1, 3, t);
                        if (j + SB < n_it) ok = issue_s(j + SB);  // reuses the buffer this P V has just read
                    }
                    gt += (uint32_t)n_it;
                }
            }
        }
    } else if (C::EPI && warp >= 1 + C::MMA_WARPS + 8 * NRB) {
        // ------------------------------------------------------------------ output (4 warps, one thread per query row)
        // Takes a finished unit's accumulator out of TMEM while the other warps are already in the next unit.
        const int lg = warp & 3;  // TMEM lane group of this warp
        const int row = lg * 32 + lane;
        const uint32_t t_lane = tmem_base + ((uint32_t)(lg * 32) << 16);
        const int tix = (int)threadIdx.x - (32 * (1 + C::MMA_WARPS) + 256 * NRB);
        const uint32_t all_bar = bar(C::B_ALL);
        uint32_t use_all = 0;
        bool ok = true;
        for (uint32_t u = 0; ok; ++u) {
            const int slot = (int)(u & 1u);
            ok = twait(0, bar(C::B_UFULL + slot), (u >> 1) & 1u);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            const int valid = ring[slot].valid, b = ring[slot].b, hkv = ring[slot].hkv, rb = ring[slot].rb;
            const int n_splits = ring[slot].n_splits, n_it = ring[slot].n_it, item = ring[slot].item;
            const int item0 = ring[slot].item0;
            mbar_arrive(bar(C::B_UEMPTY + slot));
            if (!valid) break;
            const int ob = (int)(u % OB);
            const int gr = rb * a.rows_per_block + row;
            const bool row_ok = row < a.rows_per_block && gr < a.rows;
            // ---- the row's sum (two shares) and reference maximum, left by the softmax threads at the end of the unit
            ok = twait(1, bar(C::B_HFULL), u & 1u);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            const float lt = hand[row] + hand[128 + row];
            const float m_used = hand[256 + row];
            mbar_arrive(bar(C::B_HFREE));
            // ---- the unit's last P V (operations complete in issue order, so it covers all)
            ok = twait(2, bar(C::B_OFULL + ob), (u / OB) & 1u);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            if (lane == 0 && lg == 2) SR_TRACE(3, 3, u);
            const uint32_t o_t = t_lane + C::O_COL + 128u * (uint32_t)ob;
            const int n = row_ok ? gr / G : 0, g = row_ok ? gr % G : 0;
            const bool direct = (n_splits == 1);
            const float inv = direct ? (lt > 0.f ? 1.0f / lt : 0.f) : 1.0f;
            __nv_bfloat16 *dst_o = a.O + (((size_t)b * N + n) * a.Hq + hkv * G + g) * D;
            // partials are stored [unit][float4 column][row] so that a warp's stores are contiguous
            const size_t pbase = ((size_t)item * a.Hkv + hkv) * (size_t)(D / 4) * a.rows_pad;
            float4 *dst_p = reinterpret_cast<float4 *>(a.part_o) + pbase + (row_ok ? gr : 0);
#pragma unroll 1
            for (int c = 0; c < D; c += 32) {
                uint32_t o[32];
                if (n_it > 0) {
                    tmem_ld32(o_t + (uint32_t)c, o);
                    tmem_ld_wait();
                } else {
#pragma unroll
                    for (int i2 = 0; i2 < 32; ++i2) o[i2] = 0u;
                }
                if (c + 32 >= D) {  // everything has been read: the accumulator may be overwritten (two units on)
                    tc_fence_before();
                    mbar_arrive(bar(C::B_OFREE + ob));
                }
                if (!row_ok) continue;
                if (direct) {
#pragma unroll
                    for (int i2 = 0; i2 < 32; i2 += 8) {
                        uint4 q4;
                        q4.x = pack_bf16x2(__uint_as_float(o[i2]) * inv, __uint_as_float(o[i2 + 1]) * inv);
                        q4.y = pack_bf16x2(__uint_as_float(o[i2 + 2]) * inv, __uint_as_float(o[i2 + 3]) * inv);
                        q4.z = pack_bf16x2(__uint_as_float(o[i2 + 4]) * inv, __uint_as_float(o[i2 + 5]) * inv);
                        q4.w = pack_bf16x2(__uint_as_float(o[i2 + 6]) * inv, __uint_as_float(o[i2 + 7]) * inv);
                        *reinterpret_cast<uint4 *>(dst_o + c + i2) = q4;
                    }
                } else {
#pragma unroll
                    for (int i2 = 0; i2 < 32; i2 += 4)
                        dst_p[(size_t)((c + i2) / 4) * a.rows_pad] =
                            make_float4(__uint_as_float(o[i2]), __uint_as_float(o[i2 + 1]), __uint_as_float(o[i2 + 2]),
                                        __uint_as_float(o[i2 + 3]));
                }
            }
            const size_t prow = ((size_t)item * a.Hkv + hkv) * a.rows_pad + (row_ok ? gr : 0);
            if (row_ok) {
                if (direct) {
                    if (a.lse) a.lse[((size_t)b * N + n) * a.Hq + hkv * G + g] = (m_used + log2f(lt)) * 0.6931471805599453f;
                } else {
                    a.part_ml[prow * 2] = m_used;
                    a.part_ml[prow * 2 + 1] = lt;
                }
            }
            if (!direct && a.merge_mode == 0) {
                // Unless a later kernel does the merging: the chunk whose ticket comes last merges all chunks
                // of this (sequence, kv head, row block).  Nobody waits for anybody.
                __threadfence();
                bool ok3 = group_sync(all_bar, use_all, abort_flag);
                if (tix == 0) tickets[0] = atomicAdd(a.split_counters + (b * a.Hkv + hkv) * a.n_rb + rb, 1);
                ok3 = group_sync(all_bar, use_all, abort_flag) && ok3;
                if (ok3 && tickets[0] == n_splits - 1) {
                    __threadfence();
                    merge_rows(b, hkv, rb, n_splits, item0, row, 0, D);
                }
            }
            if (lane == 0 && lg == 2) SR_TRACE(3, 4, u);
        }
    } else {
        // ------------------------------------------------------------------ softmax (8 warps per row block)
        const int ws = warp - (1 + C::MMA_WARPS);
        const int blk = ws >> 3;            // row block of the unit
        const int half = (ws & 7) >> 2;     // which 64 of a tile's 128 columns, and which D/2 output columns
        const int lg = warp & 3;            // TMEM lane group of this warp
        const int row = lg * 32 + lane;
        const uint32_t t_lane = tmem_base + ((uint32_t)(lg * 32) << 16);
        const uint32_t o_t0 = t_lane + C::O_COL + 128u * (uint32_t)(blk * OB) + (uint32_t)(half * DH);
        const float sc = a.scale_log2;
        // exchange area of this (row block, lane group), 256 bytes, touched by the group's two warps only:
        // maxima as bf16 [2 slots][2 halves][32 lanes]; row sums as fp32 [2 halves][32 lanes]
        volatile unsigned short *xm = reinterpret_cast<volatile unsigned short *>(xch_base + blk * 1024 + lg * 256);
        volatile float *xl = reinterpret_cast<volatile float *>(xch_base + blk * 1024 + lg * 256);
        volatile int *ticket = tickets + blk;
        const int tix = (ws & 7) * 32 + lane;  // thread index within the row block
        uint32_t gt = 0;  // tiles processed so far (all units)
        uint32_t use_pair = 0, use_all = 0;
        const uint32_t pair_bar = bar(C::B_PAIR + blk * 4 + lg), all_bar = bar(C::B_ALL + blk);
        bool ok = true;
        for (uint32_t u = 0; ok; ++u) {
            const int slot = (int)(u & 1u);
            ok = twait(0, bar(C::B_UFULL + slot), (u >> 1) & 1u);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            const int valid = ring[slot].valid, b = ring[slot].b, hkv = ring[slot].hkv, rb = ring[slot].rb + blk;
            const int n_splits = ring[slot].n_splits, L = ring[slot].L, t_lo = ring[slot].t_lo;
            const int n_it = ring[slot].n_it, has_tree = ring[slot].has_tree, item = ring[slot].item;
            const int item0 = ring[slot].item0;
            mbar_arrive(bar(C::B_UEMPTY + slot));
            if (!valid) break;
            const int gr = rb * a.rows_per_block + row;
            const bool row_ok = row < a.rows_per_block && gr < a.rows;
            const uint64_t anc = row_ok ? mask.anc[gr / G] : 0ull;
            const uint32_t o_t = o_t0 + 128u * (uint32_t)(u % OB);  // this unit's accumulator
            float m_used = -INFINITY, l = 0.f;  // l: this thread's share (its 64 columns of every tile)
            for (int j = 0; j < n_it; ++j) {
                const uint32_t t = gt + (uint32_t)j;
                const int sb = blk * SB + (int)(t % SB);
                ok = twait(1, bar(C::B_SFULL + sb), (t / SB) & 1u);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
                if ((ws & 7) == 0 && lane == 0) SR_TRACE(2 + blk, 1, t);
                const uint32_t s_t = t_lane + C::S_COL + 128u * (uint32_t)sb;
                const bool tree = has_tree && (j == n_it - 1);
                // columns >= limit are outside the sequence; this thread's columns start at 64 * half
                const int limit = (tree ? 64 : (L - (t_lo + j) * BN)) - 64 * half;
                const bool full = !tree && limit >= 64;
                uint32_t bits0, bits1;  // admissible columns among this thread's 64, in two groups of 32
                if (full) {
                    bits0 = bits1 = 0xffffffffu;
                } else if (tree) {
                    bits0 = half == 0 ? (uint32_t)anc : 0u;
                    bits1 = half == 0 ? (uint32_t)(anc >> 32) : 0u;
                } else {
                    bits0 = limit >= 32 ? 0xffffffffu : (limit <= 0 ? 0u : ((1u << limit) - 1u));
                    bits1 = limit >= 64 ? 0xffffffffu : (limit <= 32 ? 0u : ((1u << (limit - 32)) - 1u));
                }
                // ---- pass 1: maximum of this thread's 64 columns
                uint32_t r0[32], r1[32];
                float mx0 = -INFINITY, mx1 = -INFINITY;
                auto max_group = [&](const uint32_t(&src)[32], uint32_t bc) {
                    if (full) {
#pragma unroll
                        for (int i2 = 0; i2 < 32; i2 += 2) {
                            mx0 = fmaxf(mx0, __uint_as_float(src[i2]));
                            mx1 = fmaxf(mx1, __uint_as_float(src[i2 + 1]));
                        }
                    } else {
#pragma unroll
                        for (int i2 = 0; i2 < 32; ++i2)
                            if ((bc >> i2) & 1u) mx0 = fmaxf(mx0, __uint_as_float(src[i2]));
                    }
                };
                if constexpr (NRB == 1) {
                    tmem_ld32(s_t + 64u * half, r0);
                    tmem_ld32(s_t + 64u * half + 32u, r1);
                    tmem_ld_wait();
                    max_group(r0, bits0);
                    max_group(r1, bits1);
                } else {  // fewer registers: one group at a time, and both are read again in pass 2
                    tmem_ld32(s_t + 64u * half, r0);
                    tmem_ld_wait();
                    max_group(r0, bits0);
                    tmem_ld32(s_t + 64u * half + 32u, r0);
                    tmem_ld_wait();
                    max_group(r0, bits1);
                }
                // ---- exchange the partial maximum with the thread that has the row's other 64 columns.  It
                //      travels as bf16: any common reference close to the true maximum will do.  Two slots,
                //      alternating, so that a fast thread's next write cannot overtake a slow read.
                const unsigned short mine = bf16_bits_rn(fmaxf(mx0, mx1));
                const int px = (int)(use_pair & 1u) * 64;
                xm[px + half * 32 + lane] = mine;
#ifdef SPECROLL_TRACE
                const long long tps_ = clock64();
#endif
                ok = group_sync(pair_bar, use_pair, abort_flag);
#ifdef SPECROLL_TRACE
                prof[4] += (unsigned long long)(clock64() - tps_);
#endif
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                const float mt = fmaxf(bf16_bits_to_float(mine), bf16_bits_to_float(xm[px + (half ^ 1) * 32 + lane])) * sc;
                float alpha = 1.f;
                const bool need = mt > m_used + RESCALE_LOG2;  // also true on the first admissible tile
                if (need) {
                    alpha = (m_used == -INFINITY) ? 0.f : ex2_approx(m_used - mt);
                    m_used = mt;
                    l *= alpha;
                }
                if (__any_sync(0xffffffffu, need) && j > 0) {
                    // rows of this warp change their reference maximum: rescale this thread's half of their
                    // running outputs in TMEM.  The previous tile's P V must have landed first.
                    const int sbp = blk * SB + (int)((t - 1u) % SB);
                    ok = twait(2, bar(C::B_PVDONE + sbp), ((t - 1u) / SB) & 1u);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    tc_fence_after();
#pragma unroll 1
                    for (int c = 0; c < DH; c += 32) {
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
                // ---- pass 2: p = 2^(s*scale - m) as packed bf16 pairs.  Each 32-column group becomes 16 packed
                //      columns, stored over S columns this thread has already read: [0,32) for the first thread
                //      of the pair, [96,128) for the second.
                float ls0 = 0.f, ls1 = 0.f;
                auto exp_group = [&](const uint32_t(&src)[32], uint32_t bc, uint32_t dst_col) {
                    uint32_t pk[16];
#pragma unroll
                    for (int i2 = 0; i2 < 32; i2 += 2) {
                        float p0 = ex2_approx(fmaf(__uint_as_float(src[i2]), sc, -mref));
                        float p1 = ex2_approx(fmaf(__uint_as_float(src[i2 + 1]), sc, -mref));
                        if (!full) {
                            p0 = ((bc >> i2) & 1u) ? p0 : 0.f;
                            p1 = ((bc >> (i2 + 1)) & 1u) ? p1 : 0.f;
                        }
                        ls0 += p0;
                        ls1 += p1;
                        pk[i2 >> 1] = pack_bf16x2(p0, p1);
                    }
                    tmem_st16(dst_col, pk);
                };
                if constexpr (NRB == 1) {
                    exp_group(r0, bits0, s_t + 96u * half);
                    exp_group(r1, bits1, s_t + 96u * half + 16u);
                } else {
                    // second read of S; the second thread of a pair takes its upper group first, so that P
                    // never lands on columns it has yet to read
                    if (half == 0) {
                        tmem_ld32(s_t, r0);
                        tmem_ld_wait();
                        exp_group(r0, bits0, s_t);
                        tmem_ld32(s_t + 32u, r0);
                        tmem_ld_wait();
                        exp_group(r0, bits1, s_t + 16u);
                    } else {
                        tmem_ld32(s_t + 96u, r0);
                        tmem_ld_wait();
                        exp_group(r0, bits1, s_t + 112u);
                        tmem_ld32(s_t + 64u, r0);
                        tmem_ld_wait();
                        exp_group(r0, bits0, s_t + 96u);
                    }
                }
                tmem_st_wait();
                l += ls0 + ls1;
                tc_fence_before();
                mbar_arrive(bar(C::B_PREADY + sb));
                if ((ws & 7) == 0 && lane == 0) SR_TRACE(2 + blk, 2, t);
            }
            if constexpr (C::EPI) {
                // ---- hand the row's reference maximum and this thread's share of its sum to the output warps
                //      and go on with the next unit; they wait for the unit's last P V themselves
                gt += (uint32_t)n_it;
                if ((ws & 7) == 0 && lane == 0) SR_TRACE(2 + blk, 3, u);
                ok = twait(3, bar(C::B_HFREE), (u & 1u) ^ 1u);  // the values of the unit before have been taken
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                hand[half * 128 + row] = l;
                if (half == 0) hand[256 + row] = m_used;
                mbar_arrive(bar(C::B_HFULL));
                continue;
            }
            // ---- wait for the unit's last P V of this block (operations complete in issue order, so it covers all)
            if (ok && n_it > 0) {
                const uint32_t tl = gt + (uint32_t)n_it - 1u;
                ok = twait(2, bar(C::B_PVDONE + blk * SB + (int)(tl % SB)), (tl / SB) & 1u);
                ok = __all_sync(0xffffffffu, ok);
            }
            gt += (uint32_t)n_it;
            if ((ws & 7) == 0 && lane == 0) SR_TRACE(2 + blk, 3, u);
            // ---- row sum = the pair's two shares (fp32 through the same area: rendezvous before reusing it)
            if (ok) ok = group_sync(pair_bar, use_pair, abort_flag);
            xl[half * 32 + lane] = l;
            if (ok) ok = group_sync(pair_bar, use_pair, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const float lt = l + xl[(half ^ 1) * 32 + lane];
            if (ok) ok = group_sync(pair_bar, use_pair, abort_flag);  // both have read before the area is reused
            {
                // ---- output (or this chunk's partial): this thread's D/2 columns of its row
                const int n = row_ok ? gr / G : 0, g = row_ok ? gr % G : 0;
                const bool direct = (n_splits == 1);
                const float inv = direct ? (lt > 0.f ? 1.0f / lt : 0.f) : 1.0f;
                __nv_bfloat16 *dst_o = a.O + (((size_t)b * N + n) * a.Hq + hkv * G + g) * D + half * DH;
                // partials are stored [unit][float4 column][row] so that a warp's stores are contiguous
                const size_t pbase = ((size_t)item * a.Hkv + hkv) * (size_t)(D / 4) * a.rows_pad;
                float4 *dst_p = reinterpret_cast<float4 *>(a.part_o) + pbase + (size_t)(half * (DH / 4)) * a.rows_pad +
                                (row_ok ? gr : 0);
#pragma unroll 1
                for (int c = 0; c < DH; c += 32) {
                    uint32_t o[32];
                    if (n_it > 0) {
                        tmem_ld32(o_t + (uint32_t)c, o);
                        tmem_ld_wait();
                    } else {
#pragma unroll
                        for (int i2 = 0; i2 < 32; ++i2) o[i2] = 0u;
                    }
                    if (!row_ok) continue;
                    if (direct) {
#pragma unroll
                        for (int i2 = 0; i2 < 32; i2 += 8) {
                            uint4 q4;
                            q4.x = pack_bf16x2(__uint_as_float(o[i2]) * inv, __uint_as_float(o[i2 + 1]) * inv);
                            q4.y = pack_bf16x2(__uint_as_float(o[i2 + 2]) * inv, __uint_as_float(o[i2 + 3]) * inv);
                            q4.z = pack_bf16x2(__uint_as_float(o[i2 + 4]) * inv, __uint_as_float(o[i2 + 5]) * inv);
                            q4.w = pack_bf16x2(__uint_as_float(o[i2 + 6]) * inv, __uint_as_float(o[i2 + 7]) * inv);
                            *reinterpret_cast<uint4 *>(dst_o + c + i2) = q4;
                        }
                    } else {
#pragma unroll
                        for (int i2 = 0; i2 < 32; i2 += 4)
                            dst_p[(size_t)((c + i2) / 4) * a.rows_pad] =
                                make_float4(__uint_as_float(o[i2]), __uint_as_float(o[i2 + 1]), __uint_as_float(o[i2 + 2]),
                                            __uint_as_float(o[i2 + 3]));
                    }
                }
                const size_t prow = ((size_t)item * a.Hkv + hkv) * a.rows_pad + (row_ok ? gr : 0);
                if (row_ok && half == 0) {
                    if (direct) {
                        if (a.lse) a.lse[((size_t)b * N + n) * a.Hq + hkv * G + g] = (m_used + log2f(lt)) * 0.6931471805599453f;
                    } else {
                        a.part_ml[prow * 2] = m_used;
                        a.part_ml[prow * 2 + 1] = lt;
                    }
                }
                if (!direct) {
                    // Unless a later kernel does the merging: the chunk whose ticket comes last merges all chunks
                    // of this (sequence, kv head, row block).  Nobody waits for anybody.
                    if (a.merge_mode == 0) {
                        __threadfence();
                        bool ok3 = group_sync(all_bar, use_all, abort_flag);
                        if (tix == 0) *ticket = atomicAdd(a.split_counters + (b * a.Hkv + hkv) * a.n_rb + rb, 1);
                        ok3 = group_sync(all_bar, use_all, abort_flag) && ok3;
                        if (ok3 && *ticket == n_splits - 1) {
                            __threadfence();
                            merge_rows(b, hkv, rb, n_splits, item0, row, half * DH, DH);
                        }
                    }
                }
            }
            if ((ws & 7) == 0 && lane == 0) SR_TRACE(2 + blk, 4, u);
            // No rendezvous is needed before the next unit: its first P V of this block (which overwrites O)
            // waits for the P of all 256 threads of the block, and each arrives only after reading O here.
            tc_fence_before();
        }
    }

    // ------------------------------------------------------------------ teardown
#ifdef SPECROLL_TRACE
    if (lane == 0 && (warp <= 3 || (C::EPI && warp == 1 + C::MMA_WARPS + 8 * NRB))) {
        const int role = warp <= 1 ? warp : (warp == 2 ? 4 : (warp == 3 ? 2 : 3));  // 0 producer, 1 / 4 MMA, 2 softmax, 3 output
        if (warp == 0 && blockIdx.x < 160) g_cta_ns[launch_slot][1][blockIdx.x] = globaltimer_ns();
        prof[11] = (unsigned long long)(clock64() - prof_t0);
        for (int i = 0; i < 12; ++i) atomicAdd(&g_prof[role][i], prof[i]);
    }
#endif
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0) {
        if (*abort_flag) {
            // status word 1: index of the barrier whose wait ran out, parity in bit 8 (diagnostic only)
            if (atomicExch(status, SPECROLL_ETIMEOUT) == 0)
                status[1] = (int)((((uint32_t)*abort_flag & 0xffffffu) - bar0) / 8u) | (((*abort_flag >> 24) & 1) << 8) |
                            (int)(blockIdx.x << 16);
        }
        // the CTA that leaves last clears the scheduling counters, so the same plan can be launched again
        __threadfence();
        tickets[0] = (atomicAdd(a.work_counter + 1, 1) == (int)gridDim.x - 1) ? 1 : 0;
    }
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
    __syncthreads();
    if (tickets[0]) {
        const int n_split = a.B * a.Hkv * a.n_rb;
        for (int i = threadIdx.x; i < n_split; i += THREADS) a.split_counters[i] = 0;
        if (threadIdx.x == 0) {
            a.work_counter[0] = 0;
            a.work_counter[1] = 0;
#ifdef SPECROLL_TRACE
            g_launch_n = g_launch_n + 1u;
#endif
        }
    }
}

template <int D, int NRB>
static int launch_tc(const AttnArgs &a, const TopoMask &mask, long long T_kv, int32_t *status, cudaStream_t st) {
    using C = attc::Cfg<D, NRB>;
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
        SR_CUDA_TRY(cudaFuncSetAttribute(tree_attn_tc_kernel<D, NRB>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM));
    }
    const unsigned grid = (unsigned)(a.total_work < n_sm ? a.total_work : n_sm);
    tree_attn_tc_kernel<D, NRB><<<grid, C::THREADS, C::SMEM, st>>>(tmQ, tmK, tmV, tmKt, tmVt, a, mask, status);
    SR_LAUNCH_CHECK();
    return SPECROLL_OK;
}

// Sums the chunks of every split sequence (the plan uses this instead of merging inside the attention kernel
// when some sequence has many chunks: there the last chunk's CTA would sit on a long chain of dependent loads).
// grid = (chunks in work order, Hkv * n_rb, D / 32); only the block of a split sequence's first chunk works.
// 256 threads: 128 rows x 2 groups of 4 float4 columns.
template <int D>
__global__ void __launch_bounds__(256) attn_merge_tc_kernel(AttnArgs a) {
    const int4 e0 = __ldg(reinterpret_cast<const int4 *>(a.unit_tab) + 2 * (size_t)blockIdx.x);
    const int b = e0.x, n_splits = e0.z, item0 = e0.w;
    if (e0.y != 0 || n_splits < 2) return;
    const int hkv = blockIdx.y / a.n_rb, rb = blockIdx.y % a.n_rb;
    const int row = threadIdx.x & 127, cg = threadIdx.x >> 7;
    const int gr = rb * a.rows_per_block + row;
    if (row >= a.rows_per_block || gr >= a.rows) return;
    const int c4 = blockIdx.z * 8 + cg * 4;  // first of this thread's 4 float4 columns
    const size_t unit_ml = (size_t)a.Hkv * a.rows_pad, unit_o = (size_t)a.Hkv * (D / 4) * a.rows_pad;
    const float *ml = a.part_ml + 2 * (((size_t)item0 * a.Hkv + hkv) * a.rows_pad + gr);
    const float4 *po = reinterpret_cast<const float4 *>(a.part_o) + ((size_t)item0 * a.Hkv + hkv) * (size_t)(D / 4) * a.rows_pad +
                       (size_t)c4 * a.rows_pad + gr;
    float Mx = -INFINITY;
    for (int s = 0; s < n_splits; ++s) Mx = fmaxf(Mx, __ldcg(ml + 2 * s * unit_ml));
    float lsum = 0.f;
    float4 acc[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) acc[i] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
    for (int s = 0; s < n_splits; ++s) {
        const float ms = __ldcg(ml + 2 * s * unit_ml), ls = __ldcg(ml + 2 * s * unit_ml + 1);
        const float wgt = (ms == -INFINITY) ? 0.f : ex2_approx(ms - Mx);
        lsum += wgt * ls;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float4 x = __ldcg(po + s * unit_o + (size_t)i * a.rows_pad);
            acc[i].x += wgt * x.x;
            acc[i].y += wgt * x.y;
            acc[i].z += wgt * x.z;
            acc[i].w += wgt * x.w;
        }
    }
    const float inv = lsum > 0.f ? 1.0f / lsum : 0.f;
    const int n = gr / a.G, g = gr % a.G;
    __nv_bfloat16 *dst = a.O + (((size_t)b * a.N + n) * a.Hq + hkv * a.G + g) * D + c4 * 4;
    uint4 q0, q1;
    q0.x = pack_bf16x2(acc[0].x * inv, acc[0].y * inv);
    q0.y = pack_bf16x2(acc[0].z * inv, acc[0].w * inv);
    q0.z = pack_bf16x2(acc[1].x * inv, acc[1].y * inv);
    q0.w = pack_bf16x2(acc[1].z * inv, acc[1].w * inv);
    q1.x = pack_bf16x2(acc[2].x * inv, acc[2].y * inv);
    q1.y = pack_bf16x2(acc[2].z * inv, acc[2].w * inv);
    q1.z = pack_bf16x2(acc[3].x * inv, acc[3].y * inv);
    q1.w = pack_bf16x2(acc[3].z * inv, acc[3].w * inv);
    reinterpret_cast<uint4 *>(dst)[0] = q0;
    reinterpret_cast<uint4 *>(dst)[1] = q1;
    if (a.lse && c4 == 0) a.lse[((size_t)b * a.N + n) * a.Hq + hkv * a.G + g] = (Mx + log2f(lsum)) * 0.6931471805599453f;
}

int launch_attn_merge_tc(const AttnArgs &a, int D, int items, cudaStream_t st) {
    const dim3 grid((unsigned)items, (unsigned)(a.Hkv * a.n_rb), (unsigned)(D / 32));
    if (D == 128)
        attn_merge_tc_kernel<128><<<grid, 256, 0, st>>>(a);
    else
        attn_merge_tc_kernel<64><<<grid, 256, 0, st>>>(a);
    SR_LAUNCH_CHECK();
    return SPECROLL_OK;
}

#ifdef SPECROLL_TRACE
extern "C" int specroll_debug_prof_read(unsigned long long *dst) {  // 5 roles x 12 counters; clears them
    if (cudaMemcpyFromSymbol(dst, g_prof, sizeof(unsigned long long) * 60) != cudaSuccess) return 4;
    unsigned long long z[60] = {0};
    return cudaMemcpyToSymbol(g_prof, z, sizeof(z)) == cudaSuccess ? 0 : 4;
}
extern "C" int specroll_debug_cta_read(unsigned long long *dst, unsigned int *n_launches) {  // [8][2][160] times in ns
    if (cudaMemcpyFromSymbol(n_launches, g_launch_n, 4) != cudaSuccess) return 4;
    return cudaMemcpyFromSymbol(dst, g_cta_ns, sizeof(unsigned long long) * 8 * 2 * 160) == cudaSuccess ? 0 : 4;
}
extern "C" int specroll_debug_trace_reset(void) {
    unsigned int z[4] = {0, 0, 0, 0};
    return cudaMemcpyToSymbol(g_trace_n, z, sizeof(z)) == cudaSuccess ? 0 : 4;
}
extern "C" int specroll_debug_trace_read(unsigned long long *dst, unsigned int *counts) {
    if (cudaMemcpyFromSymbol(counts, g_trace_n, 16) != cudaSuccess) return 4;
    return cudaMemcpyFromSymbol(dst, g_trace, sizeof(unsigned long long) * 4 * 8192) == cudaSuccess ? 0 : 4;
}
#endif

int launch_attn_tc(const AttnArgs &a, const TopoMask &mask, int D, long long T_kv, int32_t *status, cudaStream_t st) {
    if (a.nrb == 2) {
        if (D == 128) return launch_tc<128, 2>(a, mask, T_kv, status, st);
        return launch_tc<64, 2>(a, mask, T_kv, status, st);
    }
    if (D == 128) return launch_tc<128, 1>(a, mask, T_kv, status, st);
    return launch_tc<64, 1>(a, mask, T_kv, status, st);
}

}  // namespace specroll
