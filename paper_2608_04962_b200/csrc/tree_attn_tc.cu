// Tree-verification attention on the 5th-generation tensor cores (tcgen05 + TMEM), one layer.
//
// Decomposition: for one (sequence, KV head) the N*G query rows form the M dimension, cut into row
// blocks of up to 128 rows (whole nodes).  A work unit is one row block times one chunk of the cache
// (split-KV), streamed as 128-token K/V tiles.  The row blocks of one (chunk, KV head) are neighbours
// in the work order: they run side by side on different SMs and the later ones find the tiles in L2.
// The kernel is persistent: one CTA per SM takes work units from a global counter, in an order
// prepared on the device (longest chunks first), and its pipeline runs across unit boundaries.
// Warp roles (480 threads):
//   warp 0     scheduler + TMA producer: fetches the next unit, publishes its descriptor in a
//              two-slot ring, loads the unit's Q block (3-D box over [node, head, D]; two buffers, so
//              the next unit's Q arrives while this unit is still being worked on) and the K and V
//              tiles (3-D boxes over [token, kv head, D], 128-byte swizzle) into ONE ring of five
//              stages, in the order they are consumed: K0 K1 K2 V0 K3 V1 K4 V2 ...
//   warp 1     allocates TMEM; one thread issues every  S = Q K^T  (M=128, N=128, operands from
//              shared memory) into one of three S buffers, up to three tiles ahead of the P V thread,
//              also across a unit boundary.
//   warp 2     one thread issues every  O += P V  (M=128, N=D, A = P from TMEM, B = V tile read
//              MN-major from shared memory).  Two issuing threads, because one thread that also sits
//              in the barrier waits left the tensor pipe idle more than half of the time.
//   warps 3-10 softmax, in one of two forms (template flag TEAMS, chosen by the number of row blocks):
//              one row block (HBM-bound): TWO threads per query row (warps w and w+4 own the same 32 TMEM
//              lanes and take columns 0-63 / 64-127 of each S tile); the pair exchanges one value per tile
//              through shared memory.  More row blocks (bound by the loop S -> softmax -> P V): two TEAMS of four warps, one thread
//              per row, team (t mod 2) takes tile t, so that one team's loads, stores and barrier round trips
//              run under the other team's exponentials; the row's reference maximum travels from team to
//              team through shared memory.  After the first tile(s) of a unit a tile takes one pass: the
//              exponentials against the reference as it stands, the tile's sum as the alarm for a reference
//              that has to move (then two passes from the S tile, which is still intact).  At the end of a
//              unit the threads leave their reference maxima and their shares of the row sums in the
//              workspace (one area per CTA) and go straight on to the next unit.
//   warps 11-14 output: one thread per query row takes the finished accumulator out of TMEM (after
//              the unit's last P V), normalises and stores it, or stores this chunk's fp32 partial.
// P is written back to TMEM over parts of S that its writer has already read (pairs: columns [0,32) by
// the first thread, [96,128) by the second; teams: columns [0,64)), as packed bf16.  The output accumulator is
// rescaled only when a row's reference maximum grows by more than 2^8 (rare).  Chunks of a split
// sequence leave fp32 partials in the workspace; the CTA that finishes a sequence's last chunk
// (atomic ticket, nobody waits) merges them, unless the plan leaves that to a kernel of its own.
// TMEM columns: O: [0, 128);  S/P buffer i: [128 + 128 i, +128).
// The kernel is launched as a programmatic dependent of the kernel before it in the stream: its CTAs are set up
// while that kernel's last CTAs finish, and (when the caller has said that cache and plan are older than that
// kernel) the loading thread fetches its first cache tiles before the wait that precedes every other access.
#include <math.h>

#include "tc05.cuh"
#include "tree_attn.cuh"

namespace specroll {

namespace attc {
constexpr int BN = 128;  // KV tokens per tile
constexpr int TMEM_COLS = 512;
constexpr float RESCALE_LOG2 = 8.0f;
constexpr int BOX_BYTES = BN * 128;  // 128 rows x 128 bytes (64 bf16)

struct UnitDesc {
    int32_t valid, b, hkv, rb, n_splits, kv0, L, t_lo, n_it, has_tree, item, item0;
};

template <int D, bool TEAMS>
struct Cfg {
    static constexpr int NBOX = D / 64;
    static constexpr int SB = 3;   // S buffers
    // K and V tiles share ONE ring, filled in the order they are consumed (K0 K1 K2 V0 K3 V1 K4 V2 ...: S runs
    // three tiles ahead of P V), so every load has the whole ring's depth to land; separate rings would need
    // three stages each for that, which does not fit beside two Q buffers.
    static constexpr int RS = 5;   // ring stages
    static constexpr int QS = 2;   // Q buffers (units)
    static constexpr int MMA_WARPS = 2;  // issuing threads (one lane of each)
    static constexpr int SOFTMAX_THREADS = 256, OUT_THREADS = 128;
    static constexpr int THREADS = 32 * (1 + MMA_WARPS) + SOFTMAX_THREADS + OUT_THREADS;
    static constexpr int Q_BYTES = NBOX * BOX_BYTES;   // the Q block of one unit
    static constexpr int KV_BYTES = NBOX * BOX_BYTES;  // one K tile or one V tile
    // barrier slots
    static constexpr int B_FULL = 0, B_EMPTY = B_FULL + RS, B_SFULL = B_EMPTY + RS, B_PREADY = B_SFULL + SB,
                         B_PVDONE = B_PREADY + SB, B_QFULL = B_PVDONE + SB, B_QFREE = B_QFULL + QS,
                         B_UFULL = B_QFREE + QS, B_UEMPTY = B_UFULL + 2, B_X = B_UEMPTY + 2, B_ALL = B_X + 4,
                         B_OFULL = B_ALL + 1, B_OFREE = B_OFULL + 1, B_HFULL = B_OFREE + 1, B_HFREE = B_HFULL + 1,
                         N_BARS = B_HFREE + 1;
    static constexpr int BAR_BYTES = (8 * N_BARS + 15) / 16 * 16;
    // exchange area: the rows' reference maxima as one softmax team leaves them for the other ([2][128] fp32), or
    // the partial row maxima of the pairs (per lane group [2 slots][2 halves][32 lanes] bf16)
    static constexpr int XCH_BYTES = 1024;
    static constexpr int EXTRA = BAR_BYTES + 16 + XCH_BYTES + 2 * 64;  // barriers, slot/abort/ticket, exchange, ring
    // hand-over from the softmax warps to the output warps (per row: each team's share of the sum and the
    // reference maximum it is relative to): in global memory, one area per CTA, because shared memory is full
    static constexpr int HAND_FLOATS = 4 * 128;
    // The operand tiles need 1024-byte alignment.  The dynamic shared window starts 1024-aligned on this
    // architecture (checked at run time: the kernel reports an error instead of running misaligned).
    static constexpr int USED = QS * Q_BYTES + RS * KV_BYTES + EXTRA;
    // at least ~118 KB so that two CTAs can never share an SM (each allocates all of TMEM)
    static constexpr int SMEM = USED > 120832 ? USED : 120832;
    static constexpr uint32_t O_COL = 0, S_COL = 128;
    static_assert(sizeof(UnitDesc) <= 64, "ring slot");
    static_assert(USED <= 232448, "shared memory budget");
    static_assert(S_COL + 128 * SB <= 512, "tensor memory columns");
};

// Rendezvous on an mbarrier (count = number of participants) with the same bounded wait as every other
// wait here: a hardware named barrier would hang if a participant had left through the abort path.
__device__ __forceinline__ bool group_sync(uint32_t bar, uint32_t &uses, volatile int *abort_flag) {
    mbar_arrive(bar);
    const bool ok = mbar_wait(bar, uses & 1u, abort_flag);
    ++uses;
    return ok;
}

// Two fp32 operations in one instruction (packed pairs in 64-bit registers): the softmax phase follows its
// instruction count, and the scale-and-shift before the exponential and the running sums are pairwise anyway.
__device__ __forceinline__ uint64_t pack_f32x2(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack_f32x2(uint64_t v, float &lo, float &hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma_f32x2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ uint64_t add_f32x2(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}

__device__ __forceinline__ unsigned short bf16_bits_rn(float x) {
    return __bfloat16_as_ushort(__float2bfloat16_rn(x));
}
__device__ __forceinline__ float bf16_bits_to_float(unsigned short b) { return __uint_as_float((uint32_t)b << 16); }
}  // namespace attc

template <int D, bool TEAMS>
__global__ void __launch_bounds__(attc::Cfg<D, TEAMS>::THREADS, 1)
tree_attn_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                    const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmKt,
                    const __grid_constant__ CUtensorMap tmVt, AttnArgs a, TopoMask mask,
                    int32_t *__restrict__ status) {
    using namespace attc;
    using C = Cfg<D, TEAMS>;
    constexpr int DH = D / 2;  // accumulator columns per thread of a pair (rescaling)
    constexpr int SB = C::SB, RS = C::RS, QS = C::QS, THREADS = C::THREADS;
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    unsigned char *aligned = smem_raw + (base - raw);
    const uint32_t q_s = base;
    const uint32_t r_s = base + QS * C::Q_BYTES;  // the K/V ring
    const uint32_t bar0 = r_s + RS * C::KV_BYTES;
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };
    unsigned char *extra = aligned + QS * C::Q_BYTES + RS * C::KV_BYTES + C::BAR_BYTES;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(extra);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(extra + 4);
    volatile int *tickets = reinterpret_cast<volatile int *>(extra + 8);
    unsigned char *xch_base = extra + 16;
    volatile UnitDesc *ring = reinterpret_cast<volatile UnitDesc *>(extra + 16 + C::XCH_BYTES);  // 2 slots of 64 bytes
    float *hand = a.hand + (size_t)blockIdx.x * C::HAND_FLOATS;  // [l of team 0 | l of team 1 | m of team 0 | m of team 1][128 rows]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int N = a.N, G = a.G;
    auto twait = [&](int, uint32_t b_, uint32_t par_) { return mbar_wait(b_, par_, abort_flag); };
    // Ring stage and phase of tile t's K and V (t counts tiles over all units of this CTA): in load order
    // K0 K1 K2 V0 K3 V1 K4 V2 ... K(t) is load number 2t - 2 (t for the first two) and V(t) load number 2t + 3.
    auto k_slot = [&](uint32_t t, int &st, uint32_t &ph) {
        const uint32_t pos = t < 2u ? t : 2u * t - 2u;
        st = (int)(pos % RS);
        ph = (pos / RS) & 1u;
    };
    auto v_slot = [&](uint32_t t, int &st, uint32_t &ph) {
        const uint32_t pos = 2u * t + 3u;
        st = (int)(pos % RS);
        ph = (pos / RS) & 1u;
    };
    auto stage_addr = [&](int st) { return r_s + (uint32_t)st * C::KV_BYTES; };
    if (base != raw) {  // uniform: the whole CTA leaves before touching anything
        if (threadIdx.x == 0) atomicExch(status, SPECROLL_ECUDA);
        return;
    }

    if (threadIdx.x == 0) {
        for (int i = 0; i < C::N_BARS; ++i) {
            uint32_t count = 1;
            // a tile's P comes from one team, or from all softmax threads
            if (i >= C::B_PREADY && i < C::B_PREADY + SB) count = TEAMS ? C::SOFTMAX_THREADS / 2 : C::SOFTMAX_THREADS;
            // a unit's descriptor is read by the MMA threads, the softmax threads and the output threads
            if (i >= C::B_UEMPTY && i < C::B_UEMPTY + 2) count = C::MMA_WARPS + C::SOFTMAX_THREADS + C::OUT_THREADS;
            // exchange barriers: per team (reference maxima), or per lane group (the pairs' partial maxima)
            if (i >= C::B_X && i < C::B_X + 4) count = TEAMS ? C::SOFTMAX_THREADS / 2 : 64;
            if (i == C::B_ALL || i == C::B_OFREE || i == C::B_HFREE) count = C::OUT_THREADS;
            if (i == C::B_HFULL) count = C::SOFTMAX_THREADS;
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
    // Launched as a programmatic dependent of the kernel before it in the stream, this CTA may have done all
    // of the above while that kernel was still finishing.  From here on it reads what earlier kernels wrote
    // (the plan, the counters the launch before cleared, Q and the tree's K/V), so it waits for them to be
    // complete.  The kernel after this one may be set up as early as its CTAs find room.
    // Exception: when the caller has said that the plan and the cache were complete before that kernel was
    // even launched, the loading thread fetches its first cache tiles right away and waits just before it
    // needs Q (below).
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const bool early = a.early_cache != 0;
    if (!(early && warp == 0)) asm volatile("griddepcontrol.wait;" ::: "memory");

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
                if (!twait(0, bar(C::B_EMPTY + s), ph ^ 1u)) return false;
                const uint32_t dst = stage_addr(s);
                mbar_arrive_expect_tx(bar(C::B_FULL + s), C::KV_BYTES);
#pragma unroll
                for (int bx = 0; bx < C::NBOX; ++bx)
                    tma_load_3d(dst + bx * BOX_BYTES, mv, bx * 64, hkv, tok, bar(C::B_FULL + s));
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
                // ---- decode: w = (chunk position in work order * Hkv + hkv) * n_rb + row block
                int t = w;
                const int rb = t % a.n_rb;
                t /= a.n_rb;
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
                // ---- the unit's Q block, into the buffer whose unit (two back) has had every S computed
                const int qb = (int)(u % QS);
                if (u >= (uint32_t)QS && !twait(2, bar(C::B_QFREE + qb), (u / QS - 1u) & 1u)) {
                    ok = false;
                    break;
                }
                auto load_q = [&]() {
                    mbar_arrive_expect_tx(bar(C::B_QFULL + qb), (uint32_t)(C::NBOX * 128 * a.rows_per_block));
#pragma unroll
                    for (int bx = 0; bx < C::NBOX; ++bx)
                        tma_load_3d(q_s + qb * C::Q_BYTES + bx * BOX_BYTES, &tmQ, bx * 64, hkv * G,
                                    b * N + rb * a.nodes_per_block, bar(C::B_QFULL + qb));
                };
                // Early cache loads: the first unit's first three cache tiles (their stages are free, nothing
                // here can block) go out before the kernel in front of this one has finished; Q and the tree's
                // K/V may be that kernel's output, so they follow the wait.
                bool q_pending = early && u == 0;
                auto settle = [&]() {
                    asm volatile("griddepcontrol.wait;" ::: "memory");
                    load_q();
                    q_pending = false;
                };
                if (!q_pending) load_q();
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
                    if (!twait(3, bar(C::B_EMPTY + s), kph ^ 1u)) {
                        ok = false;
                        break;
                    }
                    const bool tree = has_tree && (it == n_it - 1);
                    if (q_pending && (tree || it >= 3)) settle();
                    const int tok = tree ? b * N : (pt ? pg0 * BN : kv0 + (t_lo + it) * BN);
                    pg0 = pg1;
                    pg1 = pg2;
                    const CUtensorMap *mk = tree ? &tmKt : &tmK;
                    const uint32_t dst = stage_addr(s);
                    mbar_arrive_expect_tx(bar(C::B_FULL + s), C::KV_BYTES);
#pragma unroll
                    for (int bx = 0; bx < C::NBOX; ++bx)
                        tma_load_3d(dst + bx * BOX_BYTES, mk, bx * 64, hkv, tok, bar(C::B_FULL + s));
                    ++kt;
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
                if (q_pending) settle();
                // the unit's last V tiles go out now if their stages are already free; otherwise they wait
                // behind the next unit's Q and first K tiles (never block here)
                auto v_stage_free = [&]() {
                    int s;
                    uint32_t ph;
                    v_slot(vt, s, ph);
                    return mbar_test_wait(bar(C::B_EMPTY + s), ph ^ 1u);
                };
                while (ok && n_pend > 0 && v_stage_free()) {
                    ok = load_v(pv_map[0], pv_h[0], pv_tok[0]);
                    pv_map[0] = pv_map[1];
                    pv_h[0] = pv_h[1];
                    pv_tok[0] = pv_tok[1];
                    --n_pend;
                }
            }
            // (a thread that left the loop early has not waited yet; the counters touched at the end of the
            // kernel are cleared by the launch before this one)
            asm volatile("griddepcontrol.wait;" ::: "memory");
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
        // in a barrier wait: warp 1 issues every S = Q K^T, warp 2 every O += P V.
        if (lane == 0) {
            constexpr uint32_t idesc_s = idesc_bf16(128, BN, false, false);
            constexpr uint32_t idesc_pv = idesc_bf16(128, D, false, true);  // V is read MN-major
            // Descriptors are assembled from precomputed halves: the high word is constant, the low word is
            // the operand's shared-memory address / 16 (14 bits) plus, for V, LBO / 16 << 16.
            constexpr uint32_t DESC_HI = (1024u >> 4) | (1u << 14) | (2u << 29);  // SBO 1024, version, 128B swizzle
            constexpr uint32_t V_LBO = ((uint32_t)BOX_BYTES >> 4) << 16;
            constexpr uint32_t BOXU = (uint32_t)BOX_BYTES >> 4;
            auto desc = [](uint32_t lo) -> uint64_t { return ((uint64_t)DESC_HI << 32) | (uint64_t)lo; };
            bool ok = true;
            if (warp == 1) {
                // ---- S issuer: runs up to SB tiles ahead of the P V issuer, also across a unit boundary (the
                //      next unit's Q has its own buffer)
                uint32_t ts = 0;  // S tiles issued so far (all units)
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
                        if (!twait(2, bar(C::B_FULL + ks), kph)) {
                            ok = false;
                            break;
                        }
                        tc_fence_after();
                        const uint32_t k_lo = stage_addr(ks) >> 4;
                        const uint32_t d_t = tmem_base + C::S_COL + 128u * (uint32_t)sb;
#pragma unroll
                        for (int kk = 0; kk < D / 16; ++kk) {
                            const uint32_t off = (uint32_t)(kk >> 2) * BOXU + (uint32_t)(kk & 3) * 2u;
                            umma_ss(d_t, desc(q_lo + off), desc(k_lo + off), idesc_s, kk > 0 ? 1u : 0u);
                        }
                        umma_commit(bar(C::B_SFULL + sb));
                        umma_commit(bar(C::B_EMPTY + ks));  // the stage is free once this S has been computed
                    }
                    umma_commit(bar(C::B_QFREE + qb));  // every S of the unit computed: its Q buffer may be replaced
                }
            } else {
                // ---- P V issuer
                uint32_t tp = 0;  // P V tiles issued so far (all units)
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
                        if (!twait(4, bar(C::B_PREADY + sb), (tp / SB) & 1u) || !twait(5, bar(C::B_FULL + vs), vph)) {
                            ok = false;
                            break;
                        }
                        tc_fence_after();
                        const uint32_t v_lo = (stage_addr(vs) >> 4) | V_LBO;
                        const uint32_t p_t = tmem_base + C::S_COL + 128u * (uint32_t)sb;
#pragma unroll
                        for (int kk = 0; kk < BN / 16; ++kk) {
                            // 16 tokens per operation: 2048 bytes (128 address units) down the V tile, 8 packed columns
                            // of P.  Teams: P sits in columns [0,64) of the S buffer; pairs: tokens 0-63 in columns
                            // [0,32), tokens 64-127 in columns [96,128)
                            const uint32_t pcol = TEAMS ? 8u * kk : (kk < 4 ? 8u * kk : 64u + 8u * kk);
                            umma_ts(o_t, p_t + pcol, desc(v_lo + 128u * kk), idesc_pv, (kk > 0 || j > 0) ? 1u : 0u);
                        }
                        umma_commit(bar(C::B_EMPTY + vs));
                        umma_commit(bar(C::B_PVDONE + sb));
                    }
                    if (ok) umma_commit(bar(C::B_OFULL));  // the unit's accumulator is complete when this arrives
                }
            }
        }
    } else if (warp >= 1 + C::MMA_WARPS + C::SOFTMAX_THREADS / 32) {
        // ------------------------------------------------------------------ output (4 warps, one thread per query row)
        // Takes a finished unit's accumulator out of TMEM while the other warps are already in the next unit.
        const int lg = warp & 3;  // TMEM lane group of this warp
        const int row = lg * 32 + lane;
        const uint32_t t_lane = tmem_base + ((uint32_t)(lg * 32) << 16);
        const int tix = (int)threadIdx.x - (32 * (1 + C::MMA_WARPS) + C::SOFTMAX_THREADS);
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
            const int gr = rb * a.rows_per_block + row;
            const bool row_ok = row < a.rows_per_block && gr < a.rows;
            // ---- the row's sum (two shares) and reference maximum, left by the softmax threads at the end of the unit
            ok = twait(1, bar(C::B_HFULL), u & 1u);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            // each team's share of the sum is relative to the reference as that team last knew it
            const float l0 = __ldcg(hand + row), l1 = __ldcg(hand + 128 + row);
            const float m0 = __ldcg(hand + 256 + row), m1 = __ldcg(hand + 384 + row);
            const float m_used = fmaxf(m0, m1);
            const float lt = (m0 == -INFINITY ? 0.f : l0 * ex2_approx(m0 - m_used)) +
                             (m1 == -INFINITY ? 0.f : l1 * ex2_approx(m1 - m_used));
            mbar_arrive(bar(C::B_HFREE));
            // ---- the unit's last P V (operations complete in issue order, so it covers all)
            ok = twait(2, bar(C::B_OFULL), u & 1u);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const uint32_t o_t = t_lane + C::O_COL;
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
                if (c + 32 >= D) {  // everything has been read: the next unit's first P V may overwrite the accumulator
                    tc_fence_before();
                    mbar_arrive(bar(C::B_OFREE));
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
        }
    } else {
        if constexpr (TEAMS) {
            // ------------------------------------------------------------------ softmax (two teams of 4 warps)
            // Team (t & 1) takes tile t, one thread per query row, so that the fixed latencies of a tile (TMEM
            // loads and stores, barrier round trips) of one team run under the other team's exponentials.  The
            // row's reference maximum is common to both teams, each keeps its own share of the row sum.  After the
            // first two tiles of a unit a tile takes ONE pass: the exponentials are taken against the reference as
            // this team knows it, nothing is stored yet, and the tile's sum serves as the alarm (a score more than
            // 2^8 above the reference makes the sum exceed 2^8).  Then the thread looks at what the other team
            // left after the tile before: if that reference differs from its own, or the alarm went off (both
            // rare), the tile is done again from S with the two passes of a first tile, which can move the
            // reference and rescale the accumulator.  The result is the same as doing two passes every time.
            const int ws = warp - (1 + C::MMA_WARPS);
            const int team = ws >> 2;
            const int lg = warp & 3;  // TMEM lane group of this warp
            const int row = lg * 32 + lane;
            const uint32_t t_lane = tmem_base + ((uint32_t)(lg * 32) << 16);
            const uint32_t o_t = t_lane + C::O_COL;
            const float sc = a.scale_log2;
            volatile float *mref = reinterpret_cast<volatile float *>(xch_base);  // [2 slots][128 rows]
            uint32_t gt = 0;  // tiles so far (all units, both teams)
            bool ok = true;
            for (uint32_t u = 0; ok; ++u) {
                const int slot = (int)(u & 1u);
                ok = twait(0, bar(C::B_UFULL + slot), (u >> 1) & 1u);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                const int valid = ring[slot].valid, rb = ring[slot].rb, L = ring[slot].L, t_lo = ring[slot].t_lo;
                const int n_it = ring[slot].n_it, has_tree = ring[slot].has_tree;
                mbar_arrive(bar(C::B_UEMPTY + slot));
                if (!valid) break;
                const int gr = rb * a.rows_per_block + row;
                const bool row_ok = row < a.rows_per_block && gr < a.rows;
                const uint64_t anc = row_ok ? mask.anc[gr / G] : 0ull;
                float m_used = -INFINITY, l = 0.f;  // reference maximum as this thread knows it; this team's share of the sum
                for (int j = (int)((gt ^ (uint32_t)team) & 1u); j < n_it; j += 2) {
                    const uint32_t t = gt + (uint32_t)j;
                    const int sb = (int)(t % SB);
                    ok = twait(1, bar(C::B_SFULL + sb), (t / SB) & 1u);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t s_t = t_lane + C::S_COL + 128u * (uint32_t)sb;
                    const bool tree = has_tree && (j == n_it - 1);
                    // columns >= limit are outside the sequence (a tree tile has at most 64 rows of tree K/V)
                    const int limit = tree ? 64 : (L - (t_lo + j) * BN);
                    const bool full = !tree && limit >= BN;
                    // admissible columns of 32-column group c
                    auto bits_of = [&](int c) -> uint32_t {
                        if (full) return 0xffffffffu;
                        if (tree) return c == 0 ? (uint32_t)anc : (c == 1 ? (uint32_t)(anc >> 32) : 0u);
                        const int lim = limit - 32 * c;
                        return lim >= 32 ? 0xffffffffu : (lim <= 0 ? 0u : ((1u << lim) - 1u));
                    };
                    // p = 2^(s*scale - m) of one 32-column group as 16 packed bf16 pairs; adds the values to ls0 / ls1.
                    // (Two copies of the loop: with the mask test inside one loop the compiler evaluates it for every
                    // element of the full tiles too.)
                    float ls0 = 0.f, ls1 = 0.f;
                    auto exp_group = [&](const uint32_t(&src)[32], uint32_t bc, float mref_, uint32_t *pk) {
                        if (full) {
                            // in three sweeps (scale-and-shift, exponentials, sums and packing), so that no instruction
                            // waits for the exponential issued just before it
                            const uint64_t sc2 = pack_f32x2(sc, sc), nm2 = pack_f32x2(-mref_, -mref_);
                            float v[32];
#pragma unroll
                            for (int i2 = 0; i2 < 32; i2 += 2)
                                unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(src[i2]), __uint_as_float(src[i2 + 1])), sc2, nm2),
                                             v[i2], v[i2 + 1]);
#pragma unroll
                            for (int i2 = 0; i2 < 32; ++i2) v[i2] = ex2_approx(v[i2]);
                            uint64_t ls2 = pack_f32x2(ls0, ls1), ls3 = pack_f32x2(0.f, 0.f);
#pragma unroll
                            for (int i2 = 0; i2 < 32; i2 += 4) {
                                ls2 = add_f32x2(ls2, pack_f32x2(v[i2], v[i2 + 1]));
                                ls3 = add_f32x2(ls3, pack_f32x2(v[i2 + 2], v[i2 + 3]));
                                pk[i2 >> 1] = pack_bf16x2(v[i2], v[i2 + 1]);
                                pk[(i2 >> 1) + 1] = pack_bf16x2(v[i2 + 2], v[i2 + 3]);
                            }
                            unpack_f32x2(add_f32x2(ls2, ls3), ls0, ls1);
                        } else {
#pragma unroll
                            for (int i2 = 0; i2 < 32; i2 += 2) {
                                const bool b0 = (bc >> i2) & 1u, b1 = (bc >> (i2 + 1)) & 1u;
                                const float p0 = b0 ? ex2_approx(fmaf(__uint_as_float(src[i2]), sc, -mref_)) : 0.f;
                                const float p1 = b1 ? ex2_approx(fmaf(__uint_as_float(src[i2 + 1]), sc, -mref_)) : 0.f;
                                ls0 += p0;
                                ls1 += p1;
                                pk[i2 >> 1] = pack_bf16x2(p0, p1);
                            }
                        }
                    };
                    // The reference the other team left after tile t - 1.  Every tile waits for its predecessor's (also
                    // the first tile of a unit, which does not use the value), so a slot is never written twice
                    // between two reads.
                    float m_pub = -INFINITY;
                    auto predecessor = [&]() -> bool {
                        if (t == 0u) return true;
                        bool k_ = twait(4, bar(C::B_X + (int)((t - 1u) & 1u)), ((t - 1u) >> 1) & 1u);
                        k_ = __all_sync(0xffffffffu, k_);
                        if (k_ && j > 0) m_pub = mref[((t - 1u) & 1u) * 128u + row];
                        return k_;
                    };
                    uint32_t x[32];
                    bool done = false;
                    if (j >= 2) {
                        // ---- one pass against the reference as it stands; P stays in registers until the check below
                        uint32_t pk[64];
                        const float mref_ = (m_used == -INFINITY) ? 0.f : m_used;
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            tmem_ld32(s_t + 32u * (uint32_t)c, x);
                            tmem_ld_wait();
                            exp_group(x, bits_of(c), mref_, pk + 16 * c);
                        }
                        ok = predecessor();
                        if (!ok) break;
                        const bool bad = !(ls0 + ls1 <= 256.0f) || m_pub != m_used;
                        if (!__any_sync(0xffffffffu, bad)) {
                            // the reference stands: say so before storing P, the next tile's check waits for this
                            mref[(t & 1u) * 128u + row] = m_used;
                            mbar_arrive(bar(C::B_X + (int)(t & 1u)));
#pragma unroll
                            for (int c = 0; c < 4; ++c) {
                                uint32_t q[16];
#pragma unroll
                                for (int i2 = 0; i2 < 16; ++i2) q[i2] = pk[16 * c + i2];
                                tmem_st16(s_t + 16u * (uint32_t)c, q);
                            }
                            tmem_st_wait();
                            l += ls0 + ls1;
                            done = true;
                        }
                    }
                    if (!done) {
                        // ---- two passes.  First the row's maximum over the tile ...
                        ls0 = ls1 = 0.f;
                        float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            tmem_ld32(s_t + 32u * (uint32_t)c, x);
                            tmem_ld_wait();
                            const uint32_t bc = bits_of(c);
                            if (full) {
#pragma unroll
                                for (int i2 = 0; i2 < 32; i2 += 2) {
                                    mx0 = fmaxf(mx0, __uint_as_float(x[i2]));
                                    mx1 = fmaxf(mx1, __uint_as_float(x[i2 + 1]));
                                }
                            } else {
#pragma unroll
                                for (int i2 = 0; i2 < 32; ++i2)
                                    if ((bc >> i2) & 1u) mx0 = fmaxf(mx0, __uint_as_float(x[i2]));
                            }
                        }
                        const float mt = fmaxf(mx0, mx1) * sc;
                        // ... then the reference: the other team's after the tile before (this thread's share of the sum
                        // moves with it), raised if this tile's maximum is more than 2^8 above it
                        ok = predecessor();
                        if (!ok) break;
                        if (j > 0 && m_pub != m_used) {
                            l *= (m_used == -INFINITY) ? 0.f : ex2_approx(m_used - m_pub);
                            m_used = m_pub;
                        }
                        float alpha = 1.f;
                        const bool need = mt > m_used + RESCALE_LOG2;  // also true on the first admissible tile
                        if (need) {
                            alpha = (m_used == -INFINITY) ? 0.f : ex2_approx(m_used - mt);
                            m_used = mt;
                            l *= alpha;
                        }
                        mref[(t & 1u) * 128u + row] = m_used;  // known before the exponentials: the next tile need not wait for them
                        mbar_arrive(bar(C::B_X + (int)(t & 1u)));
                        if (__any_sync(0xffffffffu, need) && j > 0) {
                            // rows of this warp change their reference maximum: rescale their running outputs in TMEM.
                            // The previous tile's P V must have landed first (this tile's waits for the P written below).
                            ok = twait(2, bar(C::B_PVDONE + (int)((t - 1u) % SB)), ((t - 1u) / SB) & 1u);
                            ok = __all_sync(0xffffffffu, ok);
                            if (!ok) break;
                            tc_fence_after();
#pragma unroll 1
                            for (int c = 0; c < D; c += 32) {
                                tmem_ld32(o_t + (uint32_t)c, x);
                                tmem_ld_wait();
#pragma unroll
                                for (int i2 = 0; i2 < 32; ++i2) x[i2] = __float_as_uint(__uint_as_float(x[i2]) * alpha);
                                tmem_st32(o_t + (uint32_t)c, x);
                            }
                            tmem_st_wait();
                        }
                        // ... then p = 2^(s*scale - m) as packed bf16 pairs, group by group; 16 packed columns go over S
                        // columns that have been read already
                        const float mref_ = (m_used == -INFINITY) ? 0.f : m_used;
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            uint32_t q[16];
                            tmem_ld32(s_t + 32u * (uint32_t)c, x);
                            tmem_ld_wait();
                            exp_group(x, bits_of(c), mref_, q);
                            tmem_st16(s_t + 16u * (uint32_t)c, q);
                        }
                        tmem_st_wait();
                        l += ls0 + ls1;
                    }
                    tc_fence_before();
                    mbar_arrive(bar(C::B_PREADY + sb));
                }
                if (!ok) break;
                // ---- end of the unit: each team leaves its share of the sum and the reference it is relative to for
                //      the output warps and goes on with the next unit.  Those wait for the unit's last P V themselves.
                gt += (uint32_t)n_it;
                ok = twait(3, bar(C::B_HFREE), (u & 1u) ^ 1u);  // the values of the unit before have been taken
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                hand[team * 128 + row] = l;
                hand[256 + team * 128 + row] = m_used;
                mbar_arrive(bar(C::B_HFULL));
            }
        } else {
            // ------------------------------------------------------------------ softmax (8 warps, two threads per query row)
            const int ws = warp - (1 + C::MMA_WARPS);
            const int half = ws >> 2;  // which 64 of a tile's 128 columns, and which D/2 accumulator columns
            const int lg = warp & 3;   // TMEM lane group of this warp
            const int row = lg * 32 + lane;
            const uint32_t t_lane = tmem_base + ((uint32_t)(lg * 32) << 16);
            const uint32_t o_t = t_lane + C::O_COL + (uint32_t)(half * DH);
            const float sc = a.scale_log2;
            // exchange area of this lane group, 256 bytes, touched by the group's two warps only: the partial maxima
            // as bf16 [2 slots][2 halves][32 lanes]
            volatile unsigned short *xm = reinterpret_cast<volatile unsigned short *>(xch_base + lg * 256);
            uint32_t gt = 0;  // tiles processed so far (all units)
            uint32_t use_pair = 0;
            const uint32_t pair_bar = bar(C::B_X + lg);
            bool ok = true;
            for (uint32_t u = 0; ok; ++u) {
                const int slot = (int)(u & 1u);
                ok = twait(0, bar(C::B_UFULL + slot), (u >> 1) & 1u);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                const int valid = ring[slot].valid, rb = ring[slot].rb, L = ring[slot].L, t_lo = ring[slot].t_lo;
                const int n_it = ring[slot].n_it, has_tree = ring[slot].has_tree;
                mbar_arrive(bar(C::B_UEMPTY + slot));
                if (!valid) break;
                const int gr = rb * a.rows_per_block + row;
                const bool row_ok = row < a.rows_per_block && gr < a.rows;
                const uint64_t anc = row_ok ? mask.anc[gr / G] : 0ull;
                float m_used = -INFINITY, l = 0.f;  // l: this thread's share (its 64 columns of every tile)
                for (int j = 0; j < n_it; ++j) {
                    const uint32_t t = gt + (uint32_t)j;
                    const int sb = (int)(t % SB);
                    ok = twait(1, bar(C::B_SFULL + sb), (t / SB) & 1u);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    tc_fence_after();
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
                    // Exchanges the partial maximum with the thread that has the row's other 64 columns and returns the
                    // row's maximum (scaled).  It travels as bf16: any common reference close to the true maximum
                    // will do.  Two slots, alternating, so that a fast thread's next write cannot overtake a slow read.
                    auto row_max = [&](float &mt) -> bool {
                        const unsigned short mine = bf16_bits_rn(fmaxf(mx0, mx1));
                        const int px = (int)(use_pair & 1u) * 64;
                        xm[px + half * 32 + lane] = mine;
                        bool k_ = group_sync(pair_bar, use_pair, abort_flag);
                        k_ = __all_sync(0xffffffffu, k_);
                        mt = fmaxf(bf16_bits_to_float(mine), bf16_bits_to_float(xm[px + (half ^ 1) * 32 + lane])) * sc;
                        return k_;
                    };
                    // p = 2^(s*scale - m) of one 32-column group as 16 packed bf16 pairs; adds the values to ls0 / ls1
                    // and, if asked to, folds the scores into mx0 / mx1.  (Two copies of each loop: with the mask test
                    // inside one loop the compiler evaluates it for every element of the full tiles too.)
                    float ls0 = 0.f, ls1 = 0.f;
                    auto exp_group = [&](const uint32_t(&src)[32], uint32_t bc, float mref, bool with_max, uint32_t(&pk)[16]) {
                        if (full) {
                            const uint64_t sc2 = pack_f32x2(sc, sc), nm2 = pack_f32x2(-mref, -mref);
                            uint64_t ls2 = pack_f32x2(ls0, ls1);
#pragma unroll
                            for (int i2 = 0; i2 < 32; i2 += 2) {
                                const float s0 = __uint_as_float(src[i2]), s1 = __uint_as_float(src[i2 + 1]);
                                if (with_max) {
                                    mx0 = fmaxf(mx0, s0);
                                    mx1 = fmaxf(mx1, s1);
                                }
                                float t0, t1;
                                unpack_f32x2(fma_f32x2(pack_f32x2(s0, s1), sc2, nm2), t0, t1);
                                const float p0 = ex2_approx(t0), p1 = ex2_approx(t1);
                                ls2 = add_f32x2(ls2, pack_f32x2(p0, p1));
                                pk[i2 >> 1] = pack_bf16x2(p0, p1);
                            }
                            unpack_f32x2(ls2, ls0, ls1);
                        } else {
#pragma unroll
                            for (int i2 = 0; i2 < 32; i2 += 2) {
                                const float s0 = __uint_as_float(src[i2]), s1 = __uint_as_float(src[i2 + 1]);
                                const bool b0 = (bc >> i2) & 1u, b1 = (bc >> (i2 + 1)) & 1u;
                                if (with_max) {
                                    if (b0) mx0 = fmaxf(mx0, s0);
                                    if (b1) mx0 = fmaxf(mx0, s1);
                                }
                                const float p0 = b0 ? ex2_approx(fmaf(s0, sc, -mref)) : 0.f;
                                const float p1 = b1 ? ex2_approx(fmaf(s1, sc, -mref)) : 0.f;
                                ls0 += p0;
                                ls1 += p1;
                                pk[i2 >> 1] = pack_bf16x2(p0, p1);
                            }
                        }
                    };
                    // P is stored over S columns this thread has already read: [0,32) for the first thread of the pair,
                    // [96,128) for the second
                    const uint32_t p_col = s_t + 96u * half;
                    bool done = false;
                    if (j > 0) {
                        // ---- one pass with the reference maximum as it stands: the exponentials of the first group run
                        //      while the second group is still on its way from TMEM, and the row maximum (found on the
                        //      side) only has to confirm that the reference may stay; if it may not, for some row of
                        //      this warp, the tile is done again below with the two passes of a first tile.
                        uint32_t pk0[16], pk1[16];
                        const float mref = (m_used == -INFINITY) ? 0.f : m_used;
                        tmem_ld32(s_t + 64u * half, r0);
                        tmem_ld_wait();
                        tmem_ld32(s_t + 64u * half + 32u, r1);
                        exp_group(r0, bits0, mref, false, pk0);
                        tmem_ld_wait();
                        exp_group(r1, bits1, mref, false, pk1);
                        // A score above the reference by more than 2^8 makes its p, and so the sum, exceed 2^8: the
                        // sum (which is there anyway) serves as the alarm; the two-pass path then decides exactly.
                        mx0 = mx1 = (ls0 + ls1 <= 256.0f) ? -INFINITY : INFINITY;
                        float mt;
                        ok = row_max(mt);
                        if (!ok) break;
                        if (!__any_sync(0xffffffffu, mt > m_used + RESCALE_LOG2)) {
                            tmem_st16(p_col, pk0);
                            tmem_st16(p_col + 16u, pk1);
                            tmem_st_wait();
                            l += ls0 + ls1;
                            done = true;
                        }
                    }
                    if (!done) {
                        // ---- pass 1: maximum of this thread's 64 columns
                        mx0 = mx1 = -INFINITY;
                        ls0 = ls1 = 0.f;
                        tmem_ld32(s_t + 64u * half, r0);
                        tmem_ld32(s_t + 64u * half + 32u, r1);
                        tmem_ld_wait();
                        max_group(r0, bits0);
                        max_group(r1, bits1);
                        float mt;
                        ok = row_max(mt);
                        if (!ok) break;
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
                            ok = twait(2, bar(C::B_PVDONE + (int)((t - 1u) % SB)), ((t - 1u) / SB) & 1u);
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
                        // ---- pass 2: p = 2^(s*scale - m) as packed bf16 pairs, 16 packed columns per 32-column group
                        const float mref = (m_used == -INFINITY) ? 0.f : m_used;
                        uint32_t pk[16];
                        exp_group(r0, bits0, mref, false, pk);
                        tmem_st16(p_col, pk);
                        exp_group(r1, bits1, mref, false, pk);
                        tmem_st16(p_col + 16u, pk);
                        tmem_st_wait();
                        l += ls0 + ls1;
                    }
                    tc_fence_before();
                    mbar_arrive(bar(C::B_PREADY + sb));
                }
                if (!ok) break;
                // ---- hand the row's reference maximum and this thread's share of its sum to the output warps
                //      and go on with the next unit; they wait for the unit's last P V themselves
                gt += (uint32_t)n_it;
                ok = twait(3, bar(C::B_HFREE), (u & 1u) ^ 1u);  // the values of the unit before have been taken
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                hand[half * 128 + row] = l;
                hand[256 + half * 128 + row] = m_used;  // the same value from both threads of the pair
                mbar_arrive(bar(C::B_HFULL));
            }
        }
    }

    // ------------------------------------------------------------------ teardown
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
        }
    }
}

template <int D, bool TEAMS>
static int launch_tc(const AttnArgs &a, const TopoMask &mask, long long T_kv, int32_t *status, cudaStream_t st) {
    using C = attc::Cfg<D, TEAMS>;
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
    int n_sm = 0;
    if ((rc = device_setup(reinterpret_cast<const void *>(tree_attn_tc_kernel<D, TEAMS>), C::SMEM, &n_sm)) != SPECROLL_OK) return rc;
    const int ctas = n_sm < ATTN_HAND_CTAS ? n_sm : ATTN_HAND_CTAS;  // every CTA has a hand-over area of its own
    const unsigned grid = (unsigned)(a.total_work < ctas ? a.total_work : ctas);
    // Programmatic stream serialization: the CTAs may be set up (barriers, tensor memory, zeroed Q buffers) while
    // the kernel before this one in the stream is still running its last CTAs; the kernel itself waits for
    // that kernel's completion before it reads anything (griddepcontrol.wait).
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(C::THREADS);
    cfg.dynamicSmemBytes = C::SMEM;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = a.no_pdl ? 0 : 1;
    SR_CUDA_TRY(cudaLaunchKernelEx(&cfg, tree_attn_tc_kernel<D, TEAMS>, tmQ, tmK, tmV, tmKt, tmVt, a, mask, status));
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


int launch_attn_tc(const AttnArgs &a, const TopoMask &mask, int D, long long T_kv, int32_t *status, cudaStream_t st) {
    // One row block per (sequence, KV head): the kernel is bound by HBM and the softmax with two threads per row
    // is (slightly) the better one; more blocks: bound by the softmax, where the two alternating teams are faster.
    const bool teams = a.n_rb > 1;
    if (D == 128) return teams ? launch_tc<128, true>(a, mask, T_kv, status, st) : launch_tc<128, false>(a, mask, T_kv, status, st);
    return teams ? launch_tc<64, true>(a, mask, T_kv, status, st) : launch_tc<64, false>(a, mask, T_kv, status, st);
}

}  // namespace specroll
