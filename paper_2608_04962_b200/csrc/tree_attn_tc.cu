// Tree-verification attention on the 5th-generation tensor cores (tcgen05 + TMEM), one layer.
//
// Same decomposition as the legacy kernel: for one (sequence, KV head) the N*G query rows form the
// M dimension; a CTA owns up to 128 of them and one chunk of the cache (split-KV), and streams
// 128-token K/V tiles.  Warp roles (192 threads, one CTA per SM):
//   warp 0    TMA producer: K and V tiles (3-D tensor maps over [token, kv head, D], 128-byte
//             swizzle), three stages, separate barriers for K and V
//   warp 1    allocates TMEM, issues  S = Q K^T  (M=128, N=128, A and B from shared memory) and
//             O += P V  (M=128, N=D, A = P from TMEM, B = V tile read MN-major from shared memory)
//   warps 2-5 softmax: thread = query row = TMEM lane, so row max / row sum need no shuffles;
//             P goes back to TMEM as packed bf16; the running output stays in TMEM and is rescaled
//             only when a row's maximum grows by more than 2^8 (rare), by the thread that owns the row
// S is double-buffered so the next tile's Q K^T overlaps this tile's softmax.
// TMEM columns: O [0,128)  S0 [128,256)  S1 [256,384)  P0 [384,448)  P1 [448,512).
#include <math.h>

#include "tc05.cuh"
#include "tree_attn.cuh"

namespace specroll {

namespace attc {
constexpr int BN = 128;
constexpr int THREADS = 192;
constexpr int STAGES = 3;
constexpr int TMEM_COLS = 512;
constexpr uint32_t O_COL = 0, S_COL = 128, P_COL = 384;  // S_COL + 128*buf, P_COL + 64*buf
constexpr float RESCALE_LOG2 = 8.0f;
constexpr int BOX_BYTES = BN * 128;  // 128 rows x 128 bytes (64 bf16) = one TMA box

template <int D>
struct Cfg {
    static constexpr int NBOX = D / 64;
    static constexpr int Q_BYTES = NBOX * BOX_BYTES;
    static constexpr int KV_BYTES = NBOX * BOX_BYTES;  // one K tile or one V tile
    static constexpr int STAGE_BYTES = 2 * KV_BYTES;
    static constexpr int USED = Q_BYTES + STAGES * STAGE_BYTES + 1024 + 256;
    // at least ~118 KB so that two CTAs can never share an SM (each allocates all of TMEM)
    static constexpr int SMEM = USED > 120832 ? USED : 120832;
};
}  // namespace attc

template <int D>
__global__ void __launch_bounds__(attc::THREADS, 1)
tree_attn_tc_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                    const __grid_constant__ CUtensorMap tmKt, const __grid_constant__ CUtensorMap tmVt, AttnArgs a,
                    TopoMask mask, int32_t *__restrict__ status) {
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
    auto s_full = [&](int b) { return bar0 + 8u * (3 * STAGES + b); };
    auto p_ready = [&](int b) { return bar0 + 8u * (3 * STAGES + 2 + b); };
    const uint32_t pv_done = bar0 + 8u * (3 * STAGES + 4);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(aligned + C::Q_BYTES + STAGES * C::STAGE_BYTES +
                                                       8 * (3 * STAGES + 5));
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // ---- which work item (same mapping as the legacy kernel)
    int bid = blockIdx.x;
    const int rb = bid % a.n_rb;
    bid /= a.n_rb;
    const int hkv = bid % a.Hkv;
    const int item = bid / a.Hkv;
    int lo = 0, hi = a.B;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (a.item_start[mid] <= item) lo = mid; else hi = mid;
    }
    const int b = lo;
    const int split = item - a.item_start[b];
    const int n_splits = a.item_start[b + 1] - a.item_start[b];
    const int kv0 = a.kv_indptr[b];
    const int L = a.kv_indptr[b + 1] - kv0;
    const int tiles_b = (L + BN - 1) / BN;
    const int tps = (tiles_b + n_splits - 1) / n_splits;
    const int t_lo = min(tiles_b, split * tps), t_hi = min(tiles_b, t_lo + tps);
    const bool has_tree = (split == n_splits - 1);
    const int n_it = (t_hi - t_lo) + (has_tree ? 1 : 0);
    const int row0 = rb * a.rows_per_block;
    const int N = a.N, G = a.G;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(k_full(s), 1);
            mbar_init(v_full(s), 1);
            mbar_init(kv_empty(s), 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(s_full(i), 1);
            mbar_init(p_ready(i), 128);
        }
        mbar_init(pv_done, 1);
        *abort_flag = 0;
        fence_mbar_init();
        prefetch_tmap(&tmK);
        prefetch_tmap(&tmV);
        prefetch_tmap(&tmKt);
        prefetch_tmap(&tmVt);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), TMEM_COLS);
        tmem_relinquish();
    }
    // ---- Q block -> shared memory in the K-major 128-byte-swizzled operand layout (rows beyond
    //      the block are zero).  Row r of the block is query row row0 + r = (node, head-in-group).
    {
        constexpr int CH = D / 8;  // 16-byte chunks per row
        for (int c = threadIdx.x; c < 128 * CH; c += THREADS) {
            const int r = c / CH, ch = c % CH;
            const int gr = row0 + r;
            uint4 v = make_uint4(0u, 0u, 0u, 0u);
            if (r < a.rows_per_block && gr < a.rows) {
                const int n = gr / G, g = gr % G;
                v = *reinterpret_cast<const uint4 *>(a.Q + (((size_t)b * N + n) * a.Hq + hkv * G + g) * D + ch * 8);
            }
            const int bx = ch >> 3, cc = ch & 7;
            *reinterpret_cast<uint4 *>(aligned + bx * BOX_BYTES + r * 128 + ((cc ^ (r & 7)) << 4)) = v;
        }
    }
    fence_proxy_async();  // generic-proxy writes above must be visible to the tensor core's reads
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            int issued[STAGES];
#pragma unroll
            for (int s = 0; s < STAGES; ++s) issued[s] = -1;
            bool ok = true;
            for (int it = 0; it < n_it; ++it) {
                const int s = it % STAGES;
                const uint32_t ph = (uint32_t)(it / STAGES) & 1u;
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
                for (int bx = 0; bx < C::NBOX; ++bx) tma_load_3d(ks + bx * BOX_BYTES, mk, bx * 64, hkv, tok, k_full(s));
                mbar_arrive_expect_tx(v_full(s), C::KV_BYTES);
#pragma unroll
                for (int bx = 0; bx < C::NBOX; ++bx) tma_load_3d(vs + bx * BOX_BYTES, mv, bx * 64, hkv, tok, v_full(s));
                issued[s] = (int)ph;
            }
            if (!ok) {
#pragma unroll
                for (int s = 0; s < STAGES; ++s)
                    if (issued[s] >= 0) {
                        const unsigned long long t0 = globaltimer_ns();
                        while (!(mbar_try_wait(k_full(s), (uint32_t)issued[s]) &&
                                 mbar_try_wait(v_full(s), (uint32_t)issued[s])) &&
                               globaltimer_ns() - t0 < 100000000ull) {
                        }
                    }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0 && n_it > 0) {
            constexpr uint32_t idesc_s = idesc_bf16(128, BN, false, false);
            constexpr uint32_t idesc_pv = idesc_bf16(128, D, false, true);  // V is read MN-major
            auto issue_s = [&](int j) {
                const uint32_t ks = kv_s + (j % STAGES) * C::STAGE_BYTES;
                const uint32_t d_t = tmem_base + S_COL + 128u * (uint32_t)(j & 1);
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint32_t off = (uint32_t)(kk >> 2) * BOX_BYTES + (uint32_t)(kk & 3) * 32u;
                    umma_ss(d_t, smem_desc_sw128(q_s + off, 1024, 0), smem_desc_sw128(ks + off, 1024, 0), idesc_s,
                            kk > 0 ? 1u : 0u);
                }
                umma_commit(s_full(j & 1));
            };
            bool ok = mbar_wait(k_full(0), 0u, abort_flag);
            if (ok) {
                tc_fence_after();
                issue_s(0);
            }
            for (int j = 0; j < n_it && ok; ++j) {
                if (j + 1 < n_it) {
                    if (!mbar_wait(k_full((j + 1) % STAGES), (uint32_t)((j + 1) / STAGES) & 1u, abort_flag)) break;
                    tc_fence_after();
                    issue_s(j + 1);
                }
                if (!mbar_wait(p_ready(j & 1), (uint32_t)(j >> 1) & 1u, abort_flag)) break;
                const int s = j % STAGES;
                if (!mbar_wait(v_full(s), (uint32_t)(j / STAGES) & 1u, abort_flag)) break;
                tc_fence_after();
                const uint32_t vs = kv_s + s * C::STAGE_BYTES + C::KV_BYTES;
                const uint32_t p_t = tmem_base + P_COL + 64u * (uint32_t)(j & 1);
#pragma unroll
                for (int kk = 0; kk < BN / 16; ++kk) {
                    // 16 tokens per step: 2048 bytes down the V tile, 8 packed columns along P
                    umma_ts(tmem_base + O_COL, p_t + 8u * kk, smem_desc_sw128(vs + kk * 2048, 1024, BOX_BYTES), idesc_pv,
                            (j > 0 || kk > 0) ? 1u : 0u);
                }
                umma_commit(kv_empty(s));
                umma_commit(pv_done);
            }
        }
    } else {
        // ------------------------------------------------------------------ softmax / output (warps 2..5)
        const int lg = warp & 3;
        const int row = lg * 32 + lane;
        const int gr = row0 + row;
        const bool row_ok = row < a.rows_per_block && gr < a.rows;
        const uint64_t anc = row_ok ? mask.anc[gr / G] : 0ull;
        const uint32_t t_lane = tmem_base + ((uint32_t)(lg * 32) << 16);
        const float sc = a.scale_log2;
        float m_used = -INFINITY, l = 0.f;
        bool ok = true;
        for (int j = 0; j < n_it; ++j) {
            const int buf = j & 1;
            ok = mbar_wait(s_full(buf), (uint32_t)(j >> 1) & 1u, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const bool tree = has_tree && (j == n_it - 1);
            const int limit = tree ? 64 : (L - (t_lo + j) * BN);  // columns >= limit are not in this sequence
            const uint32_t s_t = t_lane + S_COL + 128u * (uint32_t)buf;
            // pass 1: row maximum over the admissible columns
            float mx = -INFINITY;
#pragma unroll 1
            for (int c = 0; c < BN; c += 32) {
                uint32_t r[32];
                tmem_ld32(s_t + (uint32_t)c, r);
                tmem_ld_wait();
                if (tree) {
                    const uint32_t bits = (c < 64) ? (uint32_t)(anc >> c) : 0u;
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if ((bits >> i) & 1u) mx = fmaxf(mx, __uint_as_float(r[i]));
                } else if (c + 32 <= limit) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) mx = fmaxf(mx, __uint_as_float(r[i]));
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (c + i < limit) mx = fmaxf(mx, __uint_as_float(r[i]));
                }
            }
            const float mt = mx * sc;  // scale > 0; -inf stays -inf
            float alpha = 1.f;
            const bool need = mt > m_used + RESCALE_LOG2;  // also true on the first admissible tile
            if (need) {
                alpha = (m_used == -INFINITY) ? 0.f : ex2_approx(m_used - mt);
                m_used = mt;
                l *= alpha;
            }
            if (__any_sync(0xffffffffu, need) && j > 0) {
                // rows of this warp change their reference maximum: rescale their running outputs in TMEM.
                // The previous tile's P V must have landed first.
                ok = mbar_wait(pv_done, (uint32_t)(j - 1) & 1u, abort_flag);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
#pragma unroll 1
                for (int c = 0; c < D; c += 32) {
                    uint32_t r[32];
                    tmem_ld32(t_lane + O_COL + (uint32_t)c, r);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * alpha);
                    tmem_st32(t_lane + O_COL + (uint32_t)c, r);
                }
                tmem_st_wait();
            }
            const float mref = (m_used == -INFINITY) ? 0.f : m_used;
            // pass 2: p = 2^(s*scale - m), packed bf16 pairs into the P buffer
            float lsum = 0.f;
            const uint32_t p_t = t_lane + P_COL + 64u * (uint32_t)buf;
#pragma unroll 1
            for (int c = 0; c < BN; c += 32) {
                uint32_t r[32];
                tmem_ld32(s_t + (uint32_t)c, r);
                tmem_ld_wait();
                uint32_t bits;
                if (tree) bits = (c < 64) ? (uint32_t)(anc >> c) : 0u;
                else bits = (c + 32 <= limit) ? 0xffffffffu : ((c >= limit) ? 0u : ((1u << (limit - c)) - 1u));
                uint32_t pk[16];
#pragma unroll
                for (int i = 0; i < 32; i += 2) {
                    float p0 = ex2_approx(fmaf(__uint_as_float(r[i]), sc, -mref));
                    float p1 = ex2_approx(fmaf(__uint_as_float(r[i + 1]), sc, -mref));
                    p0 = ((bits >> i) & 1u) ? p0 : 0.f;
                    p1 = ((bits >> (i + 1)) & 1u) ? p1 : 0.f;
                    lsum += p0 + p1;
                    pk[i >> 1] = pack_bf16x2(p0, p1);
                }
                tmem_st16(p_t + (uint32_t)(c >> 1), pk);
            }
            tmem_st_wait();
            l += lsum;
            tc_fence_before();
            mbar_arrive(p_ready(buf));
        }
        // ---- output
        if (ok && n_it > 0) {
            ok = mbar_wait(pv_done, (uint32_t)(n_it - 1) & 1u, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
        }
        if (ok) {
            tc_fence_after();
            const int n = row_ok ? gr / G : 0, g = row_ok ? gr % G : 0;
            const bool direct = (n_splits == 1);
            const float inv = (direct && l > 0.f) ? 1.0f / l : (direct ? 0.f : 1.0f);
            __nv_bfloat16 *dst_o = a.O + (((size_t)b * N + n) * a.Hq + hkv * G + g) * D;
            const size_t prow = ((size_t)item * a.Hkv + hkv) * a.rows_pad + (row_ok ? gr : 0);
            float *dst_p = a.part_o + prow * D;
#pragma unroll 1
            for (int c = 0; c < D; c += 32) {
                uint32_t r[32];
                if (n_it > 0) {
                    tmem_ld32(t_lane + O_COL + (uint32_t)c, r);
                    tmem_ld_wait();
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) r[i] = 0u;
                }
                if (!row_ok) continue;
                if (direct) {
#pragma unroll
                    for (int i = 0; i < 32; i += 8) {
                        uint4 v;
                        v.x = pack_bf16x2(__uint_as_float(r[i]) * inv, __uint_as_float(r[i + 1]) * inv);
                        v.y = pack_bf16x2(__uint_as_float(r[i + 2]) * inv, __uint_as_float(r[i + 3]) * inv);
                        v.z = pack_bf16x2(__uint_as_float(r[i + 4]) * inv, __uint_as_float(r[i + 5]) * inv);
                        v.w = pack_bf16x2(__uint_as_float(r[i + 6]) * inv, __uint_as_float(r[i + 7]) * inv);
                        *reinterpret_cast<uint4 *>(dst_o + c + i) = v;
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 32; i += 4)
                        *reinterpret_cast<uint4 *>(dst_p + c + i) = make_uint4(r[i], r[i + 1], r[i + 2], r[i + 3]);
                }
            }
            if (row_ok) {
                if (direct) {
                    if (a.lse) a.lse[((size_t)b * N + n) * a.Hq + hkv * G + g] = (m_used + log2f(l)) * 0.6931471805599453f;
                } else {
                    a.part_ml[prow * 2] = m_used;
                    a.part_ml[prow * 2 + 1] = l;
                }
            }
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
static int launch_tc(const AttnArgs &a, const TopoMask &mask, int items, long long T_kv, int32_t *status,
                     cudaStream_t st) {
    using C = attc::Cfg<D>;
    CUtensorMap tmK, tmV, tmKt, tmVt;
    int rc;
    const uint64_t tree_rows = (uint64_t)a.B * a.N;
    // an empty cache still needs well-formed maps; they are never used for a load then
    const void *kc = T_kv > 0 ? (const void *)a.Kc : (const void *)a.Kt;
    const void *vc = T_kv > 0 ? (const void *)a.Vc : (const void *)a.Vt;
    const uint64_t cache_rows = T_kv > 0 ? (uint64_t)T_kv : tree_rows;
    if ((rc = make_tmap_3d_bf16(&tmK, kc, D, a.Hkv, cache_rows, attc::BN)) != SPECROLL_OK) return rc;
    if ((rc = make_tmap_3d_bf16(&tmV, vc, D, a.Hkv, cache_rows, attc::BN)) != SPECROLL_OK) return rc;
    if ((rc = make_tmap_3d_bf16(&tmKt, a.Kt, D, a.Hkv, tree_rows, attc::BN)) != SPECROLL_OK) return rc;
    if ((rc = make_tmap_3d_bf16(&tmVt, a.Vt, D, a.Hkv, tree_rows, attc::BN)) != SPECROLL_OK) return rc;
    static bool configured = false;
    if (!configured) {
        SR_CUDA_TRY(cudaFuncSetAttribute(tree_attn_tc_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM));
        configured = true;
    }
    const unsigned grid = (unsigned)items * a.Hkv * a.n_rb;
    tree_attn_tc_kernel<D><<<grid, attc::THREADS, C::SMEM, st>>>(tmK, tmV, tmKt, tmVt, a, mask, status);
    SR_LAUNCH_CHECK();
    return SPECROLL_OK;
}

int launch_attn_tc(const AttnArgs &a, const TopoMask &mask, int D, int items, long long T_kv, int32_t *status,
                   cudaStream_t st) {
    if (D == 128) return launch_tc<128>(a, mask, items, T_kv, status, st);
    return launch_tc<64>(a, mask, items, T_kv, status, st);
}

}  // namespace specroll
