// Tree-verification attention on the 5th-generation tensor cores (tcgen05 + TMEM), one layer.
//
// Same decomposition as the legacy kernel: for one (sequence, KV head) the N*G query rows form the
// M dimension; a CTA owns up to 128 of them and one chunk of the cache (split-KV), and streams
// 128-token K/V tiles.  Warp roles (320 threads, one CTA per SM):
//   warp 0     TMA producer: K and V tiles (3-D tensor maps over [token, kv head, D], 128-byte
//              swizzle), three stages, separate barriers for K and V
//   warp 1     allocates TMEM, issues  S = Q K^T  (M=128, N=128, A and B from shared memory) and
//              O += P V  (M=128, N=D, A = P from TMEM, B = V tile read MN-major from shared memory)
//   warps 2-5  softmax group 0: even tiles      } thread = query row = TMEM lane, so row max and
//   warps 6-9  softmax group 1: odd tiles       } row sum need no shuffles
// The two softmax groups are independent: each keeps its own running (reference max, sum) per row
// and its own output accumulator in TMEM, exactly like two KV splits, and they are merged at the
// end of the CTA.  P overwrites the first half of its S buffer in place (packed bf16).  An output
// accumulator is rescaled only when a row's maximum grows by more than 2^8 (rare), by the thread
// that owns the row.
// TMEM columns: O0 [0,128)  O1 [128,256)  S0/P0 [256,384)  S1/P1 [384,512).
#include <math.h>

#include "tc05.cuh"
#include "tree_attn.cuh"

namespace specroll {

namespace attc {
constexpr int BN = 128;
constexpr int THREADS = 320;
constexpr int STAGES = 3;
constexpr int TMEM_COLS = 512;
constexpr uint32_t O_COL = 0, S_COL = 256;  // O_COL + 128*group, S_COL + 128*group
constexpr float RESCALE_LOG2 = 8.0f;
constexpr int BOX_BYTES = BN * 128;  // 128 rows x 128 bytes (64 bf16) = one TMA box

template <int D>
struct Cfg {
    static constexpr int NBOX = D / 64;
    static constexpr int Q_BYTES = NBOX * BOX_BYTES;
    static constexpr int KV_BYTES = NBOX * BOX_BYTES;  // one K tile or one V tile
    static constexpr int STAGE_BYTES = 2 * KV_BYTES;
    static constexpr int N_BARS = 3 * STAGES + 6;
    static constexpr int EXTRA = 8 * N_BARS + 16 + 128 * 8;  // barriers, TMEM slot + abort flag, merge scratch
    static constexpr int USED = Q_BYTES + STAGES * STAGE_BYTES + 1024 + EXTRA;
    // at least ~118 KB so that two CTAs can never share an SM (each allocates all of TMEM)
    static constexpr int SMEM = USED > 120832 ? USED : 120832;
};

__device__ __forceinline__ void named_barrier_sync(int id, int nthreads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}
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
    auto s_full = [&](int g) { return bar0 + 8u * (3 * STAGES + g); };
    auto p_ready = [&](int g) { return bar0 + 8u * (3 * STAGES + 2 + g); };
    auto pv_done = [&](int g) { return bar0 + 8u * (3 * STAGES + 4 + g); };
    unsigned char *extra = aligned + C::Q_BYTES + STAGES * C::STAGE_BYTES + 8 * C::N_BARS;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(extra);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(extra + 4);
    float2 *merge_ml = reinterpret_cast<float2 *>(extra + 16);  // group 1's (max, sum) per row

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
            mbar_init(pv_done(i), 1);
        }
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
        // tcgen05.mma operations of one thread execute in issue order, which is what lets S of
        // tile j+2 overwrite the buffer whose P (tile j) the previous P V has read.
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
                const int g = j & 1;
                if (!mbar_wait(p_ready(g), (uint32_t)(j >> 1) & 1u, abort_flag)) break;
                const int s = j % STAGES;
                if (!mbar_wait(v_full(s), (uint32_t)(j / STAGES) & 1u, abort_flag)) break;
                tc_fence_after();
                const uint32_t vs = kv_s + s * C::STAGE_BYTES + C::KV_BYTES;
                const uint32_t p_t = tmem_base + S_COL + 128u * (uint32_t)g;
                const uint32_t o_t = tmem_base + O_COL + 128u * (uint32_t)g;
#pragma unroll
                for (int kk = 0; kk < BN / 16; ++kk) {
                    // 16 tokens per step: 2048 bytes down the V tile, 8 packed columns along P
                    umma_ts(o_t, p_t + 8u * kk, smem_desc_sw128(vs + kk * 2048, 1024, BOX_BYTES), idesc_pv,
                            (j > 1 || kk > 0) ? 1u : 0u);
                }
                umma_commit(kv_empty(s));
                umma_commit(pv_done(g));
            }
        }
    } else {
        // ------------------------------------------------------------------ softmax groups (warps 2..9)
        const int grp = (warp - 2) >> 2;  // 0: even tiles, 1: odd tiles
        const int lg = warp & 3;          // TMEM lane group of this warp
        const int row = lg * 32 + lane;
        const int gr = row0 + row;
        const bool row_ok = row < a.rows_per_block && gr < a.rows;
        const uint64_t anc = row_ok ? mask.anc[gr / G] : 0ull;
        const uint32_t t_lane = tmem_base + ((uint32_t)(lg * 32) << 16);
        const uint32_t s_t = t_lane + S_COL + 128u * (uint32_t)grp;
        const uint32_t o_t = t_lane + O_COL + 128u * (uint32_t)grp;
        const float sc = a.scale_log2;
        float m_used = -INFINITY, l = 0.f;
        bool ok = true;
        int n_mine = 0;
        for (int j = grp; j < n_it; j += 2, ++n_mine) {
            const int i = j >> 1;  // this group's i-th tile
            ok = mbar_wait(s_full(grp), (uint32_t)i & 1u, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const bool tree = has_tree && (j == n_it - 1);
            const int limit = tree ? 64 : (L - (t_lo + j) * BN);  // columns >= limit are outside the sequence
            const bool full = !tree && limit >= BN;
            uint32_t r[4][32];
#pragma unroll
            for (int c = 0; c < 4; ++c) tmem_ld32(s_t + 32u * c, r[c]);
            tmem_ld_wait();
            // admissible-column masks of the four 32-column groups
            uint32_t bits[4];
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                if (full) bits[c] = 0xffffffffu;
                else if (tree) bits[c] = (c < 2) ? (uint32_t)(anc >> (32 * c)) : 0u;
                else bits[c] = (32 * c + 32 <= limit) ? 0xffffffffu : ((32 * c >= limit) ? 0u : ((1u << (limit - 32 * c)) - 1u));
            }
            float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
            if (full) {
#pragma unroll
                for (int i2 = 0; i2 < 32; ++i2) {
                    mx0 = fmaxf(mx0, __uint_as_float(r[0][i2]));
                    mx1 = fmaxf(mx1, __uint_as_float(r[1][i2]));
                    mx2 = fmaxf(mx2, __uint_as_float(r[2][i2]));
                    mx3 = fmaxf(mx3, __uint_as_float(r[3][i2]));
                }
            } else {
#pragma unroll
                for (int i2 = 0; i2 < 32; ++i2) {
                    if ((bits[0] >> i2) & 1u) mx0 = fmaxf(mx0, __uint_as_float(r[0][i2]));
                    if ((bits[1] >> i2) & 1u) mx1 = fmaxf(mx1, __uint_as_float(r[1][i2]));
                    if ((bits[2] >> i2) & 1u) mx2 = fmaxf(mx2, __uint_as_float(r[2][i2]));
                    if ((bits[3] >> i2) & 1u) mx3 = fmaxf(mx3, __uint_as_float(r[3][i2]));
                }
            }
            const float mt = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * sc;  // scale > 0; -inf stays -inf
            float alpha = 1.f;
            const bool need = mt > m_used + RESCALE_LOG2;  // also true on the first admissible tile
            if (need) {
                alpha = (m_used == -INFINITY) ? 0.f : ex2_approx(m_used - mt);
                m_used = mt;
                l *= alpha;
            }
            if (__any_sync(0xffffffffu, need) && i > 0) {
                // rows of this warp change their reference maximum: rescale their running outputs in
                // TMEM.  This group's previous P V must have landed first.
                ok = mbar_wait(pv_done(grp), (uint32_t)(i - 1) & 1u, abort_flag);
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
            // p = 2^(s*scale - m), packed bf16 pairs written over the first 64 columns of the S buffer
            float ls0 = 0.f, ls1 = 0.f;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t pk[16];
#pragma unroll
                for (int i2 = 0; i2 < 32; i2 += 2) {
                    float p0 = ex2_approx(fmaf(__uint_as_float(r[c][i2]), sc, -mref));
                    float p1 = ex2_approx(fmaf(__uint_as_float(r[c][i2 + 1]), sc, -mref));
                    if (!full) {
                        p0 = ((bits[c] >> i2) & 1u) ? p0 : 0.f;
                        p1 = ((bits[c] >> (i2 + 1)) & 1u) ? p1 : 0.f;
                    }
                    ls0 += p0;
                    ls1 += p1;
                    pk[i2 >> 1] = pack_bf16x2(p0, p1);
                }
                tmem_st16(s_t + 16u * c, pk);
            }
            tmem_st_wait();
            l += ls0 + ls1;
            tc_fence_before();
            mbar_arrive(p_ready(grp));
        }
        // ---- wait for this group's last P V, then merge the two groups and write the output
        if (ok && n_mine > 0) {
            ok = mbar_wait(pv_done(grp), (uint32_t)(n_mine - 1) & 1u, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
        }
        if (grp == 1) merge_ml[row] = make_float2(m_used, (ok && n_mine > 0) ? l : 0.f);
        tc_fence_before();
        named_barrier_sync(1, 256);
        tc_fence_after();
        const bool all_ok = !*abort_flag;
        if (grp == 0 && all_ok) {
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
                        uint4 u;
                        u.x = pack_bf16x2(v[i2], v[i2 + 1]);
                        u.y = pack_bf16x2(v[i2 + 2], v[i2 + 3]);
                        u.z = pack_bf16x2(v[i2 + 4], v[i2 + 5]);
                        u.w = pack_bf16x2(v[i2 + 6], v[i2 + 7]);
                        *reinterpret_cast<uint4 *>(dst_o + c + i2) = u;
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
