// Tree-verification attention, one layer: every tree node of every sequence attends to the
// sequence's KV cache plus its own ancestors' tree rows.
//
// Work decomposition.  For one (sequence, KV head) all N*G query rows (G = Hq/Hkv query heads per
// KV head) share the same keys and values, so they form the M dimension of one skinny GEMM pair:
// each cached K/V element is read once for all of them.  A CTA owns a block of <= 128 of those
// rows (one warp per 16 rows) and a contiguous chunk of the cache ("split-KV"); chunks are
// sized on the host from the KV lengths so that long sequences are spread over many CTAs.
// The tree's own K/V rows form one extra 64-token tile masked by the per-node ancestor bitmask;
// it is processed by the CTA that owns the last chunk.  A sequence that needs a single chunk
// writes its output directly; otherwise fp32 partials (O, running max, running sum) go to the
// workspace and a second kernel combines them.
//
// Legacy tensor-core path: mma.sync m16n8k16 bf16 with fp32 accumulation, cp.async staging,
// warp-shuffle online softmax in the log2 domain.
#include <math.h>

#include "common.cuh"
#include <string.h>

#include <algorithm>
#include <functional>
#include <mutex>
#include <queue>
#include <vector>

#include "tree_attn.cuh"

namespace specroll {

SR_CHECK_TU()

constexpr int AT_BN = 64;       // KV tokens per tile
constexpr int AT_STAGES = 3;
constexpr int AT_MAX_WARPS = 8; // 128 query rows per CTA
constexpr float LOG2E = 1.4426950408889634f;

constexpr int PREP_THREADS = 1024;
constexpr int PREP_MAX_B = 4096;  // sequences the prep kernel can order (4 per thread)

// Exclusive scan of n <= 4 * PREP_THREADS ints held in shared memory, in place; returns the total.
__device__ int block_exclusive_scan(int *data, int n, int *warp_tot) {
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    int v[4], s = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int idx = 4 * t + i;
        v[i] = idx < n ? data[idx] : 0;
        s += v[i];
    }
    int incl = s;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int x = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += x;
    }
    if (lane == 31) warp_tot[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        int w = warp_tot[lane];
        int wi = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int x = __shfl_up_sync(0xffffffffu, wi, o);
            if (lane >= o) wi += x;
        }
        warp_tot[lane] = wi - w;  // exclusive prefix of the warp totals
        if (lane == 31) warp_tot[32] = wi;
    }
    __syncthreads();
    int run = warp_tot[warp] + incl - s;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int idx = 4 * t + i;
        if (idx < n) data[idx] = run;
        run += v[i];
    }
    const int total = warp_tot[32];
    __syncthreads();
    return total;
}

// One block.  Per sequence: number of chunks ns = max(1, ceil(tiles / chunk_tiles)).
//   item_start[b]   exclusive prefix of ns in sequence order            (both kernels)
//   seq_at_rank[r], sorted_start[r]   work order: sequences by decreasing tiles-per-chunk, and the
//                   exclusive prefix of ns in that order                  (tcgen05 kernel, B <= PREP_MAX_B)
// Also clears the status word and the scheduling counters.
__global__ void __launch_bounds__(PREP_THREADS)
attn_prep_kernel(const int32_t *__restrict__ kv_indptr, const int32_t *__restrict__ kv_len,
                 const int32_t *__restrict__ page_indptr, int B, int chunk_tiles, int tile_tokens,
                 int32_t *__restrict__ item_start, int32_t *__restrict__ sorted_start,
                 int32_t *__restrict__ seq_at_rank, int32_t *__restrict__ unit_tab, int32_t *__restrict__ status,
                 int32_t *__restrict__ counters, int n_counters) {
    __shared__ unsigned short sh_ns[PREP_MAX_B];  // chunk counts fit 16 bits (checked on the host)
    __shared__ int sh_cost[PREP_MAX_B];
    __shared__ int sh_tmp[PREP_MAX_B];
    __shared__ int warp_tot[33];
    const int t = threadIdx.x;
    if (t == 0) *status = 0;
    for (int i = t; i < n_counters; i += PREP_THREADS) counters[i] = 0;
    if (B > PREP_MAX_B) {
        // too many sequences to order here: sequence-order prefix only (legacy kernel)
        if (t == 0) {
            int acc = 0;
            for (int b = 0; b < B; ++b) {
                item_start[b] = acc;
                const int L = kv_len ? kv_len[b] : kv_indptr[b + 1] - kv_indptr[b];
                const int tiles = (L + tile_tokens - 1) / tile_tokens;
                const int ns = (tiles + chunk_tiles - 1) / chunk_tiles;
                acc += ns < 1 ? 1 : ns;
            }
            item_start[B] = acc;
        }
        return;
    }
    for (int b = t; b < B; b += PREP_THREADS) {
        int L = kv_len ? kv_len[b] : kv_indptr[b + 1] - kv_indptr[b];
#ifdef SPECROLL_CHECK
        if (L < 0) {  // the device copy of the lengths disagrees with any host copy the planner can have seen
            SR_CHECK_FAIL(b);
            L = 0;
        }
#endif
        const int tiles = (L + tile_tokens - 1) / tile_tokens;
        int ns = (tiles + chunk_tiles - 1) / chunk_tiles;
        if (ns < 1) ns = 1;
        sh_ns[b] = (unsigned short)ns;
        sh_cost[b] = (tiles + ns - 1) / ns;  // tiles per chunk
        sh_tmp[b] = ns;
    }
    __syncthreads();
    const int total = block_exclusive_scan(sh_tmp, B, warp_tot);
    for (int b = t; b < B; b += PREP_THREADS) item_start[b] = sh_tmp[b];
    if (t == 0) item_start[B] = total;
    if (!sorted_start) return;
    __syncthreads();
    // rank by counting: position of b in the order (cost descending, index ascending)
    for (int b = t; b < B; b += PREP_THREADS) {
        const int c = sh_cost[b];
        int r = 0;
        for (int o = 0; o < B; ++o) {
            const int co = sh_cost[o];
            r += (co > c) || (co == c && o < b);
        }
        seq_at_rank[r] = b;
        sh_tmp[r] = (int)sh_ns[b];
    }
    __syncthreads();
    const int total2 = block_exclusive_scan(sh_tmp, B, warp_tot);
    for (int r = t; r < B; r += PREP_THREADS) sorted_start[r] = sh_tmp[r];
    if (t == 0) sorted_start[B] = total2;
    // per-chunk table in work order, so that the scheduler decodes a work unit with one 32-byte load
    if (unit_tab) {
        __syncthreads();
        for (int b = t; b < B; b += PREP_THREADS) {
            // recompute this sequence's rank (same rule as above) to find where its chunks go
            const int c = sh_cost[b];
            int r = 0;
            for (int o = 0; o < B; ++o) {
                const int co = sh_cost[o];
                r += (co > c) || (co == c && o < b);
            }
            const int ns = (int)sh_ns[b];
            // contiguous cache: first token and length; paged cache: first slot of the page table and length
            const int kv0 = kv_len ? page_indptr[b] : kv_indptr[b];
            const int L = kv_len ? kv_len[b] : kv_indptr[b + 1] - kv0;
            const int first = item_start[b];  // written by this block; visible after the barriers above
            int4 *dst = reinterpret_cast<int4 *>(unit_tab) + 2 * (size_t)sh_tmp[r];
            for (int s = 0; s < ns; ++s) {
                dst[2 * s] = make_int4(b, s, ns, first);
                dst[2 * s + 1] = make_int4(kv0, L, 0, 0);
            }
        }
    }
}

template <int D>
struct AttnSmem {
    static constexpr int ROW_BYTES = D * 2;
    static constexpr int CHUNKS = D / 8;  // 16-byte chunks per row
    static constexpr int Q_BYTES = AT_MAX_WARPS * 16 * ROW_BYTES;
    static constexpr int KV_BYTES = AT_BN * ROW_BYTES;
    static constexpr int STAGE_BYTES = 2 * KV_BYTES;
    static constexpr int TOTAL = Q_BYTES + AT_STAGES * STAGE_BYTES;
    static __device__ __forceinline__ uint32_t off(int row, int chunk) {
        return row * ROW_BYTES + ((chunk ^ (row & 7)) << 4);
    }
};

template <int D>
__global__ void __launch_bounds__(AT_MAX_WARPS * 32, 1)
tree_attn_kernel(AttnArgs a, TopoMask mask) {
    using S = AttnSmem<D>;
    extern __shared__ __align__(128) unsigned char smem[];
    const uint32_t sq = smem_u32(smem), skv = sq + S::Q_BYTES;
    const int nthreads = blockDim.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // ---- which work item
    int bid = blockIdx.x;
    const int rb = bid % a.n_rb;
    bid /= a.n_rb;
    const int hkv = bid % a.Hkv;
    const int item = bid / a.Hkv;
    int lo = 0, hi = a.B;  // largest b with item_start[b] <= item
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (a.item_start[mid] <= item) lo = mid; else hi = mid;
    }
    const int b = lo;
    const int split = item - a.item_start[b];
    const int n_splits = a.item_start[b + 1] - a.item_start[b];
    const int kv0 = a.kv_indptr[b];
    const int L = a.kv_indptr[b + 1] - kv0;
    const int tiles_b = (L + AT_BN - 1) / AT_BN;
    const int tps = (tiles_b + n_splits - 1) / n_splits;
    const int t_lo = min(tiles_b, split * tps), t_hi = min(tiles_b, t_lo + tps);
    const bool has_tree = (split == n_splits - 1);
    const int n_it = (t_hi - t_lo) + (has_tree ? 1 : 0);

    const int row0 = rb * a.rows_per_block;  // first query row (n*G+g) of this CTA
    const int N = a.N, G = a.G;

    // ---- Q tile -> smem (zero rows beyond `rows`)
    {
        const int nrow = a.rows_per_block;
        for (int c = threadIdx.x; c < nrow * S::CHUNKS; c += nthreads) {
            const int r = c / S::CHUNKS, ch = c % S::CHUNKS;
            const int gr = row0 + r;
            const bool ok = gr < a.rows;
            const int n = ok ? gr / G : 0, g = ok ? gr % G : 0;
            const __nv_bfloat16 *src = a.Q + (((size_t)b * N + n) * a.Hq + hkv * G + g) * D + ch * 8;
            cp_async16(sq + S::off(r, ch), src, ok);
        }
        cp_async_commit();
    }

    auto load_tile = [&](int it, int stage) {
        const uint32_t sk = skv + stage * S::STAGE_BYTES, sv = sk + S::KV_BYTES;
        const bool tree = has_tree && (it == n_it - 1);
        for (int c = threadIdx.x; c < AT_BN * S::CHUNKS; c += nthreads) {
            const int r = c / S::CHUNKS, ch = c % S::CHUNKS;
            const __nv_bfloat16 *ksrc, *vsrc;
            bool ok;
            if (!tree) {
                const int tok = (t_lo + it) * AT_BN + r;
                ok = tok < L;
                const size_t o = ((size_t)(kv0 + (ok ? tok : 0)) * a.Hkv + hkv) * D + ch * 8;
                ksrc = a.Kc + o;
                vsrc = a.Vc + o;
            } else {
                ok = r < N;
                const size_t o = (((size_t)b * N + (ok ? r : 0)) * a.Hkv + hkv) * D + ch * 8;
                ksrc = a.Kt + o;
                vsrc = a.Vt + o;
            }
            cp_async16(sk + S::off(r, ch), ksrc, ok);
            cp_async16(sv + S::off(r, ch), vsrc, ok);
        }
    };

#pragma unroll
    for (int s = 0; s < AT_STAGES - 1; ++s) {
        if (s < n_it) load_tile(s, s);
        cp_async_commit();
    }

    // ---- per-thread state: rows g0 = lane/4 and g0+8 of this warp's 16-row slab
    const int wrow = warp * 16;
    const int r_lo = row0 + wrow + (lane >> 2), r_hi = r_lo + 8;
    uint64_t anc_lo = 0, anc_hi = 0;
    if (r_lo < a.rows) anc_lo = mask.anc[r_lo / G];
    if (r_hi < a.rows) anc_hi = mask.anc[r_hi / G];

    uint32_t qf[D / 16][4];
    float oacc[D / 8][4];
#pragma unroll
    for (int j = 0; j < D / 8; ++j)
#pragma unroll
        for (int t = 0; t < 4; ++t) oacc[j][t] = 0.f;
    float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;

    for (int it = 0; it < n_it; ++it) {
        cp_async_wait<AT_STAGES - 2>();
        __syncthreads();
        if (it == 0) {
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk)
                ldmatrix_x4(qf[kk], sq + S::off(wrow + (lane & 15), kk * 2 + (lane >> 4)));
        }
        {
            const int nx = it + AT_STAGES - 1;
            if (nx < n_it) load_tile(nx, nx % AT_STAGES);
            cp_async_commit();
        }
        const uint32_t sk = skv + (it % AT_STAGES) * S::STAGE_BYTES, sv = sk + S::KV_BYTES;
        const bool tree = has_tree && (it == n_it - 1);

        // ---- S = Q K^T   (16 x 64 per warp)
        float sacc[AT_BN / 8][4];
#pragma unroll
        for (int j = 0; j < AT_BN / 8; ++j)
#pragma unroll
            for (int t = 0; t < 4; ++t) sacc[j][t] = 0.f;
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
#pragma unroll
            for (int jp = 0; jp < AT_BN / 16; ++jp) {
                uint32_t r[4];
                const int row = jp * 16 + (lane & 7) + ((lane >> 4) << 3), ch = kk * 2 + ((lane >> 3) & 1);
                ldmatrix_x4(r, sk + S::off(row, ch));
                mma_bf16_16816(sacc[2 * jp], qf[kk], r[0], r[1]);
                mma_bf16_16816(sacc[2 * jp + 1], qf[kk], r[2], r[3]);
            }
        }

        // ---- scale, mask, online softmax (log2 domain)
        const int tok0 = (t_lo + it) * AT_BN;
        float mx_lo = -INFINITY, mx_hi = -INFINITY;
#pragma unroll
        for (int j = 0; j < AT_BN / 8; ++j) {
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int col = j * 8 + (lane & 3) * 2 + e;
                bool ok_lo, ok_hi;
                if (tree) {
                    ok_lo = (anc_lo >> col) & 1;
                    ok_hi = (anc_hi >> col) & 1;
                } else {
                    ok_lo = ok_hi = (tok0 + col) < L;
                }
                const float v_lo = ok_lo ? sacc[j][e] * a.scale_log2 : -INFINITY;
                const float v_hi = ok_hi ? sacc[j][2 + e] * a.scale_log2 : -INFINITY;
                sacc[j][e] = v_lo;
                sacc[j][2 + e] = v_hi;
                mx_lo = fmaxf(mx_lo, v_lo);
                mx_hi = fmaxf(mx_hi, v_hi);
            }
        }
        mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
        mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
        mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
        mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
        const float mn_lo = fmaxf(m_lo, mx_lo), mn_hi = fmaxf(m_hi, mx_hi);
        const float ms_lo = (mn_lo == -INFINITY) ? 0.f : mn_lo, ms_hi = (mn_hi == -INFINITY) ? 0.f : mn_hi;
        const float al_lo = ex2_approx(m_lo - ms_lo), al_hi = ex2_approx(m_hi - ms_hi);
        m_lo = mn_lo;
        m_hi = mn_hi;
        float ps_lo = 0.f, ps_hi = 0.f;
        uint32_t pf[AT_BN / 16][4];
#pragma unroll
        for (int j = 0; j < AT_BN / 8; ++j) {
            const float p0 = ex2_approx(sacc[j][0] - ms_lo), p1 = ex2_approx(sacc[j][1] - ms_lo);
            const float p2 = ex2_approx(sacc[j][2] - ms_hi), p3 = ex2_approx(sacc[j][3] - ms_hi);
            ps_lo += p0 + p1;
            ps_hi += p2 + p3;
            pf[j >> 1][(j & 1) * 2] = pack_bf16x2(p0, p1);
            pf[j >> 1][(j & 1) * 2 + 1] = pack_bf16x2(p2, p3);
        }
        l_lo = l_lo * al_lo + ps_lo;
        l_hi = l_hi * al_hi + ps_hi;
#pragma unroll
        for (int j = 0; j < D / 8; ++j) {
            oacc[j][0] *= al_lo;
            oacc[j][1] *= al_lo;
            oacc[j][2] *= al_hi;
            oacc[j][3] *= al_hi;
        }

        // ---- O += P V
#pragma unroll
        for (int kk = 0; kk < AT_BN / 16; ++kk) {
#pragma unroll
            for (int dp = 0; dp < D / 16; ++dp) {
                uint32_t r[4];
                const int row = kk * 16 + (lane & 7) + (((lane >> 3) & 1) << 3), ch = dp * 2 + (lane >> 4);
                ldmatrix_x4_trans(r, sv + S::off(row, ch));
                mma_bf16_16816(oacc[2 * dp], pf[kk], r[0], r[1]);
                mma_bf16_16816(oacc[2 * dp + 1], pf[kk], r[2], r[3]);
            }
        }
    }
    cp_async_wait<0>();

    // ---- finish
    l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
    l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
#pragma unroll
    for (int half = 0; half < 2; ++half) {
        const int gr = half ? r_hi : r_lo;
        if (gr >= a.rows) continue;
        const float mrow = half ? m_hi : m_lo, lrow = half ? l_hi : l_lo;
        const int n = gr / G, g = gr % G;
        if (n_splits == 1) {
            const float inv = lrow > 0.f ? 1.0f / lrow : 0.f;
            __nv_bfloat16 *dst = a.O + (((size_t)b * N + n) * a.Hq + hkv * G + g) * D;
#pragma unroll
            for (int j = 0; j < D / 8; ++j) {
                const uint32_t v = pack_bf16x2(oacc[j][half * 2] * inv, oacc[j][half * 2 + 1] * inv);
                *reinterpret_cast<uint32_t *>(dst + j * 8 + (lane & 3) * 2) = v;
            }
            if (a.lse && (lane & 3) == 0)
                a.lse[((size_t)b * N + n) * a.Hq + hkv * G + g] = (mrow + log2f(lrow)) * 0.6931471805599453f;
        } else {
            const size_t prow = ((size_t)item * a.Hkv + hkv) * a.rows_pad + gr;
            float *dst = a.part_o + prow * D;
#pragma unroll
            for (int j = 0; j < D / 8; ++j)
                *reinterpret_cast<float2 *>(dst + j * 8 + (lane & 3) * 2) =
                    make_float2(oacc[j][half * 2], oacc[j][half * 2 + 1]);
            if ((lane & 3) == 0) {
                a.part_ml[prow * 2] = mrow;
                a.part_ml[prow * 2 + 1] = lrow;
            }
        }
    }
}

// One warp per (b, n, hq): merges the chunks of sequences that were split.
template <int D>
__global__ void __launch_bounds__(128) attn_combine_kernel(AttnArgs a) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const size_t idx = (size_t)blockIdx.x * 4 + warp;
    const size_t total = (size_t)a.B * a.N * a.Hq;
    if (idx >= total) return;
    const int hq = idx % a.Hq;
    const int n = (idx / a.Hq) % a.N;
    const int b = idx / ((size_t)a.Hq * a.N);
    const int it0 = a.item_start[b], ns = a.item_start[b + 1] - it0;
    if (ns == 1) return;
    const int hkv = hq / a.G, gr = n * a.G + hq % a.G;
    float M = -INFINITY;
    for (int s = 0; s < ns; ++s) {
        const size_t prow = ((size_t)(it0 + s) * a.Hkv + hkv) * a.rows_pad + gr;
        M = fmaxf(M, a.part_ml[prow * 2]);
    }
    constexpr int PER = D / 32;
    float acc[PER];
#pragma unroll
    for (int t = 0; t < PER; ++t) acc[t] = 0.f;
    float lsum = 0.f;
    for (int s = 0; s < ns; ++s) {
        const size_t prow = ((size_t)(it0 + s) * a.Hkv + hkv) * a.rows_pad + gr;
        const float ms = a.part_ml[prow * 2];
        const float w = (ms == -INFINITY) ? 0.f : ex2_approx(ms - M);
        lsum += w * a.part_ml[prow * 2 + 1];
        const float *src = a.part_o + prow * D + lane * PER;
#pragma unroll
        for (int t = 0; t < PER; ++t) acc[t] += w * src[t];
    }
    const float inv = lsum > 0.f ? 1.0f / lsum : 0.f;
    __nv_bfloat16 *dst = a.O + idx * D + lane * PER;
#pragma unroll
    for (int t = 0; t < PER; ++t) dst[t] = __float2bfloat16_rn(acc[t] * inv);
    if (a.lse && lane == 0) a.lse[idx] = (M + log2f(lsum)) * 0.6931471805599453f;
}

// ------------------------------------------------------------------------------ host side

constexpr int PLAN_SMS = 148;  // SMs the chunking is planned for

// Estimated finishing time, in quarter tiles, of the persistent tcgen05 kernel when sequences of the given tile
// counts (sorted, longest first) are cut into chunks of at most ct tiles: work units go, in the order the device
// uses, to whichever of PLAN_SMS CTAs is free first.  A unit costs its K/V tiles, one more for the tree tile of a
// sequence's last chunk, one for the hand-over between units; a chunk of a split sequence adds one for its
// partial, and the last one the merge when the attention kernel does it (fewer than 5 chunks per sequence).
static long long estimate_makespan(const std::vector<int> &tiles, int ct, int copies) {
    struct Chunk { int tps, cost; };
    std::vector<Chunk> chunks;
    int max_ns = 1;
    for (int t : tiles) max_ns = std::max(max_ns, (t + ct - 1) / ct);
    const bool merge_inline = max_ns < 5;
    for (int t : tiles) {
        const int ns = std::max(1, (t + ct - 1) / ct), tps = (t + ns - 1) / ns;
        for (int s = 0; s < ns; ++s) {
            const int lo = std::min(t, s * tps), hi = std::min(t, lo + tps);
            int cost = 4 * (hi - lo) + 4;
            if (s == ns - 1) cost += 4;
            if (ns > 1) cost += 4 + ((merge_inline && s == ns - 1) ? 6 * ns : 0);
            chunks.push_back({tps, cost});
        }
    }
    std::stable_sort(chunks.begin(), chunks.end(), [](const Chunk &x, const Chunk &y) { return x.tps > y.tps; });
    std::priority_queue<long long, std::vector<long long>, std::greater<long long>> sms;
    for (int i = 0; i < PLAN_SMS; ++i) sms.push(0);
    long long end = 0;
    for (const Chunk &c : chunks)
        for (int k = 0; k < copies; ++k) {
            const long long t = sms.top() + c.cost;
            sms.pop();
            sms.push(t);
            end = std::max(end, t);
        }
    return end;
}

struct AttnPlan {
    int rows, n_rb, rows_per_block, rows_pad, chunk_tiles, items, tile_tokens, nodes_per_block, n_counters;
    int merge_mode;  // tcgen05 path: 0 = split sequences are merged inside the attention kernel, 2 = by a kernel after it
    bool use_tc;
    size_t off_status, off_items, off_sorted, off_rank, off_tab, off_counters, off_po, off_pml, off_hand, total;
};

static int compute_attn_plan(const specroll_attn_desc *d, const int32_t *indptr_host, AttnPlan *p) {
    if (!d || !indptr_host || d->B < 0 || d->N < 1 || d->N > SPECROLL_MAX_NODES || d->Hq < 1 || d->Hkv < 1 ||
        (d->Hq % d->Hkv) || (d->D != 64 && d->D != 128) || (d->flags & ~SPECROLL_ATTN_ALL_FLAGS) != 0 ||
        !(d->scale > 0.f))
        return SPECROLL_EINVAL;
    const int G = d->Hq / d->Hkv;
    // the tcgen05 kernel needs whole nodes per 128-row block and at most PREP_MAX_B sequences
    p->use_tc = !(d->flags & SPECROLL_ATTN_LEGACY_MMA) && G <= 128 && d->B <= PREP_MAX_B;
    p->tile_tokens = p->use_tc ? 128 : AT_BN;  // KV tokens per tile of the chosen kernel
    const int TT = p->tile_tokens;
    p->rows = d->N * G;
    if (p->use_tc) {
        // row blocks are whole nodes: (node, head-in-group) rows of a block are one TMA box
        // The softmax of a row block costs the same whether the block is full or not, so the rows go into as
        // few blocks as possible.  Every block is a work unit of its own; the units of one (chunk, KV head)
        // are neighbours in the work order, run side by side on different SMs, and the K/V tiles reach the
        // later ones from L2 (measured: DRAM reads stay at one pass over the cache).
        int npb = 128 / G;
        const int nb = (d->N + npb - 1) / npb;
        npb = (d->N + nb - 1) / nb;  // even out the blocks
        p->nodes_per_block = npb;
        p->n_rb = nb;
        p->rows_per_block = npb * G;
    } else {
        p->nodes_per_block = 0;
        p->n_rb = (p->rows + AT_MAX_WARPS * 16 - 1) / (AT_MAX_WARPS * 16);
        p->rows_per_block = ((p->rows + p->n_rb - 1) / p->n_rb + 15) / 16 * 16;
    }
    p->rows_pad = p->rows_per_block * p->n_rb;
    long long tiles_total = 0;
    int max_tiles = 0;
    for (int b = 0; b < d->B; ++b) {
        const int L = indptr_host[b + 1] - indptr_host[b];
        if (L < 0) return SPECROLL_EINVAL;
        const int t = (L + TT - 1) / TT;
        tiles_total += t;
        if (t > max_tiles) max_tiles = t;
    }
    // chunk length.  Legacy kernel: about four CTAs' worth of work per SM over the whole launch.  tcgen05 kernel:
    // the candidate whose estimated finishing time is lowest (the kernel hands the units, longest first, to
    // whichever CTA is free, which a few microseconds of host time can play through).  At least 512 tokens,
    // so that the fp32 partials stay a small fraction of the KV bytes.
    const long long ctas_per_tile = (long long)d->Hkv * p->n_rb;
    auto chunk_for = [&](int per_sm_pct) -> int {
        long long c = (tiles_total * ctas_per_tile * 100 + (long long)PLAN_SMS * per_sm_pct - 1) / ((long long)PLAN_SMS * per_sm_pct);
        if (c < 512 / TT) c = 512 / TT;
        if (c > max_tiles) c = max_tiles > 0 ? max_tiles : 1;
        return (int)c;
    };
    long long ct = chunk_for(p->use_tc ? 100 : 400);
    if (p->use_tc && d->B > 0 && tiles_total * ctas_per_tile <= (1LL << 22)) {
        std::vector<int> tiles((size_t)d->B);
        for (int b = 0; b < d->B; ++b) tiles[(size_t)b] = (indptr_host[b + 1] - indptr_host[b] + TT - 1) / TT;
        std::sort(tiles.begin(), tiles.end(), std::greater<int>());
        static const int pcts[] = {75, 100, 125, 150, 200, 300};
        long long best = -1;
        int seen[6], n_seen = 0;
        for (int pct : pcts) {
            const int c = chunk_for(pct);
            bool dup = false;
            for (int i = 0; i < n_seen; ++i) dup |= (seen[i] == c);
            if (dup) continue;
            seen[n_seen++] = c;
            const long long m = estimate_makespan(tiles, c, (int)ctas_per_tile);
            if (best < 0 || m < best) {
                best = m;
                ct = c;
            }
        }
    }
    p->chunk_tiles = (int)ct;
    int items = 0;
    for (int b = 0; b < d->B; ++b) {
        const int L = indptr_host[b + 1] - indptr_host[b];
        const int t = (L + TT - 1) / TT;
        const int ns = (t + p->chunk_tiles - 1) / p->chunk_tiles;
        items += ns < 1 ? 1 : ns;
    }
    p->items = items;
    if (max_tiles / p->chunk_tiles + 1 > 65535) return SPECROLL_EINVAL;
    // A sequence cut into many chunks is merged by a kernel of its own, over the whole GPU; with few chunks the
    // CTA that finishes a sequence's last chunk merges them while the others keep streaming.
    p->merge_mode = (p->use_tc && (max_tiles + p->chunk_tiles - 1) / p->chunk_tiles >= 5) ? 2 : 0;
    p->n_counters = 64 + d->B * d->Hkv * p->n_rb;  // [0]: work counter, [1]: CTAs that have left; [64 ...]: per (b, hkv, rb) arrivals
    size_t o = 0;
    p->off_status = o;
    o += 256;
    p->off_items = o;
    o += align_up((size_t)(d->B + 1) * 4, 256);
    p->off_sorted = o;
    o += align_up((size_t)(d->B + 1) * 4, 256);
    p->off_rank = o;
    o += align_up((size_t)(d->B + 1) * 4, 256);
    p->off_tab = o;
    o += align_up((size_t)items * 32, 256);
    p->off_counters = o;
    o += align_up((size_t)p->n_counters * 4, 256);
    p->off_po = o;
    o += align_up((size_t)items * d->Hkv * p->rows_pad * d->D * 4, 256);
    p->off_pml = o;
    o += align_up((size_t)items * d->Hkv * p->rows_pad * 2 * 4, 256);
    p->off_hand = o;
    o += (size_t)ATTN_HAND_CTAS * 4 * 128 * 4;
    p->total = o + 256;
    return SPECROLL_OK;
}

template <int D>
static int launch_attn(const AttnArgs &a, const TopoMask &mask, const AttnPlan &p, int Hkv, size_t n_out,
                       cudaStream_t st) {
    using S = AttnSmem<D>;
    SR_CUDA_TRY(cudaFuncSetAttribute(tree_attn_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, S::TOTAL));
    const int threads = (p.rows_per_block / 16) * 32;
    const unsigned grid = (unsigned)p.items * Hkv * p.n_rb;
    tree_attn_kernel<D><<<grid, threads, S::TOTAL, st>>>(a, mask);
    SR_LAUNCH_CHECK();
    attn_combine_kernel<D><<<(unsigned)((n_out + 3) / 4), 128, 0, st>>>(a);
    SR_LAUNCH_CHECK();
    return SPECROLL_OK;
}

}  // namespace specroll

using namespace specroll;

// Plans are remembered for the last few (shape, lengths) seen: every layer of a step asks for the same one.
static int make_attn_plan(const specroll_attn_desc *d, const int32_t *indptr_host, AttnPlan *p) {
    struct Entry {
        int key[7];
        std::vector<int32_t> indptr;
        AttnPlan plan;
    };
    static std::mutex mu;
    static Entry cache[4];
    static unsigned next = 0;
    if (!d || !indptr_host || d->B < 0 || d->B > (1 << 24)) return compute_attn_plan(d, indptr_host, p);
    // what the key leaves out is checked here, so that a remembered plan never answers for an invalid call
    if ((d->flags & ~SPECROLL_ATTN_ALL_FLAGS) != 0 || !(d->scale > 0.f)) return SPECROLL_EINVAL;
    const int key[7] = {d->B, d->N, d->Hq, d->Hkv, d->D, (int)(d->flags & SPECROLL_ATTN_LEGACY_MMA), 1};
    const size_t n = (size_t)d->B + 1;
    std::lock_guard<std::mutex> lock(mu);
    for (Entry &e : cache)
        if (memcmp(e.key, key, sizeof(key)) == 0 && e.indptr.size() == n &&
            memcmp(e.indptr.data(), indptr_host, n * sizeof(int32_t)) == 0) {
            *p = e.plan;
            return SPECROLL_OK;
        }
    const int rc = compute_attn_plan(d, indptr_host, p);
    if (rc != SPECROLL_OK) return rc;
    Entry &e = cache[next++ % 4];
    memcpy(e.key, key, sizeof(key));
    e.indptr.assign(indptr_host, indptr_host + n);
    e.plan = *p;
    return SPECROLL_OK;
}

extern "C" size_t specroll_tree_attn_workspace_bytes(const specroll_attn_desc *d,
                                                     const int32_t *kv_indptr_host) {
    AttnPlan p;
    if (make_attn_plan(d, kv_indptr_host, &p) != SPECROLL_OK) return 0;
    return p.total;
}

extern "C" int specroll_tree_attn_launches(const specroll_attn_desc *d, const int32_t *kv_indptr_host) {
    AttnPlan p;
    if (make_attn_plan(d, kv_indptr_host, &p) != SPECROLL_OK) return -1;
    if (d->B == 0) return 0;
    const bool split = p.items > d->B;
    if (p.use_tc) return ((d->flags & SPECROLL_ATTN_REUSE_PLAN) ? 0 : 1) + 1 + ((p.merge_mode == 2 && split) ? 1 : 0);
    return 1 + 1 + (split ? 1 : 0);
}

// Common body of the two entry points.  Contiguous cache: kv_indptr_dev, T_kv = cached tokens.  Paged cache:
// kv_len_dev, page_indptr_dev, page_table_dev, T_kv = tokens in the page pool.  indptr_host is the (derived)
// prefix of the host lengths either way.
static int run_tree_attn(const specroll_attn_desc *d, const void *Q, const void *Kc, const void *Vc, long long T_kv,
                         const int32_t *kv_indptr_dev, const int32_t *kv_len_dev, const int32_t *page_indptr_dev,
                         const int32_t *page_table_dev, const int32_t *indptr_host, const void *Kt, const void *Vt,
                         const int32_t *parent_host, void *O, float *lse, void *workspace, size_t workspace_bytes,
                         void *cuda_stream) {
    const bool paged = page_table_dev != nullptr;
    AttnPlan p;
    if (make_attn_plan(d, indptr_host, &p) != SPECROLL_OK) return SPECROLL_EINVAL;
    if (d->B == 0) {  // (an empty batch has empty arrays: their pointers may be NULL)
        Topo topo0;
        TopoMask mask0;
        return build_topo(parent_host, d->N, -1, -1, &topo0, &mask0) == SPECROLL_OK ? SPECROLL_OK : SPECROLL_EINVAL;
    }
    if (!Q || !Kt || !Vt || !O) return SPECROLL_EINVAL;
    if (paged ? (!kv_len_dev || !page_indptr_dev) : !kv_indptr_dev) return SPECROLL_EINVAL;
    if (paged && !p.use_tc) return SPECROLL_ELIMIT;  // the mma.sync kernel reads a contiguous cache only
    if (T_kv > 0 && (!Kc || !Vc)) return SPECROLL_EINVAL;
    Topo topo;
    TopoMask mask;
    if (build_topo(parent_host, d->N, -1, -1, &topo, &mask) != SPECROLL_OK) return SPECROLL_EINVAL;
    if (!aligned16(Q) || !aligned16(Kc) || !aligned16(Vc) || !aligned16(Kt) || !aligned16(Vt) || !aligned16(O))
        return SPECROLL_EALIGN;
    if (d->B == 0) return SPECROLL_OK;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) || workspace_bytes < p.total)
        return SPECROLL_EWORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    char *ws = static_cast<char *>(workspace);
    AttnArgs a;
    a.Q = static_cast<const __nv_bfloat16 *>(Q);
    a.Kc = static_cast<const __nv_bfloat16 *>(Kc);
    a.Vc = static_cast<const __nv_bfloat16 *>(Vc);
    a.Kt = static_cast<const __nv_bfloat16 *>(Kt);
    a.Vt = static_cast<const __nv_bfloat16 *>(Vt);
    a.kv_indptr = kv_indptr_dev;
    a.page_table = page_table_dev;
    a.item_start = reinterpret_cast<int32_t *>(ws + p.off_items);
    a.O = static_cast<__nv_bfloat16 *>(O);
    a.lse = lse;
    a.part_o = reinterpret_cast<float *>(ws + p.off_po);
    a.part_ml = reinterpret_cast<float *>(ws + p.off_pml);
    a.hand = reinterpret_cast<float *>(ws + p.off_hand);
    a.B = d->B;
    a.N = d->N;
    a.Hq = d->Hq;
    a.Hkv = d->Hkv;
    a.G = d->Hq / d->Hkv;
    a.rows = p.rows;
    a.rows_pad = p.rows_pad;
    a.n_rb = p.n_rb;
    a.rows_per_block = p.rows_per_block;
    a.chunk_tiles = p.chunk_tiles;
    a.tile_tokens = p.tile_tokens;
    a.scale_log2 = d->scale * LOG2E;
    int32_t *status = reinterpret_cast<int32_t *>(ws + p.off_status);
    int32_t *counters = reinterpret_cast<int32_t *>(ws + p.off_counters);
    int32_t *sorted_start = reinterpret_cast<int32_t *>(ws + p.off_sorted);
    int32_t *seq_at_rank = reinterpret_cast<int32_t *>(ws + p.off_rank);
    int32_t *unit_tab = reinterpret_cast<int32_t *>(ws + p.off_tab);
    a.sorted_start = sorted_start;
    a.seq_at_rank = seq_at_rank;
    a.unit_tab = unit_tab;
    a.work_counter = counters;
    a.split_counters = counters + 64;
    a.total_work = p.items * d->Hkv * p.n_rb;
    a.merge_mode = p.merge_mode;
    a.nodes_per_block = p.nodes_per_block;
    a.no_pdl = (d->flags & SPECROLL_ATTN_NO_PDL) ? 1 : 0;
    // early cache loads need a plan that is not being made by the kernel just before the attention kernel
    a.early_cache = ((d->flags & SPECROLL_ATTN_CACHE_SETTLED) && (d->flags & SPECROLL_ATTN_REUSE_PLAN)) ? 1 : 0;
    if (!(p.use_tc && (d->flags & SPECROLL_ATTN_REUSE_PLAN))) {
        // (the tcgen05 kernel leaves its scheduling counters cleared, so a kept plan can be run again as is)
        attn_prep_kernel<<<1, PREP_THREADS, 0, st>>>(kv_indptr_dev, paged ? kv_len_dev : nullptr, page_indptr_dev, d->B,
                                                     p.chunk_tiles, p.tile_tokens,
                                                     reinterpret_cast<int32_t *>(ws + p.off_items),
                                                     p.use_tc ? sorted_start : nullptr, seq_at_rank,
                                                     p.use_tc ? unit_tab : nullptr, status, counters, p.n_counters);
        SR_LAUNCH_CHECK();
    }
    const size_t n_out = (size_t)d->B * d->N * d->Hq;
    if (p.use_tc) {
        const int rc = launch_attn_tc(a, mask, d->D, T_kv, status, st);
        if (rc != SPECROLL_OK || p.merge_mode != 2 || p.items <= d->B) return rc;
        return launch_attn_merge_tc(a, d->D, p.items, st);
    }
    if (d->D == 128) return launch_attn<128>(a, mask, p, d->Hkv, n_out, st);
    return launch_attn<64>(a, mask, p, d->Hkv, n_out, st);
}

extern "C" int specroll_tree_attn(const specroll_attn_desc *d, const void *Q, const void *Kc, const void *Vc,
                                  const int32_t *kv_indptr_dev, const int32_t *kv_indptr_host, const void *Kt,
                                  const void *Vt, const int32_t *parent_host, void *O, float *lse,
                                  void *workspace, size_t workspace_bytes, void *cuda_stream) {
    // the cache tensors start at the first sequence's first token: token coordinates count from their base
    if (!d || !kv_indptr_host || d->B < 0 || kv_indptr_host[0] != 0) return SPECROLL_EINVAL;
    const long long T_kv = (long long)kv_indptr_host[d->B];
    return run_tree_attn(d, Q, Kc, Vc, T_kv, kv_indptr_dev, nullptr, nullptr, nullptr, kv_indptr_host, Kt, Vt,
                         parent_host, O, lse, workspace, workspace_bytes, cuda_stream);
}

// Prefix of the host lengths: what the planner takes.  False if a length is negative.
static bool lengths_to_indptr(const int32_t *kv_len_host, int B, std::vector<int32_t> *ip) {
    ip->assign((size_t)B + 1, 0);
    long long acc = 0;
    for (int b = 0; b < B; ++b) {
        if (kv_len_host[b] < 0) return false;
        acc += kv_len_host[b];
        if (acc > 0x7fffffffLL) return false;
        (*ip)[(size_t)b + 1] = (int32_t)acc;
    }
    return true;
}

extern "C" size_t specroll_tree_attn_paged_workspace_bytes(const specroll_attn_desc *d, const int32_t *kv_len_host) {
    if (!d || !kv_len_host || d->B < 0 || d->B > (1 << 24)) return 0;
    std::vector<int32_t> ip;
    if (!lengths_to_indptr(kv_len_host, d->B, &ip)) return 0;
    AttnPlan p;
    if (make_attn_plan(d, ip.data(), &p) != SPECROLL_OK || !p.use_tc) return 0;
    return p.total;
}

extern "C" int specroll_tree_attn_paged(const specroll_attn_desc *d, const void *Q, const void *Kp, const void *Vp,
                                        int64_t n_pages, const int32_t *page_table_dev,
                                        const int32_t *page_indptr_dev, const int32_t *kv_len_dev,
                                        const int32_t *kv_len_host, const void *Kt, const void *Vt,
                                        const int32_t *parent_host, void *O, float *lse, void *workspace,
                                        size_t workspace_bytes, void *cuda_stream) {
    if (!d || !kv_len_host || d->B < 0 || d->B > (1 << 24) || n_pages < 0 || n_pages > (1LL << 24) || !page_table_dev)
        return SPECROLL_EINVAL;
    std::vector<int32_t> ip;
    if (!lengths_to_indptr(kv_len_host, d->B, &ip)) return SPECROLL_EINVAL;
    return run_tree_attn(d, Q, Kp, Vp, n_pages * SPECROLL_PAGE_TOKENS, nullptr, kv_len_dev, page_indptr_dev,
                         page_table_dev, ip.data(), Kt, Vt, parent_host, O, lse, workspace, workspace_bytes, cuda_stream);
}
