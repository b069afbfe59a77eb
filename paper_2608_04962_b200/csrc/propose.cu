// Proposal step: LayerNorm -> K head MLPs -> bounded correction -> shared vocabulary projection
// with a fused running top-k (logits never reach memory) -> top-k merge -> tree draw.
#include <math.h>

#include "common.cuh"
#include "gemm_mma.cuh"

namespace specroll {

// ------------------------------------------------------------------------------ block reduce

template <int THREADS>
__device__ __forceinline__ float block_sum(float v, float *sh) {
    v = warp_sum(v);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    __syncthreads();
    if (lane == 0) sh[warp] = v;
    __syncthreads();
    float t = lane < THREADS / 32 ? sh[lane] : 0.f;
    return warp_sum(t);
}

// ------------------------------------------------------------------------------ P1 LayerNorm

constexpr int LN_THREADS = 256;

// h[B,d] bf16 -> xhat[KX,B,d] bf16 with KX = K when an affine (gamma/beta) is given, else 1.
__global__ void __launch_bounds__(LN_THREADS)
layernorm_kernel(const __nv_bfloat16 *__restrict__ h, const __nv_bfloat16 *__restrict__ gamma,
                 const __nv_bfloat16 *__restrict__ beta, __nv_bfloat16 *__restrict__ xhat, int B, int d,
                 int KX, float eps) {
    extern __shared__ float row[];  // d floats
    __shared__ float red[LN_THREADS / 32];
    pdl_launch_dependents();
    pdl_wait();
    const int b = blockIdx.x;
    float s = 0.f;
    for (int i = threadIdx.x; i < d; i += LN_THREADS) {
        const float v = __bfloat162float(h[(size_t)b * d + i]);
        row[i] = v;
        s += v;
    }
    const float mu = block_sum<LN_THREADS>(s, red) / d;
    float q = 0.f;
    for (int i = threadIdx.x; i < d; i += LN_THREADS) {
        const float t = row[i] - mu;
        q += t * t;
    }
    const float var = block_sum<LN_THREADS>(q, red) / d;
    const float rstd = 1.0f / sqrtf(var + eps);
    for (int hd = 0; hd < KX; ++hd) {
        for (int i = threadIdx.x; i < d; i += LN_THREADS) {
            float x = (row[i] - mu) * rstd;
            if (gamma) x *= __bfloat162float(gamma[(size_t)hd * d + i]);
            if (beta) x += __bfloat162float(beta[(size_t)hd * d + i]);
            xhat[((size_t)hd * B + b) * d + i] = __float2bfloat16_rn(x);
        }
    }
}

// ------------------------------------------------------------------------------ P2 head MLP

using HeadTile = MmaTile<128, 64, 4, 2, 3>;  // 8 warps, warp tile 32 x 32

// z[b,hd,o] = h[b,o] + SiLU(sum_i xhat[hd?,b,i] * A[hd,o,i] + bias[hd,o])      (fp32 out)
__global__ void __launch_bounds__(HeadTile::THREADS)
head_mlp_kernel(const __nv_bfloat16 *__restrict__ xhat, int KX, const __nv_bfloat16 *__restrict__ A,
                const __nv_bfloat16 *__restrict__ bias, const __nv_bfloat16 *__restrict__ h,
                float *__restrict__ z, int B, int K, int d) {
    extern __shared__ __align__(128) unsigned char smem[];
    using T = HeadTile;
    const int hd = blockIdx.z, m0 = blockIdx.y * T::BM, n0 = blockIdx.x * T::BN;
    const __nv_bfloat16 *X = xhat + (KX > 1 ? (size_t)hd * B * d : 0);
    const __nv_bfloat16 *Ah = A + (size_t)hd * d * d;
    float acc[T::MT][T::NT][4];
    T::run(smem, X, d, m0, B, Ah, d, n0, d, d, acc);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int wm0 = (warp / T::WN) * T::WTM, wn0 = (warp % T::WN) * T::WTN;
#pragma unroll
    for (int i = 0; i < T::MT; ++i)
#pragma unroll
        for (int j = 0; j < T::NT; ++j)
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                const int row = m0 + wm0 + i * 16 + (lane >> 2) + (t >> 1) * 8;
                const int col = n0 + wn0 + j * 8 + (lane & 3) * 2 + (t & 1);
                if (row < B && col < d) {
                    const float y = acc[i][j][t] + __bfloat162float(bias[(size_t)hd * d + col]);
                    const float sl = y / (1.0f + __expf(-y));
                    z[((size_t)row * K + hd) * d + col] = __bfloat162float(h[(size_t)row * d + col]) + sl;
                }
            }
}

// ------------------------------------------------------------------------------ P3 bounded correction

constexpr int RX_THREADS = 256;

// zt[r,:] = bf16(z[r,:] + coef * m[r,:]),  r = b*K + hd,
// coef = alpha * RMS(z) / (RMS(m) + eps), shrunk so that |coef * m|_2 <= clip_c * |z|_2.
__global__ void __launch_bounds__(RX_THREADS)
reflex_kernel(const float *__restrict__ z, const float *__restrict__ m, const float *__restrict__ alpha,
              __nv_bfloat16 *__restrict__ zt, int d, float rms_eps, float clip_c) {
    __shared__ float red[RX_THREADS / 32];
    pdl_launch_dependents();
    pdl_wait();
    const size_t r = blockIdx.x;
    const float *zr = z + r * d;
    const float a = (alpha && m) ? alpha[r] : 0.f;
    float coef = 0.f;
    if (a != 0.f) {  // uniform across the block
        const float *mr = m + r * d;
        float sz = 0.f, sm = 0.f;
        for (int i = threadIdx.x; i < d; i += RX_THREADS) {
            const float zv = zr[i], mv = mr[i];
            sz += zv * zv;
            sm += mv * mv;
        }
        sz = block_sum<RX_THREADS>(sz, red);
        sm = block_sum<RX_THREADS>(sm, red);
        const float rms_z = sqrtf(sz / d), rms_m = sqrtf(sm / d);
        coef = a * rms_z / (rms_m + rms_eps);
        const float nd = fabsf(coef) * sqrtf(sm), nz = sqrtf(sz);
        if (clip_c > 0.f && nd > clip_c * nz) coef *= clip_c * nz / nd;
        for (int i = threadIdx.x; i < d; i += RX_THREADS) zt[r * d + i] = __float2bfloat16_rn(zr[i] + coef * mr[i]);
    } else {
        for (int i = threadIdx.x; i < d; i += RX_THREADS) zt[r * d + i] = __float2bfloat16_rn(zr[i]);
    }
}

// Secondary form of the correction (SPECROLL_REFLEX_PRE_HEAD): applied to the last hidden state, one memory row
// and one ratio per sequence.  ht[b,:] = bf16(h[b,:] + coef * m[b,:]), coef = alpha RMS(h) / (RMS(m) + eps), shrunk
// so that |coef * m|_2 <= clip_c * |h|_2; alpha = 0 or no memory: ht = h bit for bit.
__global__ void __launch_bounds__(RX_THREADS)
prehead_kernel(const __nv_bfloat16 *__restrict__ h, const float *__restrict__ m, const float *__restrict__ alpha,
               __nv_bfloat16 *__restrict__ ht, int d, float rms_eps, float clip_c) {
    __shared__ float red[RX_THREADS / 32];
    pdl_launch_dependents();
    const size_t r = blockIdx.x;
    const __nv_bfloat16 *hr = h + r * d;
    const float a = (alpha && m) ? alpha[r] : 0.f;
    if (a != 0.f) {  // uniform across the block
        const float *mr = m + r * d;
        float sh = 0.f, sm = 0.f;
        for (int i = threadIdx.x; i < d; i += RX_THREADS) {
            const float hv = __bfloat162float(hr[i]), mv = mr[i];
            sh += hv * hv;
            sm += mv * mv;
        }
        sh = block_sum<RX_THREADS>(sh, red);
        sm = block_sum<RX_THREADS>(sm, red);
        const float rms_h = sqrtf(sh / d), rms_m = sqrtf(sm / d);
        float coef = a * rms_h / (rms_m + rms_eps);
        const float nd = fabsf(coef) * sqrtf(sm), nh = sqrtf(sh);
        if (clip_c > 0.f && nd > clip_c * nh) coef *= clip_c * nh / nd;
        for (int i = threadIdx.x; i < d; i += RX_THREADS) ht[r * d + i] = __float2bfloat16_rn(__bfloat162float(hr[i]) + coef * mr[i]);
    } else {
        for (int i = threadIdx.x; i < d; i += RX_THREADS) ht[r * d + i] = hr[i];
    }
}

// ------------------------------------------------------------------------------ P4 projection + top-k

// Sorted (descending value; earlier insertion wins ties) list of the KMAX best seen so far.
template <int KMAX>
struct TopList {
    float v[KMAX];
    int32_t id[KMAX];
    __device__ __forceinline__ void init() {
#pragma unroll
        for (int i = 0; i < KMAX; ++i) {
            v[i] = -INFINITY;
            id[i] = 0x7fffffff;
        }
    }
    // candidates arrive in increasing id order, so "strictly greater" keeps the lowest id on ties
    __device__ __forceinline__ void push(float x, int32_t t) {
        if (!(x > v[KMAX - 1])) return;
#pragma unroll
        for (int i = KMAX - 1; i > 0; --i) {
            if (x > v[i - 1]) {
                v[i] = v[i - 1];
                id[i] = id[i - 1];
            } else if (x > v[i]) {  // v[i-1] >= x > v[i]
                v[i] = x;
                id[i] = t;
            }
        }
        if (x > v[0]) {
            v[0] = x;
            id[0] = t;
        }
    }
};

using LmTile = MmaTile<128, 128, 2, 4, 3>;  // 8 warps, warp tile 64 x 32
constexpr int LM_CSTRIDE = 129;            // fp32 staging tile row stride (conflict-free row scans)

// Each CTA owns one block of 128 rows and a contiguous range of vocabulary tiles; thread r < 128
// keeps the running top list of row r across those tiles.  Partial lists go to
// pval/pid[M, n_groups, k]; a merge kernel finishes.
template <int KMAX>
__global__ void __launch_bounds__(LmTile::THREADS)
lm_head_topk_kernel(const __nv_bfloat16 *__restrict__ Zt, const __nv_bfloat16 *__restrict__ W, int M,
                    int V, int d, int k, int n_mblocks, int n_groups, int tiles_per_group,
                    float *__restrict__ pval, int32_t *__restrict__ pid) {
    extern __shared__ __align__(128) unsigned char smem[];
    using T = LmTile;
    const int mb = blockIdx.x % n_mblocks, grp = blockIdx.x / n_mblocks;
    const int m0 = mb * T::BM;
    const int n_tiles = (V + T::BN - 1) / T::BN;
    const int t_lo = grp * tiles_per_group, t_hi = min(n_tiles, t_lo + tiles_per_group);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int wm0 = (warp / T::WN) * T::WTM, wn0 = (warp % T::WN) * T::WTN;
    float *ctile = reinterpret_cast<float *>(smem);
    TopList<KMAX> top;
    top.init();
    for (int tile = t_lo; tile < t_hi; ++tile) {
        const int n0 = tile * T::BN;
        float acc[T::MT][T::NT][4];
        T::run(smem, Zt, d, m0, M, W, d, n0, V, d, acc);  // ends with a barrier: smem is free
#pragma unroll
        for (int i = 0; i < T::MT; ++i)
#pragma unroll
            for (int j = 0; j < T::NT; ++j)
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    const int row = wm0 + i * 16 + (lane >> 2) + (t >> 1) * 8;
                    const int col = wn0 + j * 8 + (lane & 3) * 2 + (t & 1);
                    ctile[row * LM_CSTRIDE + col] = acc[i][j][t];
                }
        __syncthreads();
        if (threadIdx.x < T::BM) {
            const float *rp = ctile + threadIdx.x * LM_CSTRIDE;
            const int ncol = min(T::BN, V - n0);
            for (int c = 0; c < ncol; ++c) top.push(rp[c], n0 + c);
        }
        __syncthreads();
    }
    if (threadIdx.x < T::BM && m0 + threadIdx.x < M) {
        const size_t o = ((size_t)(m0 + threadIdx.x) * n_groups + grp) * k;
#pragma unroll
        for (int i = 0; i < KMAX; ++i)
            if (i < k) {
                pval[o + i] = top.v[i];
                pid[o + i] = top.id[i];
            }
    }
}

// One warp per row: k rounds of arg-best over the n_cand partial entries, order (value desc, id asc).
__global__ void __launch_bounds__(128)
topk_merge_kernel(const float *__restrict__ pval, const int32_t *__restrict__ pid, int M, int n_cand, int k,
                  int32_t *__restrict__ cand_id, float *__restrict__ cand_logit) {
    pdl_launch_dependents();
    pdl_wait();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int r = blockIdx.x * 4 + warp;
    if (r >= M) return;
    const float *v = pval + (size_t)r * n_cand;
    const int32_t *id = pid + (size_t)r * n_cand;
    float last_v = INFINITY;
    int32_t last_id = -1;
    for (int j = 0; j < k; ++j) {
        float bv = -INFINITY;
        int32_t bi = 0x7fffffff;
        for (int c = lane; c < n_cand; c += 32) {
            const float x = v[c];
            const int32_t t = id[c];
            // strictly after the previous pick in the (value desc, id asc) order
            const bool after = (x < last_v) || (x == last_v && t > last_id);
            if (after && (x > bv || (x == bv && t < bi))) {
                bv = x;
                bi = t;
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
            const int32_t oi = __shfl_xor_sync(0xffffffffu, bi, o);
            if (ov > bv || (ov == bv && oi < bi)) {
                bv = ov;
                bi = oi;
            }
        }
        if (lane == 0) {
            cand_id[(size_t)r * k + j] = bi;
            cand_logit[(size_t)r * k + j] = bv;
        }
        last_v = bv;
        last_id = bi;
    }
}

// The same for k <= 8, the size of the tensor-core projection's partial lists: every lane first keeps the k best of
// its own share of the partial entries in registers (one pass, the loads independent of each other), then k rounds of
// arg-best over the lanes' current best, the winner moving on to its next one.  (Re-reading all entries in each of
// the k rounds made this kernel a tenth of the call at small batch.)
struct Top8 {
    float v[8];
    int32_t i[8];
};
__device__ __forceinline__ bool tk_better(float x, int32_t t, float y, int32_t u) { return x > y || (x == y && t < u); }
__device__ __forceinline__ void tk_init(Top8 &L) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        L.v[i] = -INFINITY;
        L.i[i] = 0x7fffffff;
    }
}
// insert into the sorted list (best first) if it belongs there
__device__ __forceinline__ void tk_insert(Top8 &L, float x, int32_t t) {
    if (!tk_better(x, t, L.v[7], L.i[7])) return;
#pragma unroll
    for (int i = 7; i > 0; --i) {
        if (tk_better(x, t, L.v[i - 1], L.i[i - 1])) {
            L.v[i] = L.v[i - 1];
            L.i[i] = L.i[i - 1];
        } else if (tk_better(x, t, L.v[i], L.i[i])) {
            L.v[i] = x;
            L.i[i] = t;
        }
    }
    if (tk_better(x, t, L.v[0], L.i[0])) {
        L.v[0] = x;
        L.i[0] = t;
    }
}
// the best of the lanes' current best; the lane that held it moves on to its next one (ids are distinct: one lane)
__device__ __forceinline__ void tk_pop_best(Top8 &L, float &bv, int32_t &bi) {
    bv = L.v[0];
    bi = L.i[0];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
        const int32_t oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (tk_better(ov, oi, bv, bi)) {
            bv = ov;
            bi = oi;
        }
    }
    if (L.v[0] == bv && L.i[0] == bi) {
#pragma unroll
        for (int i = 0; i < 7; ++i) {
            L.v[i] = L.v[i + 1];
            L.i[i] = L.i[i + 1];
        }
        L.v[7] = -INFINITY;
        L.i[7] = 0x7fffffff;
    }
}
// a lane's share of the entries [c_lo, c_hi) of one row's partial lists, four independent loads at a time
__device__ __forceinline__ void tk_scan(Top8 &L, const float *__restrict__ v, const int32_t *__restrict__ id, int c_lo,
                                        int c_hi, int lane) {
    for (int c0 = c_lo + lane; c0 < c_hi; c0 += 4 * 32) {
        float x[4];
        int32_t t[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int c = c0 + q * 32;
            x[q] = c < c_hi ? v[c] : -INFINITY;
            t[q] = c < c_hi ? id[c] : 0x7fffffff;
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) tk_insert(L, x[q], t[q]);
    }
}

__global__ void __launch_bounds__(128)
topk_merge8_kernel(const float *__restrict__ pval, const int32_t *__restrict__ pid, int M, int n_cand, int k,
                   int32_t *__restrict__ cand_id, float *__restrict__ cand_logit) {
    pdl_launch_dependents();
    pdl_wait();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int r = blockIdx.x * 4 + warp;
    if (r >= M) return;
    Top8 L;
    tk_init(L);
    tk_scan(L, pval + (size_t)r * n_cand, pid + (size_t)r * n_cand, 0, n_cand, lane);
    for (int j = 0; j < k; ++j) {
        float bv;
        int32_t bi;
        tk_pop_best(L, bv, bi);
        if (lane == 0) {
            cand_id[(size_t)r * k + j] = bi;
            cand_logit[(size_t)r * k + j] = bv;
        }
    }
}

// The same with a CTA of eight warps per row, for rows with 32 or more partial lists (few rows in the projection, so
// many CTAs of the projection kernel have a list for each of them): a warp merges an eighth of the entries, warp 0
// the eight results.  (One warp per row took 24 us on 32 rows of 148 lists, a tenth of the call.)
constexpr int MERGE_WIDE_WARPS = 8;
__global__ void __launch_bounds__(MERGE_WIDE_WARPS * 32)
topk_merge8_wide_kernel(const float *__restrict__ pval, const int32_t *__restrict__ pid, int M, int n_cand, int k,
                        int32_t *__restrict__ cand_id, float *__restrict__ cand_logit) {
    pdl_launch_dependents();
    pdl_wait();
    __shared__ float sv[MERGE_WIDE_WARPS * 8];
    __shared__ int32_t si[MERGE_WIDE_WARPS * 8];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int r = blockIdx.x;
    const float *v = pval + (size_t)r * n_cand;
    const int32_t *id = pid + (size_t)r * n_cand;
    const int per = (n_cand + MERGE_WIDE_WARPS - 1) / MERGE_WIDE_WARPS;
    Top8 L;
    tk_init(L);
    tk_scan(L, v, id, min(n_cand, warp * per), min(n_cand, warp * per + per), lane);
    for (int j = 0; j < 8; ++j) {
        float bv;
        int32_t bi;
        tk_pop_best(L, bv, bi);
        if (lane == 0) {
            sv[warp * 8 + j] = bv;
            si[warp * 8 + j] = bi;
        }
    }
    __syncthreads();
    if (warp != 0) return;
    tk_init(L);
    tk_scan(L, sv, si, 0, MERGE_WIDE_WARPS * 8, lane);
    for (int j = 0; j < k; ++j) {
        float bv;
        int32_t bi;
        tk_pop_best(L, bv, bi);
        if (lane == 0) {
            cand_id[(size_t)r * k + j] = bi;
            cand_logit[(size_t)r * k + j] = bv;
        }
    }
}

// ------------------------------------------------------------------------------ P5 tree draw

constexpr int DRAW_WARPS = 8;

__device__ __forceinline__ double warp_incl_scan_f64(double v, int lane) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const double t = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += t;
    }
    return v;
}

// One CTA per sequence, one warp per parent node.  A child's distribution depends on what its earlier siblings
// drew and on nothing else, so the children of different parents are drawn at the same time and only siblings
// wait for each other; within a draw the work over the k candidates is spread over the lanes (lane j holds
// candidates j and j + 32): their total, the running sums of the inverse-CDF walk and the first candidate whose
// running sum exceeds the uniform come from warp scans and ballots.  (Node after node on one warp, a draw of 48
// nodes took 32 us: some twenty dependent fp64 operations and shuffles per node.)
__global__ void __launch_bounds__(DRAW_WARPS * 32)
tree_draw_kernel(Topo topo, int B, int K, int k, double T, const int32_t *__restrict__ anchor,
                 const int32_t *__restrict__ cand_id, const float *__restrict__ cand_logit,
                 const float *__restrict__ u_draw, int32_t *__restrict__ tree_tok,
                 uint8_t *__restrict__ tree_cand, float *__restrict__ slot_q) {
    // Softmax weights of every head's candidates, relative to the head's largest logit, once per sequence: a
    // child's distribution is these weights renormalised over the candidates its earlier siblings left.
    __shared__ double sh_w[SPECROLL_MAX_HEADS][SPECROLL_MAX_TOPK];
    __shared__ int32_t sh_id[SPECROLL_MAX_HEADS][SPECROLL_MAX_TOPK];
    __shared__ float sh_u[SPECROLL_MAX_NODES];
    __shared__ int8_t sh_parent[SPECROLL_MAX_NODES];
    pdl_wait();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int b = blockIdx.x;
    const int N = topo.N;
    const double inv_T = 1.0 / T;  // (the largest logit minus itself over T would be a division with a zero numerator)
    for (int hd = warp; hd < K; hd += DRAW_WARPS) {
        const float *cl = cand_logit + ((size_t)b * K + hd) * k;
        float mxf = -INFINITY;
        for (int j = lane; j < k; j += 32) mxf = fmaxf(mxf, cl[j]);
        mxf = warp_max(mxf);
        for (int j = lane; j < k; j += 32) {
            sh_w[hd][j] = exp(((double)cl[j] - (double)mxf) * inv_T);
            sh_id[hd][j] = cand_id[((size_t)b * K + hd) * k + j];
        }
    }
    for (int n = threadIdx.x; n < N; n += DRAW_WARPS * 32) {
        sh_u[n] = u_draw[(size_t)b * N + n];
        sh_parent[n] = topo.parent[n];
    }
    if (threadIdx.x == 0) {
        tree_tok[(size_t)b * N] = anchor[b];
        tree_cand[(size_t)b * N] = 255;
        slot_q[(size_t)b * N] = 1.0f;
    }
    __syncthreads();
    int idx = 0;
    for (int u = 0; u < N; ++u) {
        if (topo.n_child[u] == 0) continue;
        if ((idx++ % DRAW_WARPS) != warp) continue;
        const int hd = topo.depth[u];  // the children of u are drawn by head depth(u) (0-based)
        const double *w = sh_w[hd];
        // children of u (a child's index is larger than its parent's), in slot order
        const unsigned cm_lo = __ballot_sync(0xffffffffu, lane > u && lane < N && sh_parent[lane < N ? lane : 0] == u);
        const unsigned cm_hi =
            __ballot_sync(0xffffffffu, lane + 32 > u && lane + 32 < N && sh_parent[lane + 32 < N ? lane + 32 : 0] == u);
        unsigned long long cm = ((unsigned long long)cm_hi << 32) | cm_lo;
        unsigned long long taken = 0ull;
        while (cm) {
            const int n = __ffsll((long long)cm) - 1;
            cm &= cm - 1;
            const bool ok0 = lane < k && !((taken >> lane) & 1ull);
            const bool ok1 = lane + 32 < k && !((taken >> (lane + 32)) & 1ull);
            double w0 = ok0 ? w[lane] : 0.0, w1 = ok1 ? w[lane + 32] : 0.0;
            // running sums over the remaining candidates; their total is the last one
            double c0 = warp_incl_scan_f64(w0, lane);
            double c1 = __shfl_sync(0xffffffffu, c0, 31);
            if (k > 32) c1 += warp_incl_scan_f64(w1, lane);
            double s = __shfl_sync(0xffffffffu, c1, 31);
            if (!(s > 0.0)) {
                // every remaining weight underflowed against a taken candidate's logit: take the reference among
                // the remaining ones instead
                const float *cl = cand_logit + ((size_t)b * K + hd) * k;
                float mxf = fmaxf(ok0 ? cl[lane] : -INFINITY, ok1 ? cl[lane + 32] : -INFINITY);
                mxf = warp_max(mxf);
                w0 = ok0 ? exp(((double)cl[lane] - (double)mxf) * inv_T) : 0.0;
                w1 = ok1 ? exp(((double)cl[lane + 32] - (double)mxf) * inv_T) : 0.0;
                c0 = warp_incl_scan_f64(w0, lane);
                c1 = __shfl_sync(0xffffffffu, c0, 31) + warp_incl_scan_f64(w1, lane);
                s = __shfl_sync(0xffffffffu, c1, 31);
            }
            // first remaining candidate whose cumulative probability exceeds the uniform (compared as masses)
            const double thr = (double)sh_u[n] * s;
            const unsigned hit0 = __ballot_sync(0xffffffffu, ok0 && c0 > thr), hit1 = __ballot_sync(0xffffffffu, ok1 && c1 > thr);
            const unsigned v0 = __ballot_sync(0xffffffffu, ok0), v1 = __ballot_sync(0xffffffffu, ok1);
            int sel;
            if (hit0)
                sel = __ffs(hit0) - 1;
            else if (hit1)
                sel = 32 + __ffs(hit1) - 1;
            else
                sel = v1 ? 32 + (31 - __clz(v1)) : (31 - __clz(v0));  // none: the last remaining candidate
            const double wsel = __shfl_sync(0xffffffffu, sel < 32 ? w0 : w1, sel & 31);
            taken |= 1ull << sel;
            if (lane == 0) {
                tree_tok[(size_t)b * N + n] = sh_id[hd][sel];
                tree_cand[(size_t)b * N + n] = (uint8_t)sel;
                slot_q[(size_t)b * N + n] = (float)(wsel / s);
            }
        }
    }
}

// ------------------------------------------------------------------------------ host side

struct ProposePlan {
    int KX, M, n_mblocks, n_tiles, n_groups, tiles_per_group;
    bool use_tc;  // tcgen05 projection kernel (k <= 8); otherwise the mma.sync one
    size_t off_status, off_xhat, off_z, off_zt, off_pval, off_pid, off_hc, total;
};

// head_mlp_tc.cu
int launch_head_mlp_tc(const void *xhat, int KX, const void *A, const void *bias, const void *h, float *z, int B,
                       int K, int d, int32_t *status, cudaStream_t st);

// lm_head_tc.cu
int launch_lm_head_tc(const void *Zt, const void *W, int M, int V, int d, int k, int n_mblocks, int n_groups,
                      int tiles_per_group, float *pval, int32_t *pid, int32_t *status, cudaStream_t st);

static int make_plan(const specroll_propose_desc *d, bool affine, ProposePlan *p) {
    if (!d || d->B < 0 || d->N < 1 || d->N > SPECROLL_MAX_NODES || d->K < 1 || d->K > SPECROLL_MAX_HEADS ||
        d->k < 1 || d->k > SPECROLL_MAX_TOPK || d->d < 64 || (d->d % 64) || d->V < 8 || (d->V % 8) ||
        d->k > d->V || !(d->temperature > 0.f) || !(d->ln_eps >= 0.f) || !(d->rms_eps >= 0.f) ||
        (d->flags & ~(SPECROLL_PROPOSE_LEGACY_MMA | SPECROLL_REFLEX_PRE_HEAD)) != 0 || d->d > 12288)
        return SPECROLL_EINVAL;
    p->KX = affine ? d->K : 1;
    p->M = d->B * d->K;
    p->use_tc = d->k <= 8 && !(d->flags & SPECROLL_PROPOSE_LEGACY_MMA);
    const int bn = p->use_tc ? 256 : LmTile::BN;
    p->n_mblocks = (p->M + LmTile::BM - 1) / LmTile::BM;  // both kernels use 128-row blocks
    p->n_tiles = (d->V + bn - 1) / bn;
    int want = p->n_mblocks > 0 ? ((p->use_tc ? 1 : 2) * 148) / p->n_mblocks : 1;
    if (want < 1) want = 1;
    if (want > p->n_tiles) want = p->n_tiles;
    p->tiles_per_group = (p->n_tiles + want - 1) / want;
    p->n_groups = (p->n_tiles + p->tiles_per_group - 1) / p->tiles_per_group;
    size_t o = 0;
    const size_t B = d->B, K = d->K, dd = d->d, k = d->k;
    p->off_status = o;
    o += 256;
    p->off_xhat = o;
    o += align_up((size_t)p->KX * B * dd * 2, 256);
    p->off_z = o;
    o += align_up(B * K * dd * 4, 256);
    p->off_zt = o;
    o += align_up(B * K * dd * 2, 256);
    p->off_pval = o;
    o += align_up((size_t)p->M * p->n_groups * k * 4, 256);
    p->off_pid = o;
    o += align_up((size_t)p->M * p->n_groups * k * 4, 256);
    p->off_hc = o;  // the corrected hidden state of the pre-head form
    if (d->flags & SPECROLL_REFLEX_PRE_HEAD) o += align_up(B * dd * 2, 256);
    p->total = o + 256;
    return SPECROLL_OK;
}

template <typename Kern>
static int set_smem(Kern kern, int bytes) {
    SR_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
    return SPECROLL_OK;
}

static int launch_tree_draw(bool pdl, const Topo &topo, int B, int K, int k, float T, const int32_t *anchor,
                            const int32_t *cand_id, const float *cand_logit, const float *u_draw,
                            int32_t *tree_tok, uint8_t *tree_cand, float *slot_q, cudaStream_t st) {
    if (B == 0) return SPECROLL_OK;
    SR_CUDA_TRY(launch_dependent(pdl, tree_draw_kernel, dim3(B), dim3(DRAW_WARPS * 32), 0, st, topo, B, K, k, (double)T, anchor,
                                 cand_id, cand_logit, u_draw, tree_tok, tree_cand, slot_q));
    return SPECROLL_OK;
}

}  // namespace specroll

using namespace specroll;

extern "C" size_t specroll_propose_workspace_bytes(const specroll_propose_desc *d) {
    ProposePlan p;
    if (make_plan(d, true, &p) != SPECROLL_OK) return 0;  // sized for the affine case (the larger one)
    return p.total;
}

extern "C" int specroll_workspace_status(const void *workspace, void *cuda_stream) {
    if (!workspace) return SPECROLL_EINVAL;
    int32_t word = 0;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    SR_CUDA_TRY(cudaMemcpyAsync(&word, workspace, sizeof(word), cudaMemcpyDeviceToHost, st));
    SR_CUDA_TRY(cudaStreamSynchronize(st));
    return word == 0 ? SPECROLL_OK : (int)word;
}

extern "C" int specroll_tree_draw(int32_t B, int32_t N, int32_t K, int32_t k, float temperature,
                                  const int32_t *parent_host, const int32_t *anchor_tok,
                                  const int32_t *cand_id, const float *cand_logit, const float *u_draw,
                                  int32_t *tree_tok, uint8_t *tree_cand, float *slot_q, void *cuda_stream) {
    if (B < 0 || K < 1 || K > SPECROLL_MAX_HEADS || k < 1 || k > SPECROLL_MAX_TOPK || !(temperature > 0.f))
        return SPECROLL_EINVAL;
    Topo topo;
    if (build_topo(parent_host, N, K, k, &topo, nullptr) != SPECROLL_OK) return SPECROLL_EINVAL;
    if (B == 0) return SPECROLL_OK;  // (an empty batch has empty arrays: their pointers may be NULL)
    if (!anchor_tok || !cand_id || !cand_logit || !u_draw || !tree_tok || !tree_cand || !slot_q)
        return SPECROLL_EINVAL;
    return launch_tree_draw(false, topo, B, K, k, temperature, anchor_tok, cand_id, cand_logit, u_draw, tree_tok,
                            tree_cand, slot_q, static_cast<cudaStream_t>(cuda_stream));
}

extern "C" int specroll_propose(const specroll_propose_desc *d, const void *h, const int32_t *anchor_tok,
                                const void *A, const void *bias, const void *ln_gamma, const void *ln_beta,
                                const void *W, const float *m, const float *alpha,
                                const int32_t *parent_host, const float *u_draw, int32_t *cand_id,
                                float *cand_logit, int32_t *tree_tok, uint8_t *tree_cand, float *slot_q,
                                void *workspace, size_t workspace_bytes, void *cuda_stream) {
    ProposePlan p;
    const bool affine = ln_gamma || ln_beta;
    if (make_plan(d, affine, &p) != SPECROLL_OK) return SPECROLL_EINVAL;
    Topo topo;
    if (build_topo(parent_host, d->N, d->K, d->k, &topo, nullptr) != SPECROLL_OK) return SPECROLL_EINVAL;
    if (d->B == 0) return SPECROLL_OK;  // (an empty batch has empty arrays: their pointers may be NULL)
    if (!h || !anchor_tok || !A || !bias || !W || !u_draw || !cand_id || !cand_logit || !tree_tok ||
        !tree_cand || !slot_q)
        return SPECROLL_EINVAL;
    if (!aligned16(h) || !aligned16(A) || !aligned16(bias) || !aligned16(W) || !aligned16(m) ||
        !aligned16(ln_gamma) || !aligned16(ln_beta))
        return SPECROLL_EALIGN;
    if (d->B == 0) return SPECROLL_OK;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) || workspace_bytes < p.total)
        return SPECROLL_EWORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    char *ws = static_cast<char *>(workspace);
    __nv_bfloat16 *xhat = reinterpret_cast<__nv_bfloat16 *>(ws + p.off_xhat);
    float *z = reinterpret_cast<float *>(ws + p.off_z);
    __nv_bfloat16 *zt = reinterpret_cast<__nv_bfloat16 *>(ws + p.off_zt);
    float *pval = reinterpret_cast<float *>(ws + p.off_pval);
    int32_t *pid = reinterpret_cast<int32_t *>(ws + p.off_pid);
    const __nv_bfloat16 *hb = static_cast<const __nv_bfloat16 *>(h);
    const int B = d->B, K = d->K, dd = d->d, k = d->k, V = d->V;
    int32_t *status = reinterpret_cast<int32_t *>(ws + p.off_status);
    SR_CUDA_TRY(cudaMemsetAsync(status, 0, sizeof(int32_t), st));
    const bool pre_head = (d->flags & SPECROLL_REFLEX_PRE_HEAD) != 0;
    if (pre_head) {
        // the correction moves the hidden state itself (m [B, d], alpha [B]); everything after it reads the
        // corrected state, and the heads' outputs are not corrected again
        __nv_bfloat16 *hc = reinterpret_cast<__nv_bfloat16 *>(ws + p.off_hc);
        prehead_kernel<<<B, RX_THREADS, 0, st>>>(hb, m, alpha, hc, dd, d->rms_eps, d->clip_c);
        SR_LAUNCH_CHECK();
        hb = hc;
    }

    // From here on every kernel is launched as the programmatic dependent of the one before it: it may set itself up
    // (barriers, tensor memory, tensor-map prefetch) under the tail of its predecessor and waits for the predecessor's
    // completion before it touches global memory.
    SR_CUDA_TRY(launch_dependent(pre_head, layernorm_kernel, dim3(B), dim3(LN_THREADS), dd * sizeof(float), st, hb,
                                 static_cast<const __nv_bfloat16 *>(ln_gamma), static_cast<const __nv_bfloat16 *>(ln_beta),
                                 xhat, B, dd, p.KX, d->ln_eps));

    if (!(d->flags & SPECROLL_PROPOSE_LEGACY_MMA)) {
        int rc = launch_head_mlp_tc(xhat, p.KX, A, bias, hb, z, B, K, dd, status, st);
        if (rc) return rc;
    } else {
        int rc = set_smem(head_mlp_kernel, HeadTile::SMEM_BYTES);
        if (rc) return rc;
        dim3 grid((dd + HeadTile::BN - 1) / HeadTile::BN, (B + HeadTile::BM - 1) / HeadTile::BM, K);
        head_mlp_kernel<<<grid, HeadTile::THREADS, HeadTile::SMEM_BYTES, st>>>(
            xhat, p.KX, static_cast<const __nv_bfloat16 *>(A), static_cast<const __nv_bfloat16 *>(bias), hb, z,
            B, K, dd);
        SR_LAUNCH_CHECK();
    }

    SR_CUDA_TRY(launch_dependent(true, reflex_kernel, dim3(B * K), dim3(RX_THREADS), 0, st, (const float *)z,
                                 pre_head ? (const float *)nullptr : m, pre_head ? (const float *)nullptr : alpha, zt, dd,
                                 d->rms_eps, d->clip_c));

    {
        const int grid = p.n_mblocks * p.n_groups;
        const int smem = LmTile::SMEM_BYTES;  // >= 128 * 129 * 4 staging tile
        static_assert(LmTile::SMEM_BYTES >= LmTile::BM * LM_CSTRIDE * 4, "staging tile must fit");
        if (p.use_tc) {
            int rc = launch_lm_head_tc(zt, W, p.M, V, dd, k, p.n_mblocks, p.n_groups, p.tiles_per_group, pval, pid,
                                       status, st);
            if (rc) return rc;
        } else if (k <= 8) {
            int rc = set_smem(lm_head_topk_kernel<8>, smem);
            if (rc) return rc;
            lm_head_topk_kernel<8><<<grid, LmTile::THREADS, smem, st>>>(
                zt, static_cast<const __nv_bfloat16 *>(W), p.M, V, dd, k, p.n_mblocks, p.n_groups,
                p.tiles_per_group, pval, pid);
        } else {
            int rc = set_smem(lm_head_topk_kernel<SPECROLL_MAX_TOPK>, smem);
            if (rc) return rc;
            lm_head_topk_kernel<SPECROLL_MAX_TOPK><<<grid, LmTile::THREADS, smem, st>>>(
                zt, static_cast<const __nv_bfloat16 *>(W), p.M, V, dd, k, p.n_mblocks, p.n_groups,
                p.tiles_per_group, pval, pid);
        }
        SR_LAUNCH_CHECK();
    }

    if (k <= 8 && p.n_groups * k >= 256)
        SR_CUDA_TRY(launch_dependent(true, topk_merge8_wide_kernel, dim3(p.M), dim3(MERGE_WIDE_WARPS * 32), 0, st,
                                     (const float *)pval, (const int32_t *)pid, p.M, p.n_groups * k, k, cand_id, cand_logit));
    else
        SR_CUDA_TRY(launch_dependent(true, k <= 8 ? topk_merge8_kernel : topk_merge_kernel, dim3((p.M + 3) / 4), dim3(128), 0,
                                     st, (const float *)pval, (const int32_t *)pid, p.M, p.n_groups * k, k, cand_id,
                                     cand_logit));

    return launch_tree_draw(true, topo, B, K, k, d->temperature, anchor_tok, cand_id, cand_logit, u_draw, tree_tok,
                            tree_cand, slot_q, st);
}
