// Verifier-derived feedback of matured proposals and the trajectory memory update (Sec. 3.3 Eq.
// "acceptance-gap-decomposition"; Sec. 3.4 Eq. "support", "distdir", "covdir", the RMS normalisation, Eq.
// "unified-feedback", Eq. "ema").  Per record (one matured proposal node):
//
//   p = softmax(logits / T) over the vocabulary; q = softmax(cand_logit / T) on the k candidates C
//   S = C  u  Top_kS(p)  u  {y*};   p_S, q_S = p, q renormalised on S (q lives on C, so q_S = q)
//   r_dist = sum_{v in S} (p_S(v) - q_S(v)) W_v
//   C* = Top_k(p),  O = C* \ C,  b* = weakest candidate;   r_cov = sum_{y in O} p_S(y) (W_y - W_b*)
//   d_dist = p(C) TV(p_C, q_C),   d_cov = p(C*) - p(C)
//   rbar = r / (RMS(r) + eps);  g = d_dist rbar_dist + d_cov rbar_cov;  e = (d_dist + d_cov) g / (RMS(g) + eps)
//   m <- rho m + (1 - rho) e
//
// Two kernels, one CTA per record each:
//   feedback_topk_kernel   exact Top_kS of the record's logits row, ordered by (logit desc, id asc), on the 16-bit
//                          order-preserving keys of the bf16 logits.  Two passes: a lower bound of the kS-th largest
//                          key from the threads' own maxima, then the few elements at or above it ranked in shared
//                          memory.  Fallback for rows with thousands of equal large values: a radix search by
//                          COUNT (four bits per pass) for the key of the kS-th largest value, a pass for the ids
//                          above it, an ordered pass for the first ids that tie with it, a rank sort.
//   feedback_vec_kernel    the small quantities (q, p on S, the coefficient of every support row; repeated tokens
//                          found by all threads, the rest by one warp), then the <= k + kS + 1 rows of W come
//                          through shared memory as bulk copies of whole rows, three batches in flight, and the
//                          threads accumulate both directions; three RMS reductions, and the memory update.
//                          (feedback_kernel: hidden sizes not a multiple of 8.)
#include <math.h>

#include <algorithm>

#include "common.cuh"
#include "tc05.cuh"

namespace specroll {

namespace fb {
constexpr int TOPK_THREADS = 512;
constexpr int TOPK_LIST_CAP = 2048;  // candidates of the list method
constexpr int FB_THREADS = 256;
constexpr int MAX_S = 2 * SPECROLL_MAX_TOPK + 1;  // candidates + Top_kS + y*

__device__ __forceinline__ uint32_t ord_key16(uint32_t bits) {
    if (bits == 0x8000u) bits = 0u;  // -0 counts as +0
    return (bits & 0x8000u) ? (~bits & 0xffffu) : (bits | 0x8000u);
}

template <int THREADS>
__device__ __forceinline__ int block_sum_int(int v, int *red) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();
    if (lane == 0) red[warp] = v;
    __syncthreads();
    int t = 0;
    for (int w = 0; w < THREADS / 32; ++w) t += red[w];
    return t;
}

template <int THREADS>
__device__ __forceinline__ float block_sum_f(float v, float *red) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    v = warp_sum(v);
    __syncthreads();
    if (lane == 0) red[warp] = v;
    __syncthreads();
    float t = 0.f;
    for (int w = 0; w < THREADS / 32; ++w) t += red[w];
    return t;
}
// the same for a CTA of any whole number of warps
__device__ __forceinline__ float block_sum_rt(float v, float *red) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
    v = warp_sum(v);
    __syncthreads();
    if (lane == 0) red[warp] = v;
    __syncthreads();
    float t = 0.f;
    for (int w = 0; w < nw; ++w) t += red[w];
    return t;
}
}  // namespace fb

// Shared memory of the top-k kernel: the list method and the radix fallback never run at the same time.
struct TopkRadixSmem {
    int bins[16][fb::TOPK_THREADS];
    int wsum[fb::TOPK_THREADS / 32][16];
    int red[fb::TOPK_THREADS / 32];
    int sel_id[SPECROLL_MAX_TOPK];
    uint32_t sel_key[SPECROLL_MAX_TOPK];
};
struct TopkListSmem {
    uint32_t best[fb::TOPK_THREADS];     // every thread's largest key
    // candidates (elements at or above the bound): key in the upper word, the complement of the id in the lower one,
    // so that "larger" is (key desc, id asc) and a rank is a count of one comparison per entry
    unsigned long long ent[fb::TOPK_LIST_CAP];
};

// Exact Top_kS by a radix search over the counts (any row, also one with tens of thousands of equal values);
// the fallback of the list method below.  top_id[0..kS): ids by (logit desc, id asc).
__device__ void topk_radix(TopkRadixSmem &sm, int &sh_above, int &sh_prefix, int &sh_n, const uint4 *__restrict__ p,
                           int nvec, int V, int kS, int32_t *__restrict__ top_id) {
    using namespace fb;
    auto &bins = sm.bins;
    auto &wsum = sm.wsum;
    auto &red = sm.red;
    auto &sel_id = sm.sel_id;
    auto &sel_key = sm.sel_key;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // ---- key of the kS-th largest value: four radix passes over the counts
    for (int level = 0; level < 4; ++level) {
        const int shift = 12 - 4 * level;
        const uint32_t prefix = (uint32_t)sh_prefix;
#pragma unroll
        for (int j = 0; j < 16; ++j) bins[j][tid] = 0;
        for (int i = tid; i < nvec; i += TOPK_THREADS) {
            const uint4 v = ld_nc_v4(p + i);
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int t = 0; t < 8; ++t) {
                const uint32_t key = ord_key16((t & 1) ? (w[t >> 1] >> 16) : (w[t >> 1] & 0xffffu));
                if (level == 0 || (key >> (shift + 4)) == prefix) bins[(key >> shift) & 15u][tid] += 1;
            }
        }
#pragma unroll
        for (int j = 0; j < 16; ++j) {
            int x = bins[j][tid];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
            if (lane == 0) wsum[warp][j] = x;
        }
        __syncthreads();
        if (tid == 0) {
            int cum = sh_above, sel = 0;
            for (int j = 15; j >= 0; --j) {
                int tot = 0;
                for (int w2 = 0; w2 < TOPK_THREADS / 32; ++w2) tot += wsum[w2][j];
                if (cum + tot >= kS) {  // the kS-th largest has this digit
                    sel = j;
                    break;
                }
                cum += tot;
                sel = j;  // (fewer than kS values in the row: ends at the lowest digit)
            }
            sh_above = cum;  // values whose key is larger than every key with this prefix
            sh_prefix = (int)((prefix << 4) | (uint32_t)sel);
        }
        __syncthreads();
    }
    const uint32_t thr = (uint32_t)sh_prefix;
    const int n_above = sh_above;           // keys strictly above the threshold key: all of them are winners
    const int need = max(0, kS - n_above);  // winners among the ties, lowest ids first
    // ---- winners above the threshold (any order; sorted below)
    for (int i = tid; i < nvec; i += TOPK_THREADS) {
        const uint4 v = ld_nc_v4(p + i);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int t = 0; t < 8; ++t) {
            const uint32_t key = ord_key16((t & 1) ? (w[t >> 1] >> 16) : (w[t >> 1] & 0xffffu));
            if (key > thr) {
                const int pos = atomicAdd(&sh_n, 1);
                if (pos < SPECROLL_MAX_TOPK) {
                    sel_id[pos] = i * 8 + t;
                    sel_key[pos] = key;
                }
            }
        }
    }
    __syncthreads();
    // ---- the first `need` ties in id order: every thread takes a contiguous piece of the row
    {
        const int per = (nvec + TOPK_THREADS - 1) / TOPK_THREADS;
        const int lo = min(nvec, tid * per), hi = min(nvec, lo + per);
        int cnt = 0;
        for (int i = lo; i < hi; ++i) {
            const uint4 v = ld_nc_v4(p + i);
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int t = 0; t < 8; ++t)
                cnt += ord_key16((t & 1) ? (w[t >> 1] >> 16) : (w[t >> 1] & 0xffffu)) == thr;
        }
        // exclusive prefix of the counts over the threads
        int incl = cnt;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int x = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += x;
        }
        if (lane == 31) red[warp] = incl;
        __syncthreads();
        int base = 0;
        for (int w2 = 0; w2 < warp; ++w2) base += red[w2];
        int rank = base + incl - cnt;  // ties before this thread's piece
        if (cnt > 0 && rank < need) {
            for (int i = lo; i < hi && rank < need; ++i) {
                const uint4 v = ld_nc_v4(p + i);
                const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                for (int t = 0; t < 8; ++t) {
                    if (rank < need && ord_key16((t & 1) ? (w[t >> 1] >> 16) : (w[t >> 1] & 0xffffu)) == thr) {
                        const int pos = n_above + rank;
                        if (pos < SPECROLL_MAX_TOPK) {
                            sel_id[pos] = i * 8 + t;
                            sel_key[pos] = thr;
                        }
                        ++rank;
                    }
                }
            }
        }
    }
    __syncthreads();
    // ---- order the winners by (key desc, id asc)
    const int n_sel = min(kS, min(V, SPECROLL_MAX_TOPK));
    if (tid < n_sel) {
        const uint32_t ki = sel_key[tid];
        const int ii = sel_id[tid];
        int rk = 0;
        for (int j = 0; j < n_sel; ++j) rk += (sel_key[j] > ki) || (sel_key[j] == ki && sel_id[j] < ii);
        top_id[rk] = ii;
    }
}

// top_id[r, 0..kS): ids of the kS largest logits of row rec_row[r], by (logit desc, id asc).
// List method, two passes over the row: (1) every thread finds the largest key of its strided share of the row; the
// kS-th largest of those 512 values is a lower bound of the kS-th largest key of the row (there are at least kS
// elements at or above it); (2) the elements at or above the bound, a few more than kS unless the large values
// sit in few threads' shares, go into a list in shared memory, and an entry's rank in the list by (key desc, id
// asc) is its place in the result.  A list longer than its capacity (a row with thousands of equal large values)
// falls back to the radix search.
__global__ void __launch_bounds__(fb::TOPK_THREADS)
feedback_topk_kernel(const uint16_t *__restrict__ logits, const int32_t *__restrict__ rec_row, int V, int kS,
                     int32_t *__restrict__ top_id) {
    using namespace fb;
    __shared__ union {
        TopkRadixSmem radix;
        TopkListSmem list;
    } sm;
    __shared__ int sh_above, sh_prefix, sh_n;
    __shared__ uint32_t sh_bound;
    const int r = blockIdx.x, tid = threadIdx.x;
    const uint16_t *row = logits + (size_t)rec_row[r] * V;
    const uint4 *p = reinterpret_cast<const uint4 *>(row);
    const int nvec = V >> 3;
    int32_t *out = top_id + (size_t)r * kS;
    const int n_sel = min(kS, V);
    if (tid == 0) sh_n = 0;
    // ---- pass 1: the largest key of this thread's share.  The order of the keys is the order of the values (with
    //      -0 = +0), so the maximum is taken on the bf16 pairs as they come, one instruction per two logits, and
    //      turned into a key once.
    auto as_bf162 = [](uint32_t w_) { return *reinterpret_cast<const __nv_bfloat162 *>(&w_); };
    __nv_bfloat162 mx2 = as_bf162(0xff80ff80u);  // (-inf, -inf)
    // (Taking the bound from the head of the row only, to read the row once, was tried: the bound is lower, the list
    // several hundred entries long, and ranking it costs more than the second pass over a row that sits in L2.)
    const int nvec1 = nvec;
    for (int i = tid; i < nvec1; i += 4 * TOPK_THREADS) {  // four loads in flight per thread
        uint4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int iu = i + u * TOPK_THREADS;
            v[u] = iu < nvec1 ? ld_nc_v4(p + iu) : make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u)
            mx2 = __hmax2(__hmax2(__hmax2(as_bf162(v[u].x), as_bf162(v[u].y)), __hmax2(as_bf162(v[u].z), as_bf162(v[u].w))), mx2);
    }
    const uint32_t mxb = *reinterpret_cast<const uint32_t *>(&mx2);
    const uint32_t best = max(ord_key16(mxb & 0xffffu), ord_key16(mxb >> 16));
    sm.list.best[tid] = best;
    __syncthreads();
    {
        // the n_sel-th largest of the threads' values (ties broken by thread index: any of them will do as the bound)
        // (compared as (value, thread) pairs in one word; the loads do not depend on the count: unrolled)
        const uint32_t mine = (best << 10) | (uint32_t)(TOPK_THREADS - 1 - tid);
        int rk = 0;
#pragma unroll 8
        for (int j = 0; j < TOPK_THREADS; ++j) rk += ((sm.list.best[j] << 10) | (uint32_t)(TOPK_THREADS - 1 - j)) > mine;
        if (rk == min(n_sel, TOPK_THREADS) - 1) sh_bound = best;
    }
    __syncthreads();
    const uint32_t bound = sh_bound;
    // ---- pass 2: everything at or above the bound.  Compared as values, two at a time, against the bound's
    //      value; a vector of eight with nothing to keep (nearly all of them) costs four compares and one branch.
    const uint32_t bbits = (bound & 0x8000u) ? (bound & 0x7fffu) : (~bound & 0xffffu);  // the key undone
    const __nv_bfloat162 bnd2 = as_bf162(bbits | (bbits << 16));
    for (int i0 = tid; i0 < nvec; i0 += 8 * TOPK_THREADS) {  // eight loads in flight per thread
        uint4 vv[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int iu = i0 + u * TOPK_THREADS;
            vv[u] = iu < nvec ? ld_nc_v4(p + iu) : make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u);
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int i = i0 + u * TOPK_THREADS;
            if (i >= nvec) continue;  // (a -inf filler would pass a bound of -inf)
            const uint32_t w[4] = {vv[u].x, vv[u].y, vv[u].z, vv[u].w};
            uint32_t m[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) m[j] = __hge2_mask(as_bf162(w[j]), bnd2);
            if ((m[0] | m[1] | m[2] | m[3]) == 0u) continue;
#pragma unroll
            for (int t = 0; t < 8; ++t) {
                if ((m[t >> 1] >> (16 * (t & 1))) & 0xffffu) {
                    const uint32_t key = ord_key16((t & 1) ? (w[t >> 1] >> 16) : (w[t >> 1] & 0xffffu));
                    const int pos = atomicAdd(&sh_n, 1);
                    if (pos < TOPK_LIST_CAP)
                        sm.list.ent[pos] = ((unsigned long long)key << 32) | (uint32_t)(0x7fffffff - (i * 8 + t));
                }
            }
        }
    }
    __syncthreads();
    const int n = sh_n;
    if (n > TOPK_LIST_CAP || n < n_sel) {  // (n < n_sel cannot happen; the radix search is exact for every row)
        __syncthreads();
        if (tid == 0) {
            sh_above = 0;
            sh_prefix = 0;
            sh_n = 0;
        }
        __syncthreads();
        topk_radix(sm.radix, sh_above, sh_prefix, sh_n, p, nvec, V, kS, out);
        return;
    }
    // ---- rank within the list
    for (int e = tid; e < n; e += TOPK_THREADS) {
        const unsigned long long me = sm.list.ent[e];
        int rk = 0;
#pragma unroll 8
        for (int j = 0; j < n; ++j) rk += sm.list.ent[j] > me;
        if (rk < n_sel) out[rk] = 0x7fffffff - (int)(uint32_t)(me & 0xffffffffull);
    }
}

struct FeedbackArgs {
    const uint16_t *logits;
    const int32_t *rec_row;
    const float *row_max, *row_sum;
    const int32_t *cand_id;
    const float *cand_logit;
    const int32_t *y_star;
    const __nv_bfloat16 *W;
    const float *rho;
    const int32_t *rec_mem;
    const int32_t *top_id;
    float *m;
    float *d_dist, *d_cov, *tv;
    float *severity, *e_out;  // optional outputs: w per record, the feedback vector e per record
    int R, k, kS, d, V;
    float inv_T, eps;
    int rows_per_stage;  // (vector kernel) support rows of W per batch in shared memory
    int weighted;        // the update is weighted by the severity, records below severity_min are discarded
    float severity_min;
};

// The small quantities of one record, in shared memory.
struct FeedbackSmall {
    int id[fb::MAX_S];
    float p[fb::MAX_S];      // target mass exp((l - M)/T) / row_sum of the support tokens
    float adist[fb::MAX_S];  // coefficient of W_v in r_dist
    float acov[fb::MAX_S];   // coefficient of W_v in r_cov
    float q[SPECROLL_MAX_TOPK];
    int raw_id[fb::MAX_S];   // C, Top_kS, y* as they come (with duplicates)
    float raw_p[fb::MAX_S];
    int first[fb::MAX_S];    // raw index of the first occurrence of the same token (-1: not a token of the vocabulary)
    int where[fb::MAX_S];    // the raw entry's place in S (-1: none)
    int n;
    float dd, dc, w;
};

// q, p on S, the coefficient of every support row, the scalar outputs.  All threads fetch the ids and the target
// logits at them (two rounds of independent loads); one warp does the rest from shared memory.  Ends with a barrier.
__device__ void feedback_small(const FeedbackArgs &a, int r, FeedbackSmall &s) {
    using namespace fb;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int k = a.k, kS = a.kS;
    const size_t row = (size_t)a.rec_row[r];
    const uint16_t *lg = a.logits + row * a.V;
    const float M = a.row_max[row], Ssum = a.row_sum[row];
    const int32_t *cid = a.cand_id + (size_t)r * k;
    const float *cl = a.cand_logit + (size_t)r * k;
    const int32_t *top = a.top_id + (size_t)r * kS;
    const int n_raw = k + kS + 1;
    for (int i = tid; i < n_raw; i += blockDim.x) {
        const int v = i < k ? cid[i] : (i < k + kS ? top[i - k] : a.y_star[r]);
        s.raw_id[i] = v;
        s.raw_p[i] = (v >= 0 && v < a.V) ? __expf((__uint_as_float((uint32_t)lg[v] << 16) - M) * a.inv_T) / Ssum : 0.f;
        s.first[i] = (v >= 0 && v < a.V) ? i : -1;
    }
    __syncthreads();
    // the first occurrence of every token in the concatenation: all pairs (i, j < i), spread over the CTA (matches
    // are rare: a candidate that is also among the target's largest, y* among either)
    for (int pp = tid; pp < n_raw * 64; pp += blockDim.x) {
        const int i = pp >> 6;
        for (int j = pp & 63; j < i; j += 64)
            if (s.raw_id[j] == s.raw_id[i] && s.first[i] >= 0) atomicMin(&s.first[i], j);
    }
    __syncthreads();
    if (warp == 0) {
        // ---- q on the candidates
        float mx = -INFINITY;
        for (int j = lane; j < k; j += 32) mx = fmaxf(mx, cl[j]);
        mx = warp_max(mx);
        float qs = 0.f;
        for (int j = lane; j < k; j += 32) {
            const float w = __expf((cl[j] - mx) * a.inv_T);
            s.q[j] = w;
            qs += w;
        }
        qs = warp_sum(qs);
        __syncwarp();
        for (int j = lane; j < k; j += 32) s.q[j] /= qs;
        // ---- S = C u Top_kS u {y*}, duplicates removed (first occurrence kept; the candidates come first)
        if (lane == 0) s.n = 0;
        __syncwarp();
        for (int i0 = 0; i0 < n_raw; i0 += 32) {
            const int i = i0 + lane;
            const int v = i < n_raw ? s.raw_id[i] : -1;
            const bool fresh = i < n_raw && s.first[i] == i;
            const unsigned bal = __ballot_sync(0xffffffffu, fresh);
            const int base = s.n;
            if (fresh) {
                const int pos = base + __popc(bal & ((1u << lane) - 1u));
                s.id[pos] = v;
                s.p[pos] = s.raw_p[i];
                s.where[i] = pos;
            }
            __syncwarp();
            if (lane == 0) s.n = base + __popc(bal);
            __syncwarp();
        }
        const int n = s.n;
        for (int i = lane; i < n_raw; i += 32) {  // repeated tokens: the place of their first occurrence
            const int f = s.first[i];
            if (f != i) s.where[i] = f < 0 ? -1 : s.where[f];
        }
        __syncwarp();
        // ---- masses: p(S), p(C), p(C*); TV on C
        float pS = 0.f;
        for (int i = lane; i < n; i += 32) pS += s.p[i];
        pS = warp_sum(pS);
        float pC = 0.f;
        for (int j = lane; j < k; j += 32) pC += s.p[j];  // the first k support entries are the candidates
        pC = warp_sum(pC);
        float tvs = 0.f;
        for (int j = lane; j < k; j += 32) tvs += fabsf(s.p[j] / pC - s.q[j]);
        tvs = 0.5f * warp_sum(tvs);
        // C* = the first k of Top_kS; O = C* \ C
        float pCs = 0.f, cov_b = 0.f;
        for (int i = lane; i < n; i += 32) s.acov[i] = 0.f;
        __syncwarp();
        for (int t = lane; t < k; t += 32) {
            const float pv = s.raw_p[k + t];
            pCs += pv;
            const int f = s.first[k + t];
            const bool inC = f >= 0 && f < k;  // (first seen among the candidates, which come first)
            if (!inC) {
                // an omitted target-important token: +p_S(y) on its own row, -p_S(y) on the weakest candidate's
                const int pos = s.where[k + t];
                if (pos >= k) s.acov[pos] = pv / pS;
                cov_b += pv / pS;
            }
        }
        pCs = warp_sum(pCs);
        cov_b = warp_sum(cov_b);
        __syncwarp();
        float tvS = 0.f;  // TV(p_S, q_S)
        for (int i = lane; i < n; i += 32) {
            const float ad = s.p[i] / pS - (i < k ? s.q[i] : 0.f);
            s.adist[i] = ad;
            tvS += fabsf(ad);
        }
        tvS = 0.5f * warp_sum(tvS);
        if (lane == 0) {
            // severity of the observation: w = clip(0.3 TV(p_S, q_S) + 0.7 p_out, 0, 1), p_out = 1 - p(C)
            const float w = fminf(1.f, fmaxf(0.f, 0.3f * tvS + 0.7f * (1.f - pC)));
            s.w = w;
            if (a.severity) a.severity[r] = w;
            s.acov[k - 1] -= cov_b;  // b* = last candidate (the list is sorted by logit)
            const float dd = pC * tvs, dc = pCs - pC;
            s.dd = dd;
            s.dc = dc;
            if (a.d_dist) a.d_dist[r] = dd;
            if (a.d_cov) a.d_cov[r] = dc;
            if (a.tv) a.tv[r] = tvs;
        }
    }
    __syncthreads();
}

// Hidden sizes that are not a multiple of eight: thread t owns columns t, t + 256, ...
// MAXC = columns of the hidden dimension per thread (d <= 256 * MAXC)
template <int MAXC>
__global__ void __launch_bounds__(fb::FB_THREADS) feedback_kernel(FeedbackArgs a) {
    using namespace fb;
    __shared__ FeedbackSmall sm;
    __shared__ float red[FB_THREADS / 32];
    const int r = blockIdx.x, tid = threadIdx.x;
    const int d = a.d;
    feedback_small(a, r, sm);
    const int *s_id = sm.id;
    const float *s_adist = sm.adist, *s_acov = sm.acov;
    const int s_n = sm.n;
    const float s_dd = sm.dd, s_dc = sm.dc, s_w = sm.w;
    const int n = s_n;
    const float dd = s_dd, dc = s_dc;
    // ---- both directions: thread t owns columns t, t + 256, ...; the support rows of W are read once
    float rd[MAXC], rc[MAXC];
    const int ncol = (d + FB_THREADS - 1) / FB_THREADS;
#pragma unroll
    for (int c = 0; c < MAXC; ++c) rd[c] = rc[c] = 0.f;
    for (int i = 0; i < n; ++i) {
        const __nv_bfloat16 *wr = a.W + (size_t)s_id[i] * d;
        const float ad = s_adist[i], ac = s_acov[i];
#pragma unroll
        for (int c = 0; c < MAXC; ++c) {
            const int col = tid + c * FB_THREADS;
            if (c < ncol && col < d) {
                const float w = __bfloat162float(wr[col]);
                rd[c] = fmaf(ad, w, rd[c]);
                rc[c] = fmaf(ac, w, rc[c]);
            }
        }
    }
    float sd = 0.f, scv = 0.f;
#pragma unroll
    for (int c = 0; c < MAXC; ++c) {
        sd += rd[c] * rd[c];
        scv += rc[c] * rc[c];
    }
    sd = block_sum_f<FB_THREADS>(sd, red);
    scv = block_sum_f<FB_THREADS>(scv, red);
    const float fd = dd / (sqrtf(sd / d) + a.eps), fc = dc / (sqrtf(scv / d) + a.eps);
    float sg = 0.f;
#pragma unroll
    for (int c = 0; c < MAXC; ++c) {
        rd[c] = fd * rd[c] + fc * rc[c];  // g
        sg += rd[c] * rd[c];
    }
    sg = block_sum_f<FB_THREADS>(sg, red);
    const float fe = (dd + dc) / (sqrtf(sg / d) + a.eps);
    const float rho = a.rho[r];
    const float w = s_w;
    const bool keep = !a.weighted || w >= a.severity_min;
    const float gain = (1.f - rho) * (a.weighted ? w : 1.f);
    float *mr = a.m + (size_t)a.rec_mem[r] * d;
    float *er = a.e_out ? a.e_out + (size_t)r * d : nullptr;
#pragma unroll
    for (int c = 0; c < MAXC; ++c) {
        const int col = tid + c * FB_THREADS;
        if (c < ncol && col < d) {
            const float e = fe * rd[c];
            if (er) er[col] = e;
            if (keep) mr[col] = rho * mr[col] + gain * e;
        }
    }
}

// Hidden sizes that are a multiple of eight.  The support rows of W come through shared memory in batches of rps
// rows, three batches deep, as bulk copies of whole rows issued by one thread and counted on an mbarrier per stage
// (asynchronous copies issued by all threads cost more instructions in address arithmetic than the sums they feed).
// A row is nvec 8-column vectors.  When a row is shorter than the CTA (NV = 1), the threads form groups of nvec,
// group g takes rows g, g + groups, ... of every batch, and the groups' partial sums are added through shared
// memory at the end; otherwise the CTA has ceil(nvec / NV) threads (rounded up to whole warps) and thread t owns
// the vectors t, t + blockDim, ... (NV of them) of every row.
constexpr int FBV_THREADS = 512;
constexpr int FBV_STAGES = 3;

// Row groups of the vector kernel: as many as fit the CTA, at most one per row of a batch.
__host__ __device__ inline int fbv_groups(int d, int rows_per_stage) {
    const int nvec = d >> 3;
    if (nvec >= FBV_THREADS) return 1;
    const int g = FBV_THREADS / nvec;
    return g < rows_per_stage ? g : rows_per_stage;
}
// Threads of the vector kernel's CTA for hidden size d with NV vectors per thread.
__host__ __device__ inline int fbv_threads(int d, int NV) {
    const int nvec = d >> 3;
    if (NV == 1) return FBV_THREADS;
    return ((nvec + NV - 1) / NV + 31) / 32 * 32;
}

__device__ __forceinline__ void fbv_bulk_row(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}

template <int NV>
__global__ void __launch_bounds__(FBV_THREADS, NV == 1 ? 3 : (NV == 2 ? 2 : 1)) feedback_vec_kernel(FeedbackArgs a) {
    using namespace fb;
    __shared__ FeedbackSmall sm;
    __shared__ float red[FBV_THREADS / 32];
    __shared__ __align__(8) unsigned long long full[FBV_STAGES];
    __shared__ volatile int abort_flag;
    extern __shared__ __align__(16) unsigned char fb_stage[];  // [3][rows_per_stage][d] bf16; then the groups' partial sums
    const int r = blockIdx.x, tid = threadIdx.x, tpb = blockDim.x;
    const int d = a.d, nvec = d >> 3;
    if (tid == 0) {
        for (int s = 0; s < FBV_STAGES; ++s) mbar_init(smem_u32(&full[s]), 1);
        abort_flag = 0;
        fence_mbar_init();
    }
    feedback_small(a, r, sm);  // (ends with a barrier)
    const int n = sm.n;
    const float dd = sm.dd, dc = sm.dc, sev = sm.w;
    const int *sh_id = sm.id;
    const float *sh_ad = sm.adist, *sh_ac = sm.acov;
    float rd[NV][8], rc[NV][8];
#pragma unroll
    for (int c = 0; c < NV; ++c)
#pragma unroll
        for (int t = 0; t < 8; ++t) rd[c][t] = rc[c][t] = 0.f;
    const int rps = a.rows_per_stage;
    const uint32_t row_bytes = (uint32_t)d * 2u;
    const size_t stage_bytes = (size_t)rps * row_bytes;
    const int nb = (n + rps - 1) / rps;
    const int groups = NV == 1 ? fbv_groups(d, rps) : 1;
    const int grp = NV == 1 ? tid / nvec : 0, vi0 = NV == 1 ? tid - grp * nvec : tid;
    auto issue = [&](int batch) {  // one thread
        const int s = batch % FBV_STAGES;
        const int rows = min(rps, n - batch * rps);
        const uint32_t bar = smem_u32(&full[s]);
        mbar_arrive_expect_tx(bar, (uint32_t)rows * row_bytes);
        const uint32_t dst = smem_u32(fb_stage + (size_t)s * stage_bytes);
        for (int q = 0; q < rows; ++q)
            fbv_bulk_row(dst + (uint32_t)q * row_bytes, a.W + (size_t)sh_id[batch * rps + q] * d, row_bytes, bar);
    };
    if (tid == 0)
        for (int b = 0; b < FBV_STAGES && b < nb; ++b) issue(b);
    bool ok = true;
    for (int b = 0; b < nb; ++b) {
        ok = mbar_wait(smem_u32(&full[b % FBV_STAGES]), (uint32_t)(b / FBV_STAGES) & 1u, &abort_flag);
        if (ok && grp < groups) {
            const unsigned char *src = fb_stage + (size_t)(b % FBV_STAGES) * stage_bytes;
            const int rows = min(rps, n - b * rps);
            for (int q = grp; q < rows; q += groups) {
                const int i = b * rps + q;
                const float ad = sh_ad[i], ac = sh_ac[i];
#pragma unroll
                for (int c = 0; c < NV; ++c) {
                    const int vi = vi0 + c * tpb;
                    if (vi < nvec) {
                        const uint4 v = *reinterpret_cast<const uint4 *>(src + ((size_t)q * nvec + vi) * 16);
                        const uint32_t w4[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                        for (int t = 0; t < 4; ++t) {
                            const float lo = __uint_as_float(w4[t] << 16), hi = __uint_as_float(w4[t] & 0xffff0000u);
                            rd[c][2 * t] = fmaf(ad, lo, rd[c][2 * t]);
                            rd[c][2 * t + 1] = fmaf(ad, hi, rd[c][2 * t + 1]);
                            rc[c][2 * t] = fmaf(ac, lo, rc[c][2 * t]);
                            rc[c][2 * t + 1] = fmaf(ac, hi, rc[c][2 * t + 1]);
                        }
                    }
                }
            }
        }
        // the stage is free for the batch three further on; a wait that ran out ends the record for every thread
        if (__syncthreads_or(!ok)) {
            ok = false;
            break;
        }
        if (tid == 0 && b + FBV_STAGES < nb) {
            fence_proxy_async();  // the stage's readers are done (barrier above) before the copy engine writes it again
            issue(b + FBV_STAGES);
        }
    }
    if (!ok) {
        // (cannot happen with valid arguments: a bulk copy of a readable row always completes; the record is marked
        // instead of left looking valid, and the memory is not touched)
        if (tid == 0) {
            if (a.d_dist) a.d_dist[r] = nanf("");
            if (a.d_cov) a.d_cov[r] = nanf("");
        }
        return;
    }
    if (NV == 1 && groups > 1) {
        // add the groups' partial sums: group g > 0 leaves its 16 numbers, group 0 collects
        float *part = reinterpret_cast<float *>(fb_stage);  // [groups - 1][16][nvec]; the stages are free now
        if (grp > 0 && grp < groups) {
#pragma unroll
            for (int t = 0; t < 8; ++t) {
                part[((size_t)(grp - 1) * 16 + t) * nvec + vi0] = rd[0][t];
                part[((size_t)(grp - 1) * 16 + 8 + t) * nvec + vi0] = rc[0][t];
                rd[0][t] = rc[0][t] = 0.f;
            }
        }
        __syncthreads();
        if (grp == 0) {
            for (int g = 1; g < groups; ++g)
#pragma unroll
                for (int t = 0; t < 8; ++t) {
                    rd[0][t] += part[((size_t)(g - 1) * 16 + t) * nvec + vi0];
                    rc[0][t] += part[((size_t)(g - 1) * 16 + 8 + t) * nvec + vi0];
                }
        }
    }
    // (from here on only the threads with vectors of their own hold anything but zeros)
    float sd = 0.f, scv = 0.f;
#pragma unroll
    for (int c = 0; c < NV; ++c)
#pragma unroll
        for (int t = 0; t < 8; ++t) {
            sd += rd[c][t] * rd[c][t];
            scv += rc[c][t] * rc[c][t];
        }
    sd = block_sum_rt(sd, red);
    scv = block_sum_rt(scv, red);
    const float fd = dd / (sqrtf(sd / d) + a.eps), fc = dc / (sqrtf(scv / d) + a.eps);
    float sg = 0.f;
#pragma unroll
    for (int c = 0; c < NV; ++c)
#pragma unroll
        for (int t = 0; t < 8; ++t) {
            rd[c][t] = fd * rd[c][t] + fc * rc[c][t];  // g
            sg += rd[c][t] * rd[c][t];
        }
    sg = block_sum_rt(sg, red);
    const float fe = (dd + dc) / (sqrtf(sg / d) + a.eps);
    const float rho = a.rho[r];
    const bool keep = !a.weighted || sev >= a.severity_min;
    const float gain = (1.f - rho) * (a.weighted ? sev : 1.f);
    float4 *mr = reinterpret_cast<float4 *>(a.m + (size_t)a.rec_mem[r] * d);
    float4 *er = a.e_out ? reinterpret_cast<float4 *>(a.e_out + (size_t)r * d) : nullptr;
    const bool owner = NV > 1 || grp == 0;
#pragma unroll
    for (int c = 0; c < NV; ++c) {
        const int vi = vi0 + c * tpb;
        if (owner && vi < nvec) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const float4 e = make_float4(fe * rd[c][4 * h], fe * rd[c][4 * h + 1], fe * rd[c][4 * h + 2], fe * rd[c][4 * h + 3]);
                if (er) er[2 * vi + h] = e;
                if (keep) {
                    float4 mv = mr[2 * vi + h];
                    mv.x = rho * mv.x + gain * e.x;
                    mv.y = rho * mv.y + gain * e.y;
                    mv.z = rho * mv.z + gain * e.z;
                    mv.w = rho * mv.w + gain * e.w;
                    mr[2 * vi + h] = mv;
                }
            }
        }
    }
}

}  // namespace specroll

using namespace specroll;

static int check_feedback_desc(const specroll_feedback_desc *d) {
    if (!d || d->R < 0 || d->k < 1 || d->k > SPECROLL_MAX_TOPK || d->k_support < d->k ||
        d->k_support > SPECROLL_MAX_TOPK || d->d < 8 || d->d > 12288 || d->V < 8 || (d->V % 8) || d->k_support > d->V ||
        !(d->temperature > 0.f) || !(d->eps >= 0.f) || (d->flags & ~SPECROLL_FEEDBACK_SEVERITY) != 0 ||
        ((d->flags & SPECROLL_FEEDBACK_SEVERITY) && !(d->severity_min >= 0.f)))
        return SPECROLL_EINVAL;
    return SPECROLL_OK;
}

extern "C" size_t specroll_reflex_feedback_workspace_bytes(const specroll_feedback_desc *d) {
    if (check_feedback_desc(d) != SPECROLL_OK) return 0;
    return align_up((size_t)d->R * d->k_support * sizeof(int32_t), 256) + 256;
}

extern "C" int specroll_reflex_feedback(const specroll_feedback_desc *d, const void *logits, const int32_t *rec_row,
                                        const float *row_max, const float *row_sum, const int32_t *cand_id,
                                        const float *cand_logit, const int32_t *y_star, const void *W,
                                        const float *rho, const int32_t *rec_mem, float *m, float *d_dist,
                                        float *d_cov, float *tv, void *workspace, size_t workspace_bytes,
                                        void *cuda_stream) {
    return specroll_reflex_feedback_ex(d, logits, rec_row, row_max, row_sum, cand_id, cand_logit, y_star, W, rho, rec_mem,
                                       m, d_dist, d_cov, tv, nullptr, nullptr, workspace, workspace_bytes, cuda_stream);
}

extern "C" int specroll_reflex_feedback_ex(const specroll_feedback_desc *d, const void *logits, const int32_t *rec_row,
                                           const float *row_max, const float *row_sum, const int32_t *cand_id,
                                           const float *cand_logit, const int32_t *y_star, const void *W,
                                           const float *rho, const int32_t *rec_mem, float *m, float *d_dist,
                                           float *d_cov, float *tv, float *severity, float *e_out, void *workspace,
                                           size_t workspace_bytes, void *cuda_stream) {
    if (check_feedback_desc(d) != SPECROLL_OK) return SPECROLL_EINVAL;
    if (d->R == 0) return SPECROLL_OK;  // (no records: the per-record arrays are empty and may be NULL)
    if (!logits || !rec_row || !row_max || !row_sum || !cand_id || !cand_logit || !y_star || !W || !rho || !rec_mem || !m)
        return SPECROLL_EINVAL;
    if (!aligned16(logits) || !aligned16(W)) return SPECROLL_EALIGN;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) ||
        workspace_bytes < specroll_reflex_feedback_workspace_bytes(d))
        return SPECROLL_EWORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int32_t *top_id = static_cast<int32_t *>(workspace);
    feedback_topk_kernel<<<d->R, fb::TOPK_THREADS, 0, st>>>(static_cast<const uint16_t *>(logits), rec_row, d->V,
                                                            d->k_support, top_id);
    SR_LAUNCH_CHECK();
    FeedbackArgs a;
    a.logits = static_cast<const uint16_t *>(logits);
    a.rec_row = rec_row;
    a.row_max = row_max;
    a.row_sum = row_sum;
    a.cand_id = cand_id;
    a.cand_logit = cand_logit;
    a.y_star = y_star;
    a.W = static_cast<const __nv_bfloat16 *>(W);
    a.rho = rho;
    a.rec_mem = rec_mem;
    a.top_id = top_id;
    a.m = m;
    a.d_dist = d_dist;
    a.d_cov = d_cov;
    a.tv = tv;
    a.severity = severity;
    a.e_out = e_out;
    a.weighted = (d->flags & SPECROLL_FEEDBACK_SEVERITY) ? 1 : 0;
    a.severity_min = d->severity_min;
    a.R = d->R;
    a.k = d->k;
    a.kS = d->k_support;
    a.d = d->d;
    a.V = d->V;
    a.inv_T = 1.0f / d->temperature;
    a.eps = d->eps;
    // (m and e_out rows start at multiples of d floats: 16-byte aligned when d % 8 == 0 and the bases are)
    // (bulk copies of W rows: 16-byte aligned rows)
    const bool vec = (d->d % 8) == 0 && aligned16(m) && (!e_out || aligned16(e_out)) && aligned16(W);
    // batches of at most 20 KB of W rows, three deep: three CTAs fit an SM
    a.rows_per_stage = std::max(1, std::min(8, 20480 / (d->d * 2)));
    const size_t fb_smem =
        std::max((size_t)FBV_STAGES * a.rows_per_stage * d->d * 2,
                 (size_t)(fbv_groups(d->d, a.rows_per_stage) - 1) * 16 * (size_t)(d->d >> 3) * sizeof(float));
    if (vec) {
        const void *kern = d->d <= 8 * FBV_THREADS    ? reinterpret_cast<const void *>(feedback_vec_kernel<1>)
                           : d->d <= 16 * FBV_THREADS ? reinterpret_cast<const void *>(feedback_vec_kernel<2>)
                                                      : reinterpret_cast<const void *>(feedback_vec_kernel<3>);
        const int rc_ = device_setup(kern, 112 * 1024, nullptr);
        if (rc_ != SPECROLL_OK) return rc_;
    }
    if (vec && d->d <= 8 * FBV_THREADS)
        feedback_vec_kernel<1><<<d->R, fbv_threads(d->d, 1), fb_smem, st>>>(a);
    else if (vec && d->d <= 16 * FBV_THREADS)
        feedback_vec_kernel<2><<<d->R, fbv_threads(d->d, 2), fb_smem, st>>>(a);
    else if (vec)
        feedback_vec_kernel<3><<<d->R, fbv_threads(d->d, 3), fb_smem, st>>>(a);
    else if (d->d <= 8 * fb::FB_THREADS)
        feedback_kernel<8><<<d->R, fb::FB_THREADS, 0, st>>>(a);
    else if (d->d <= 24 * fb::FB_THREADS)
        feedback_kernel<24><<<d->R, fb::FB_THREADS, 0, st>>>(a);
    else
        feedback_kernel<48><<<d->R, fb::FB_THREADS, 0, st>>>(a);
    SR_LAUNCH_CHECK();
    return SPECROLL_OK;
}
