// Exact target verification: softmax statistics of every tree node, the node-wise
// accept / resample walk, and the terminal (fallback or bonus) draw.
//
// Two launches per plain call:
//   row_stats_kernel    one CTA per (sequence, node) row: streams the bf16 logits once with
//                       128-bit loads and keeps an online (max, sum-exp) pair per thread.
//   walk_term_kernel    one CTA (or cluster) per sequence, launched to overlap the tail of the
//                       statistics kernel: the walk, then the terminal draw.  The residual of the
//                       walk differs from p only on the <= k candidates of the current node (the
//                       proposal is zero elsewhere), so it is tracked as k numbers plus one scale
//                       for the rest of the vocabulary, all in fp64; the terminal draw is an
//                       inverse CDF over the vocabulary in token order with fp64 segment sums, the
//                       walk's <= k residual entries overriding the plain softmax mass.
// The other forms (statistics only of visited rows, nucleus targets, logits that were never
// stored) use walk_kernel / walk_cta_kernel (one warp / one CTA per sequence) and
// terminal_kernel (one CTA per sequence).
#include <math.h>

#include <mutex>

#include "common.cuh"

namespace specroll {

SR_CHECK_TU()

constexpr int RS_THREADS = 256;
constexpr int WALK_WARPS = 4;
constexpr int TERM_THREADS = 512;  // two CTAs per SM
constexpr int TERM_WARPS = TERM_THREADS / 32;
constexpr float NEG_INF = -INFINITY;

// ------------------------------------------------------------------------------ row statistics

// nmc = -m c rides along with the running maximum m, so that an exponent is one fused multiply-add.
__device__ __forceinline__ void online_update(const uint4 &v, float c, float &m, float &nmc, float &s) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    float x[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        x[2 * i] = __uint_as_float(w[i] << 16);
        x[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
    float vm = x[0];
#pragma unroll
    for (int i = 1; i < 8; ++i) vm = fmaxf(vm, x[i]);
    if (vm > m) {
        s *= ex2_approx((m - vm) * c);  // m = -inf gives 0
        m = vm;
        nmc = -vm * c;
    }
    float acc = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) acc += ex2_approx(fmaf(x[i], c, nmc));
    s += acc;
}

// logits[rows, V] bf16; c = log2(e) / T.  row_max = max_v l_v, row_sum = sum_v exp((l_v - max)/T).
// The row is cut into groups of 128 8-token vectors; a warp takes one contiguous run of groups and reads a group
// with four loads of 32 consecutive vectors (2 KB in one piece per warp).  32 registers, so that eight CTAs fit an SM.
constexpr int RS_WARPS = RS_THREADS / 32;

// The run of 8-token vectors that warp w of the statistics kernel takes of a row of nvec vectors, [v_lo, v_hi).
__host__ __device__ inline void rs_run(int nvec, int w, int *v_lo, int *v_hi) {
    const int G = (nvec + 127) / 128, gpw = (G + RS_WARPS - 1) / RS_WARPS;
    const int g_lo = w * gpw < G ? w * gpw : G, g_hi = g_lo + gpw < G ? g_lo + gpw : G;
    *v_lo = g_lo * 128 < nvec ? g_lo * 128 : nvec;
    *v_hi = g_hi * 128 < nvec ? g_hi * 128 : nvec;
}
__host__ __device__ inline int rs_run_of_vec(int nvec, int vi) {
    const int G = (nvec + 127) / 128, gpw = (G + RS_WARPS - 1) / RS_WARPS;
    return (vi / 128) / gpw;
}

// run_tab (nullable): [rows][RS_WARPS] (m, s) of every warp's run, s = sum over the run of exp((l - m)/T): what the
// warps hand to the final reduction anyway.  The terminal draw of a row then finds the eighth of the row that holds
// its target from these and reads only that.
__global__ void __launch_bounds__(RS_THREADS, 8)
row_stats_kernel(const uint16_t *__restrict__ logits, int V, float c, float *__restrict__ row_max,
                 float *__restrict__ row_sum, float2 *__restrict__ run_tab) {
    // a kernel launched behind this one as its programmatic dependent may start its own prologue as SMs free up; it
    // waits for this grid's completion before it reads the statistics
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const size_t row = blockIdx.x;
    const uint4 *p = reinterpret_cast<const uint4 *>(logits + row * (size_t)V);
    const int nvec = V >> 3;
    float m = NEG_INF, nmc = 0.f, s = 0.f;
    {
        const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
        const int G = (nvec + 127) / 128, gpw = (G + RS_WARPS - 1) / RS_WARPS;
        const int g_hi = min(G, (warp + 1) * gpw);
#pragma unroll 1
        for (int g = warp * gpw; g < g_hi; ++g) {
            const int i0 = g * 128 + lane;
            if (i0 + 3 * 32 < nvec) {  // (for lane 31: the whole group is inside the row)
                uint4 v[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) v[q] = ld_nc_v4(p + i0 + q * 32);
#pragma unroll
                for (int q = 0; q < 4; ++q) online_update(v[q], c, m, nmc, s);
            } else {
                for (int q = 0; q < 4; ++q)
                    if (i0 + q * 32 < nvec) online_update(ld_nc_v4(p + i0 + q * 32), c, m, nmc, s);
            }
        }
    }

    // warp, then block reduction of (m, s)
    float mw = warp_max(m);
    s = (m == NEG_INF) ? 0.f : s * ex2_approx((m - mw) * c);
    s = warp_sum(s);
    __shared__ float sm_m[RS_THREADS / 32], sm_s[RS_THREADS / 32];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) {
        sm_m[warp] = mw;
        sm_s[warp] = s;
        if (run_tab) run_tab[row * RS_WARPS + warp] = make_float2(mw, s);
    }
    __syncthreads();
    if (warp == 0) {
        float m2 = lane < RS_THREADS / 32 ? sm_m[lane] : NEG_INF;
        float s2 = lane < RS_THREADS / 32 ? sm_s[lane] : 0.f;
        float mb = warp_max(m2);
        s2 = (m2 == NEG_INF) ? 0.f : s2 * ex2_approx((m2 - mb) * c);
        s2 = warp_sum(s2);
        if (lane == 0) {
            row_max[row] = mb;
            row_sum[row] = s2;
        }
    }
}

// ------------------------------------------------------------------------------ nucleus threshold

// Order-preserving 16-bit key of a bf16 value (-0 counts as +0): larger value <=> larger key.
__device__ __forceinline__ uint32_t ord_key(uint32_t bits) {
    if (bits == 0x8000u) bits = 0u;
    return (bits & 0x8000u) ? (~bits & 0xffffu) : (bits | 0x8000u);
}

constexpr int NUC_THREADS = 512;

// Nucleus of one row (sampling configuration of the experiments: threshold 0.95): tokens are taken in order of
// decreasing probability until their mass first reaches top_p, and every token that ties with the last one
// taken is kept too.  Equal probabilities are equal bf16 logits, so the kept set is "key >= threshold key".
// Run by all NUC_THREADS threads of a CTA; the row comes from HBM once and from L2 after.  Result: st->prefix =
// threshold key (a token is kept iff ord_key(logit) >= key), st->keep = sum of the kept exp((l - M)/T).
//
// The threshold is searched from coarse to exact:
//   A  256 bins of the distance below the maximum, e = (M - l) c in log2 units, 1/8 unit wide, 32 units in all:
//      one pass, fixed-point masses added to counters in shared memory; the bin where the mass from the
//      top reaches top_p * S is selected;
//   C  the keys of the tokens in the selected bin are collected in shared memory (a few thousand at most);
//   D  a radix search over the 16 key bits, four per pass, on that list alone finds the exact key.
// A costs about a dozen instructions per token, C half of that; the bin index is the argument of the
// exponential, which is needed anyway.  If the threshold lies beyond the bins or the list overflows, the
// radix search runs over the whole row instead (nucleus_row_radix; same result, four full passes).
// (Two passes of sixteen private bins per thread in place of A, every token a load, an add and a store in
// shared memory in each: 0.80 ms for the verification of the 1.5B shape against 0.28 without a nucleus.)
constexpr int NUC_LIST = 8192;
constexpr int NUC_BINS = 256;
constexpr float NUC_WB = 0.125f;

struct NucleusSmem {
    float bins[16][NUC_THREADS];
    float wsum[NUC_THREADS / 32][16];
    uint32_t c_lo, c_hi;  // bf16 bits of the ends of the interval of logits that fall into the selected bin
    uint32_t fine_lo[NUC_BINS], fine_hi[NUC_BINS];  // 64-bit fixed-point masses of the fine bins, in two words
    unsigned short list[NUC_LIST];
    int n_list;
    int sel;  // bin selected by the last level
    float above, keep;
    uint32_t prefix;
};

// Sums the sixteen private bins over the block; thread 0 then picks, from the first bin on, the bin at which
// above + running mass reaches the target (or the last bin with mass if rounding keeps the total below it) and
// leaves it in st->sel, the mass before it in st->above and the mass up to and including it in st->keep.
__device__ void nucleus_pick(NucleusSmem *st, float target, bool top_is_high_index) {
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        const float x = warp_sum(st->bins[j][tid]);
        if (lane == 0) st->wsum[warp][j] = x;
    }
    __syncthreads();
    if (warp == 0) {
        // lane j adds bin j over the warps (in warp order); lane 0 then walks the sixteen totals
        float x = 0.f;
        if (lane < 16)
            for (int w2 = 0; w2 < NUC_THREADS / 32; ++w2) x += st->wsum[w2][lane];
        float tot[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) tot[j] = __shfl_sync(0xffffffffu, x, top_is_high_index ? 15 - j : j);  // tot[0] = most probable bin
        if (lane == 0) {
            float cum = st->above;
            int sel = -1, last = 0;
#pragma unroll
            for (int j = 0; j < 16; ++j)
                if (tot[j] > 0.f) last = j;
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                if (sel < 0) {
                    if (cum + tot[j] >= target)
                        sel = j;
                    else
                        cum += tot[j];
                }
            }
            float tsel = 0.f;
            if (sel < 0) {
                sel = last;
                cum = st->above;
#pragma unroll
                for (int j = 0; j < 16; ++j)
                    if (j < last) cum += tot[j];
            }
#pragma unroll
            for (int j = 0; j < 16; ++j)
                if (j == sel) tsel = tot[j];
            st->above = cum;
            st->keep = cum + tsel;
            st->sel = top_is_high_index ? 15 - sel : sel;
        }
    }
    __syncthreads();
}

// One radix pass of the key search: masses of the keys whose leading bits equal `prefix`, by their next four bits.
__device__ __forceinline__ void nucleus_key_bin(NucleusSmem *st, uint32_t bits, int level, uint32_t prefix, float M,
                                                float c) {
    const int shift = 12 - 4 * level;
    const uint32_t key = ord_key(bits);
    if (level == 0 || (key >> (shift + 4)) == prefix)
        st->bins[(key >> shift) & 15u][threadIdx.x] += ex2_approx((__uint_as_float(bits << 16) - M) * c);
}

// Four vectors of a row, NUC_THREADS apart, for one thread.  All four in range (every round but the last): plain
// loads one after the other, so that all four are in flight together; a load under a condition of its own ends up
// behind the use of the one before it.  Absent vectors read as -inf.
__device__ __forceinline__ void nucleus_load4(const uint4 *__restrict__ p, int i0, int nvec, uint4 (&vv)[4]) {
    if (i0 + 3 * NUC_THREADS < nvec) {
#pragma unroll
        for (int q = 0; q < 4; ++q) vv[q] = ld_nc_v4(p + i0 + q * NUC_THREADS);
    } else {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int i = i0 + q * NUC_THREADS;
            vv[q] = i < nvec ? ld_nc_v4(p + i) : make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u);
        }
    }
}

// Exact search over the whole row (fallback): four passes, four key bits each.
__device__ void nucleus_row_radix(const uint4 *__restrict__ p, int nvec, float c, float M, float target,
                                  NucleusSmem *st) {
    const int tid = threadIdx.x;
    if (tid == 0) {
        st->above = 0.f;
        st->prefix = 0u;
    }
    __syncthreads();
    for (int level = 0; level < 4; ++level) {
        const uint32_t prefix = st->prefix;
#pragma unroll
        for (int j = 0; j < 16; ++j) st->bins[j][tid] = 0.f;
        for (int i = tid; i < nvec; i += NUC_THREADS) {
            const uint4 v = ld_nc_v4(p + i);
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int t = 0; t < 8; ++t)
                nucleus_key_bin(st, (t & 1) ? (w[t >> 1] >> 16) : (w[t >> 1] & 0xffffu), level, prefix, M, c);
        }
        nucleus_pick(st, target, true);
        if (tid == 0) st->prefix = (prefix << 4) | (uint32_t)st->sel;
        __syncthreads();
    }
}

__device__ void nucleus_row(const uint16_t *__restrict__ row_logits, int V, float c, float M, float target,
                            NucleusSmem *st) {
    const int tid = threadIdx.x;
    const uint4 *p = reinterpret_cast<const uint4 *>(row_logits);
    const int nvec = V >> 3;
    const float Mc = M * c;
    if (tid == 0) {
        st->above = 0.f;
        st->n_list = 0;
    }
    // the distance below the maximum, in log2 units, and the mass: e >= 0, mass = 2^-e
    auto dist = [&](uint32_t bits) { return Mc - __uint_as_float(bits << 16) * c; };
    // bin = e / width rounded to nearest, taken from the mantissa of e / width + 1.5 * 2^23 (float-to-int
    // conversions share the special-function unit with the exponentials; this stays on the FMA and integer
    // pipes).  Any monotone rule would do: the same one is used in every pass.
    auto to_int = [](float x) { return (int)(__float_as_uint(x + 12582912.0f) - 0x4B400000u); };
    // ---- A: one pass, 256 bins of 1/8 unit over the first 32 units below the maximum, masses as 32-bit fixed point
    //      (round to nearest; the row's largest element is 2^32) added to counters in shared memory: integer
    //      sums do not depend on the order of the atomics, so the result is the same from run to run.  Tokens
    //      further down fall outside the bins; a cut among them goes to the exact search below.
    auto bin_ab = [&](float e) { return to_int(e * (1.0f / NUC_WB)); };  // (>= 0; >= NUC_BINS: outside)
    // (one copy of the counters per warp, in the storage of the private bins of the later steps: only the lanes
    // of a warp can meet at a counter.  Rows of more than 2^20 tokens could overflow a counter: exact search.)
    if (nvec > (1 << 17)) {
        nucleus_row_radix(p, nvec, c, M, target, st);
        return;
    }
    static_assert(sizeof(st->bins) >= (NUC_THREADS / 32) * 2 * NUC_BINS * sizeof(uint32_t), "per-warp fine bins fit");
    uint32_t *wfine = reinterpret_cast<uint32_t *>(&st->bins[0][0]) + (tid >> 5) * 2 * NUC_BINS;
    for (int j = tid; j < (NUC_THREADS / 32) * 2 * NUC_BINS; j += NUC_THREADS) reinterpret_cast<uint32_t *>(&st->bins[0][0])[j] = 0u;
    __syncthreads();
    for (int i0 = tid; i0 < nvec; i0 += 4 * NUC_THREADS) {
        uint4 vv[4];  // four independent loads in flight; an absent one reads as -inf (no mass)
        nucleus_load4(p, i0, nvec, vv);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const uint32_t w[4] = {vv[q].x, vv[q].y, vv[q].z, vv[q].w};
#pragma unroll
            for (int t = 0; t < 8; ++t) {
                const float e = dist((t & 1) ? (w[t >> 1] >> 16) : (w[t >> 1] & 0xffffu));
                const int j = bin_ab(e);
                if (j < NUC_BINS) {
                    // the two halves of the 32-bit mass go to counters of their own: a warp's share of the row is at
                    // most 2^16 tokens, so neither can overflow, and the additions need no result back
                    const uint32_t v = __float2uint_rn(ex2_approx(-e) * 4294967296.0f);
                    atomicAdd(&wfine[j], v & 0xffffu);
                    if (v >> 16) atomicAdd(&wfine[NUC_BINS + j], v >> 16);  // (most tokens are far below the maximum)
                }
            }
        }
    }
    __syncthreads();
    for (int j = tid; j < NUC_BINS; j += NUC_THREADS) {
        unsigned long long tot = 0ull;
        for (int w2 = 0; w2 < NUC_THREADS / 32; ++w2) {
            const uint32_t *wf = reinterpret_cast<const uint32_t *>(&st->bins[0][0]) + w2 * 2 * NUC_BINS;
            tot += ((unsigned long long)wf[NUC_BINS + j] << 16) + wf[j];
        }
        st->fine_lo[j] = (uint32_t)tot;
        st->fine_hi[j] = (uint32_t)(tot >> 32);
    }
    __syncthreads();
    if (tid < 32) {
        // the bin at which the mass from the top reaches the target: every lane takes eight consecutive bins
        const unsigned long long tgt = (unsigned long long)((double)target * 4294967296.0);
        unsigned long long mine = 0ull;
        auto fine = [&](int j) { return ((unsigned long long)st->fine_hi[j] << 32) | st->fine_lo[j]; };
#pragma unroll
        for (int q = 0; q < NUC_BINS / 32; ++q) mine += fine(tid * (NUC_BINS / 32) + q);
        unsigned long long incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned long long x = __shfl_up_sync(0xffffffffu, incl, o);
            if (tid >= o) incl += x;
        }
        const unsigned hit = __ballot_sync(0xffffffffu, incl >= tgt);
        if (hit == 0u) {
            if (tid == 0) st->sel = -1;  // the cut lies further down than the bins reach
        } else if (tid == __ffs(hit) - 1) {
            unsigned long long cum = incl - mine;
            int j = tid * (NUC_BINS / 32);
            while (cum + fine(j) < tgt) cum += fine(j++);  // (ends inside this lane's bins)
            st->sel = j;
            st->above = (float)((double)cum * (1.0 / 4294967296.0));
            st->keep = (float)((double)(cum + fine(j)) * (1.0 / 4294967296.0));
        }
    }
    __syncthreads();
    const int jb = st->sel;
    if (jb < 0) {  // exact search over the whole row
        nucleus_row_radix(p, nvec, c, M, target, st);
        return;
    }
    // ---- C: the tokens of bin jb.  The bin index does not increase with the logit, so they are the logits of an
    //      interval, whose two ends thread 0 finds by bisection over the 16-bit keys (between the most negative finite
    //      value and the row's maximum) with the very rule of pass A; the pass then compares packed bf16 pairs with
    //      the two ends and looks closer only at vectors that hold a member (a few per cent).
    if (tid == 0) {
        auto bits_of_key = [](uint32_t key) { return (key & 0x8000u) ? (key & 0x7fffu) : (~key & 0xffffu); };
        auto bin_of_key = [&](uint32_t key) { return bin_ab(dist(bits_of_key(key))); };
        const uint32_t k_min = ord_key(0xff7fu), k_max = ord_key(__float_as_uint(M) >> 16);
        // smallest key whose bin is <= jb (the bins fall as the keys rise; bin(k_max) = 0 <= jb)
        uint32_t lo = k_min, hi = k_max;
        while (lo < hi) {
            const uint32_t mid = (lo + hi) >> 1;
            if (bin_of_key(mid) <= jb)
                hi = mid;
            else
                lo = mid + 1;
        }
        const uint32_t k_lo = lo;
        // largest key whose bin is >= jb (bin(k_lo) = jb: pass A found a token there)
        lo = k_lo;
        hi = k_max;
        while (lo < hi) {
            const uint32_t mid = (lo + hi + 1) >> 1;
            if (bin_of_key(mid) >= jb)
                lo = mid;
            else
                hi = mid - 1;
        }
        st->c_lo = bits_of_key(k_lo);
        st->c_hi = bits_of_key(lo);
    }
    __syncthreads();
    {
        auto as_bf162 = [](uint32_t w_) { return *reinterpret_cast<const __nv_bfloat162 *>(&w_); };
        const __nv_bfloat162 lo2 = as_bf162(st->c_lo | (st->c_lo << 16)), hi2 = as_bf162(st->c_hi | (st->c_hi << 16));
        // (the loop bound is the same for all lanes of a warp: the body votes and scans over the whole warp; an
        // absent vector reads as -inf, which no interval of finite ends holds)
        for (int ib = tid & ~31; ib < nvec; ib += 4 * NUC_THREADS) {
            const int i0 = ib + (tid & 31);
            uint4 vv[4];
            nucleus_load4(p, i0, nvec, vv);
            // the members among this thread's 32 logits, as one bit each; one reservation in the list per warp and
            // round: the lanes' counts are scanned over the warp
            uint32_t member = 0u;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const uint32_t w[4] = {vv[q].x, vv[q].y, vv[q].z, vv[q].w};
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    const uint32_t mk = __hge2_mask(as_bf162(w[t]), lo2) & __hle2_mask(as_bf162(w[t]), hi2);
                    member |= ((mk & 1u) | ((mk >> 15) & 2u)) << (8 * q + 2 * t);
                }
            }
            if (__ballot_sync(0xffffffffu, member != 0u) == 0u) continue;
            const int cnt = __popc(member);
            int incl = cnt;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int x = __shfl_up_sync(0xffffffffu, incl, o);
                if ((tid & 31) >= o) incl += x;
            }
            int base = 0;
            if ((tid & 31) == 31) base = atomicAdd(&st->n_list, incl);
            base = __shfl_sync(0xffffffffu, base, 31);
            int pos = base + incl - cnt;
            if (cnt) {  // (element 8 q + 2 t + half of this round)
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const uint32_t w[4] = {vv[q].x, vv[q].y, vv[q].z, vv[q].w};
#pragma unroll
                    for (int t = 0; t < 8; ++t) {
                        if ((member >> (8 * q + t)) & 1u) {
                            if (pos < NUC_LIST) st->list[pos] = (unsigned short)((t & 1) ? (w[t >> 1] >> 16) : (w[t >> 1] & 0xffffu));
                            ++pos;
                        }
                    }
                }
            }
        }
    }
    __syncthreads();
    const int n_list = st->n_list;
    if (n_list > NUC_LIST) {  // more tokens in one sub-bin than the list holds: exact search over the whole row
        __syncthreads();
        nucleus_row_radix(p, nvec, c, M, target, st);
        return;
    }
    // ---- D: st->above is the mass above the sub-bin; the key search runs on the list
    if (tid == 0) st->prefix = 0u;
    __syncthreads();
    for (int level = 0; level < 4; ++level) {
        const uint32_t prefix = st->prefix;
#pragma unroll
        for (int j = 0; j < 16; ++j) st->bins[j][tid] = 0.f;
        for (int i = tid; i < n_list; i += NUC_THREADS) nucleus_key_bin(st, st->list[i], level, prefix, M, c);
        nucleus_pick(st, target, true);
        if (tid == 0) st->prefix = (prefix << 4) | (uint32_t)st->sel;
        __syncthreads();
    }
}

// ------------------------------------------------------------------------------ walk

struct WalkArgs {
    const uint16_t *logits;
    // sparse form (logits == NULL): the target logits of every node at the candidates of the node's head only,
    // [B, N, k] bf16, as specroll_target_head_stats leaves them
    const uint16_t *cand_target;
    const int32_t *tree_tok;
    const uint8_t *tree_cand;
    const int32_t *cand_id;
    const float *cand_logit;
    const float *u_acc;
    const float *row_max;
    const float *row_sum;
    int32_t *n_acc, *path_node, *out_tok, *term_node, *term_kind;
    float *min_margin;
    // hand-over to the terminal draw
    int32_t *ws_nov;   // [B]    number of override entries (0 for a bonus draw)
    int32_t *ws_ovid;  // [B,k]  token ids whose mass is overridden
    double *ws_ovm;    // [B,k]  their mass, in units where an untouched token v weighs exp((l_v-M)/T)
    int32_t B, N, K, k, V;
    double T;
};

// What a warp carries from node to node of one sequence's walk.
struct WalkState {
    int nacc, kind;
    double sigma;  // residual of a token outside the candidate set = sigma * p(token)
    double p_off;
    float mm;
    bool have_residual;
};

// Per-warp shared scratch of the walk.
struct WalkSmem {
    double r[SPECROLL_MAX_TOPK];
    double w[SPECROLL_MAX_TOPK];
    float cl[SPECROLL_MAX_TOPK];
    int32_t id[SPECROLL_MAX_TOPK];
    double bc[2];  // broadcast slots: current max, accepted flag
    // per child of the node at hand (walk_node): 1 / s_i, the candidates taken before it, its own candidate
    double inv_s[32];
    uint32_t taken[32];
    int32_t jc[32];
};

// Everything the walk of one sequence can read, staged in shared memory in one round of independent loads (the
// plain walk; the other forms read global memory node by node): per node the row's statistics, the acceptance
// uniform, the drawn token and its slot; per head the candidate ids and proposal logits; per walkable node the
// target logits at its head's candidates.
struct WalkStage {
    const float *rmax, *rsum, *uacc;  // [N]
    const int32_t *ttok;              // [N]
    const uint8_t *tcand;             // [N]
    const int32_t *cid;               // [K, k]
    const float *clog;                // [K, k]
    const uint16_t *pre;              // [N, k]
    // optional (nullptr: computed per node): the tree's parent array, the proposal weights exp((c_j - max c)/T) of
    // every head's candidates, the target probabilities of every walkable node's candidates
    const int8_t *parent;  // [N]
    const double *e;       // [K, k]
    const double *p;       // [N, k]
};

__device__ __forceinline__ void walk_begin(const WalkArgs &a, int b, int lane, WalkState *st) {
    st->nacc = 0;
    st->kind = 0;
    st->sigma = 1.0;
    st->p_off = 0.0;
    st->mm = INFINITY;
    st->have_residual = false;
    if (lane == 0) {
        const int K = a.K;
        for (int i = 0; i <= K; ++i) a.path_node[(size_t)b * (K + 1) + i] = a.out_tok[(size_t)b * (K + 1) + i] = -1;
        a.path_node[(size_t)b * (K + 1)] = 0;
    }
}

// One node u (which has children), by one warp: the target's probabilities on the candidates of u's head -
// S is the normaliser and thr the nucleus threshold key (0: none) of u's row - then u's children in slot order.
// Returns the accepted child, or -1 when every child was rejected (the residual is then in sm->r, st->sigma).
// sg (nullable): the sequence's inputs staged in shared memory.
// emit = false: nothing is written to the results and the count of accepted tokens stays (the node is examined
// on its own, before it is known whether the walk reaches it).
__device__ int walk_node_seq(const WalkArgs &a, const Topo &topo, int b, int u, double M, double S, uint32_t thr,
                                           int lane, WalkSmem *sm, WalkState *st, const WalkStage *sg, bool emit) {
    double *r = sm->r, *w = sm->w;
    float *cl = sm->cl;
    int32_t *id = sm->id;
    const int k = a.k, N = a.N, K = a.K;
    const int hd = topo.depth[u];
    const uint16_t *lg = a.logits ? a.logits + ((size_t)b * N + u) * a.V : nullptr;
    const uint16_t *ct = a.cand_target ? a.cand_target + ((size_t)b * N + u) * k : nullptr;
    // Quotients whose numerator can be exactly zero (the largest logit minus itself, a taken candidate's weight, a
    // residual entry clamped to zero) are formed as products with a reciprocal: a double division with a zero
    // numerator leaves the division's fast path, and one lane on the slow path holds up the whole warp at every slot.
    const double inv_T = 1.0 / a.T, inv_S = 1.0 / S;
    for (int j = lane; j < k; j += 32) {
        const int t = sg ? sg->cid[hd * k + j] : SR_CHECKED(a.cand_id[((size_t)b * K + hd) * k + j], a.V, b);
        id[j] = t;
        cl[j] = sg ? sg->clog[hd * k + j] : a.cand_logit[((size_t)b * K + hd) * k + j];
        const uint32_t bits = sg ? sg->pre[u * k + j] : (lg ? lg[t] : ct[j]);
        const double l = (double)bf16_bits_to_float((uint16_t)bits);
        r[j] = ord_key(bits) >= thr ? exp((l - M) * inv_T) * inv_S : 0.0;  // r = p_u on the candidates
    }
    __syncwarp();
    // Every lane holds one or two of the k candidates (j = lane, lane + 32); sums and maxima over the candidates
    // are warp reductions, so that the state (sigma, p_off, the margin) is the same in every lane and nothing of
    // the slot loop runs on one lane alone (k-long loops of fp64 divisions on one lane were most of the walk's time).
    st->sigma = 1.0;
    {
        double pc = 0.0;
        for (int j = lane; j < k; j += 32) pc += r[j];
        pc = warp_sum(pc);
        st->p_off = pc < 1.0 ? 1.0 - pc : 0.0;
    }
    uint64_t taken = 0;
    int accepted = -1;
    for (int c = u + 1; c < N && accepted < 0; ++c) {
        if (topo.parent[c] != u) continue;
        // slot proposal q on the candidates not yet taken
        double mx = -INFINITY;
        for (int j = lane; j < k; j += 32)
            if (!((taken >> j) & 1) && (double)cl[j] > mx) mx = (double)cl[j];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx = fmax(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        double s = 0.0;
        for (int j = lane; j < k; j += 32) {
            w[j] = ((taken >> j) & 1) ? 0.0 : exp(((double)cl[j] - mx) * inv_T);
            s += w[j];
        }
        s = warp_sum(s);
        const double inv_s = 1.0 / s;
        __syncwarp();
        const int jc = SR_CHECKED((int)(sg ? sg->tcand[c] : a.tree_cand[(size_t)b * N + c]), k, b);
        const double qy = w[jc] * inv_s;
        double ratio;
        if (qy > 0.0)
            ratio = r[jc] > 0.0 ? r[jc] / qy : 0.0;
        else
            ratio = (r[jc] > 0.0) ? INFINITY : 0.0;
        const double uu = (double)(sg ? sg->uacc[c] : a.u_acc[(size_t)b * N + c]);
        const float mg = (float)fabs(uu - ratio);
        if (mg < st->mm) st->mm = mg;
        __syncwarp();
        if (uu < (ratio < 1.0 ? ratio : 1.0)) {
            accepted = c;
        } else {
            double Z = 0.0;
            for (int j = lane; j < k; j += 32) {
                const double t = r[j] - w[j] * inv_s;
                w[j] = t > 0.0 ? t : 0.0;
                Z += w[j];
            }
            Z = warp_sum(Z) + st->sigma * st->p_off;
            if (Z > 1e-300) {
                const double inv_Z = 1.0 / Z;
                for (int j = lane; j < k; j += 32) r[j] = w[j] * inv_Z;
                st->sigma *= inv_Z;
            }
            __syncwarp();
        }
        taken |= 1ull << jc;
    }
    if (accepted >= 0 && emit) {
        if (lane == 0) {
            a.out_tok[(size_t)b * (K + 1) + st->nacc] = sg ? sg->ttok[accepted] : a.tree_tok[(size_t)b * N + accepted];
            a.path_node[(size_t)b * (K + 1) + st->nacc + 1] = accepted;
        }
        ++st->nacc;
    }
    return accepted;
}

// The same node with the slots' dependent chain cut to its minimum (k <= 32 candidates and <= 32 children; anything
// else, and weights that underflow, go to walk_node_seq).  Lane j holds candidate j (replicated over the warp when
// k < 32, so that a sum over the candidates is log2 k shuffle steps), lane i holds child i.
//   - What a slot's proposal is does not depend on the decisions before it: child i sees the candidates its earlier
//     siblings did not draw, q_i(j) = e_j / s_i with e_j = exp((c_j - max c)/T) and s_i the sum of the remaining e_j
//     (the same quotient as with the maximum of the remaining ones as reference).  All s_i at once, before the chain.
//   - The residual is carried unnormalised: r = rho / Zc.  A rejection gives rho_j <- max(rho_j - Zc q_i(j), 0) and
//     Zc <- sum_j rho_j + p_off, where p_off (the target's mass outside the candidates) stays what it was: dividing
//     by Zc gives back the normalised update, with sigma = 1 / Zc.  One fused multiply-add and one sum per slot.
//   - The acceptance test of child i needs rho at its own candidate and Zc as they were when the chain reached it;
//     lane i keeps them and all ratios are formed together after the chain, which runs over all children whether or
//     not an earlier one is accepted (the first accepted child decides; what follows it is ignored).
__device__ int walk_node(const WalkArgs &a, const Topo &topo, int b, int u, double M, double S, uint32_t thr, int lane,
                         WalkSmem *sm, WalkState *st, const WalkStage *sg = nullptr, bool emit = true) {
    const int k = a.k, N = a.N, K = a.K;
    // children of u, in slot order
    const int8_t *par = (sg && sg->parent) ? sg->parent : nullptr;  // (a lane-indexed read of the by-value struct is slow)
    const unsigned cm_lo = __ballot_sync(
        0xffffffffu, lane > u && lane < N && (par ? par[lane < N ? lane : 0] : topo.parent[lane < N ? lane : 0]) == u);
    const unsigned cm_hi = __ballot_sync(0xffffffffu, lane + 32 > u && lane + 32 < N &&
                                                          (par ? par[lane + 32 < N ? lane + 32 : 0]
                                                               : topo.parent[lane + 32 < N ? lane + 32 : 0]) == u);
    const int m_lo = __popc(cm_lo), m = m_lo + __popc(cm_hi);
    if (k > 32 || m > 32) return walk_node_seq(a, topo, b, u, M, S, thr, lane, sm, st, sg, emit);
    const int hd = topo.depth[u];
    int kp = 1;
    while (kp < k) kp <<= 1;
    const int j = lane & (kp - 1);
    const bool have = j < k;
    const double inv_T = 1.0 / a.T, inv_S = 1.0 / S;
    // the candidates: token, proposal weight, target probability
    const bool staged = sg && sg->p && sg->e;
    double rho = 0.0, e = 0.0;
    if (staged) {
        if (have) {
            rho = sg->p[u * k + j];
            e = sg->e[hd * k + j];
            if (lane < k) sm->id[j] = sg->cid[hd * k + j];
        }
    } else {
        float clj = -INFINITY;
        if (have) {
            const int tok = sg ? sg->cid[hd * k + j] : SR_CHECKED(a.cand_id[((size_t)b * K + hd) * k + j], a.V, b);
            clj = sg ? sg->clog[hd * k + j] : a.cand_logit[((size_t)b * K + hd) * k + j];
            uint32_t bits;
            if (sg)
                bits = sg->pre[u * k + j];
            else if (a.logits)
                bits = a.logits[((size_t)b * N + u) * a.V + tok];
            else
                bits = a.cand_target[((size_t)b * N + u) * k + j];
            const double l = (double)bf16_bits_to_float((uint16_t)bits);
            rho = ord_key(bits) >= thr ? exp((l - M) * inv_T) * inv_S : 0.0;
            if (lane < k) sm->id[j] = tok;
        }
        float mxf = clj;
        for (int o = kp >> 1; o > 0; o >>= 1) mxf = fmaxf(mxf, __shfl_xor_sync(0xffffffffu, mxf, o));
        e = have ? exp(((double)clj - (double)mxf) * inv_T) : 0.0;
    }
    double pc = rho;
    for (int o = kp >> 1; o > 0; o >>= 1) pc += __shfl_xor_sync(0xffffffffu, pc, o);
    const double p_off = pc < 1.0 ? 1.0 - pc : 0.0;
    // the children: lane i holds child i
    int c_i = 0, jc_i = 0;
    double uu_i = 0.0;
    if (lane < m) {
        c_i = lane < m_lo ? (int)__fns(cm_lo, 0, lane + 1) : 32 + (int)__fns(cm_hi, 0, lane - m_lo + 1);
        jc_i = SR_CHECKED((int)(sg ? sg->tcand[c_i] : a.tree_cand[(size_t)b * N + c_i]), k, b);
        uu_i = (double)(sg ? sg->uacc[c_i] : a.u_acc[(size_t)b * N + c_i]);
    }
    unsigned taken_i = lane < m ? (1u << jc_i) : 0u;  // exclusive prefix OR over the children before i
    {
        unsigned incl = taken_i;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl |= t;
        }
        taken_i = incl & ~taken_i;
    }
    double s_i = 0.0;
    if (staged) {
        for (int jj = 0; jj < k; ++jj)
            if (!((taken_i >> jj) & 1u)) s_i += sg->e[hd * k + jj];
    } else {
        for (int jj = 0; jj < k; ++jj) {
            const double ej = __shfl_sync(0xffffffffu, e, jj);
            if (!((taken_i >> jj) & 1u)) s_i += ej;
        }
    }
    if (__ballot_sync(0xffffffffu, lane < m && !(s_i > 0.0 && s_i < INFINITY)))
        return walk_node_seq(a, topo, b, u, M, S, thr, lane, sm, st, sg, emit);
    // what a slot needs from its child, where every lane can read it without a shuffle
    const double inv_s_i = lane < m ? 1.0 / s_i : 0.0;
    if (lane < m) {
        sm->inv_s[lane] = inv_s_i;
        sm->taken[lane] = taken_i;
        sm->jc[lane] = jc_i;
    }
    __syncwarp();
    // the chain
    double Zc = 1.0, my_rho = 0.0, my_Zc = 1.0;
    for (int i = 0; i < m; ++i) {
        const double q = ((sm->taken[i] >> j) & 1u) ? 0.0 : e * sm->inv_s[i];
        const double rho_jc = __shfl_sync(0xffffffffu, rho, sm->jc[i]);
        if (lane == i) {
            my_rho = rho_jc;
            my_Zc = Zc;
        }
        const double t = fmax(rho - Zc * q, 0.0);
        double Zn = t;
        for (int o = kp >> 1; o > 0; o >>= 1) Zn += __shfl_xor_sync(0xffffffffu, Zn, o);
        Zn += p_off;
        if (Zn > 1e-300 * Zc) {
            rho = t;
            Zc = Zn;
        }
    }
    // child i's own proposal probability: its candidate is among those it can still draw
    const double my_q = __shfl_sync(0xffffffffu, e, jc_i) * inv_s_i;
    // every child's test at once
    bool acc_i = false;
    float mg_i = INFINITY;
    if (lane < m) {
        double ratio;
        if (my_q > 0.0)
            ratio = my_rho > 0.0 ? (my_rho / my_Zc) / my_q : 0.0;
        else
            ratio = my_rho > 0.0 ? INFINITY : 0.0;
        acc_i = uu_i < (ratio < 1.0 ? ratio : 1.0);
        mg_i = (float)fabs(uu_i - ratio);
    }
    const unsigned accmask = __ballot_sync(0xffffffffu, acc_i);
    const int first = accmask ? __ffs(accmask) - 1 : -1;
    float mg = (lane < m && (first < 0 || lane <= first)) ? mg_i : INFINITY;
    mg = -warp_max(-mg);
    if (mg < st->mm) st->mm = mg;
    if (first >= 0) {
        const int accepted = __shfl_sync(0xffffffffu, c_i, first);
        if (emit) {
            if (lane == 0) {
                a.out_tok[(size_t)b * (K + 1) + st->nacc] = sg ? sg->ttok[accepted] : a.tree_tok[(size_t)b * N + accepted];
                a.path_node[(size_t)b * (K + 1) + st->nacc + 1] = accepted;
            }
            ++st->nacc;
        }
        return accepted;
    }
    // all rejected: the residual, normalised as the callers expect it (r and sigma = 1 / Zc)
    const double inv_Zc = 1.0 / Zc;
    if (lane < k) sm->r[j] = rho * inv_Zc;
    st->sigma = inv_Zc;
    st->p_off = p_off;
    __syncwarp();
    return -1;
}

// Results of a sequence and the hand-over of the residual (S = normaliser of u's row) to the terminal draw.
__device__ __forceinline__ void walk_end(const WalkArgs &a, int b, int u, double S, int lane, WalkSmem *sm,
                                         WalkState *st) {
    const int k = a.k;
    if (st->have_residual) {
        const double sigma = __shfl_sync(0xffffffffu, st->sigma, 0);
        const double f = S / sigma;  // (one division; the entries may be zero)
        for (int j = lane; j < k; j += 32) {
            a.ws_ovid[(size_t)b * k + j] = sm->id[j];
            a.ws_ovm[(size_t)b * k + j] = sm->r[j] * f;
        }
    }
    if (lane == 0) {
        a.ws_nov[b] = st->have_residual ? k : 0;
        a.n_acc[b] = st->nacc;
        a.term_node[b] = u;
        a.term_kind[b] = st->kind;
        if (a.min_margin) a.min_margin[b] = st->mm;
    }
}

// Bytes of shared memory the staged inputs of one sequence take (16-byte multiples per array).
__host__ __device__ inline size_t walk_stage_bytes(int N, int K, int k) {
    auto up = [](size_t x) { return (x + 15) / 16 * 16; };
    return 4 * up((size_t)N * 4) + up((size_t)N) + 2 * up((size_t)K * k * 4) + up((size_t)N * k * 2);
}

// Plain target distributions: one warp per sequence.  Which nodes the walk visits depends on its decisions, but
// what it can ask for does not, so with the dense logits everything is fetched up front (WalkStage): one round
// trip to memory per sequence instead of four or five dependent ones per visited node, which is what the walk's
// time consisted of.  Dynamic shared memory: WALK_WARPS * walk_stage_bytes.
__global__ void __launch_bounds__(WALK_WARPS * 32) walk_kernel(WalkArgs a, Topo topo) {
    __shared__ WalkSmem sh[WALK_WARPS];
    extern __shared__ __align__(16) unsigned char sh_stage[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int b = blockIdx.x * WALK_WARPS + warp;
    if (b >= a.B) return;
    WalkSmem *sm = &sh[warp];
    const int N = a.N, K = a.K, k = a.k;
    WalkStage stage;
    const WalkStage *sg = nullptr;
    if (a.logits) {
        auto up = [](size_t x) { return (x + 15) / 16 * 16; };
        unsigned char *p = sh_stage + (size_t)warp * walk_stage_bytes(N, K, k);
        float *rmax = reinterpret_cast<float *>(p);
        p += up((size_t)N * 4);
        float *rsum = reinterpret_cast<float *>(p);
        p += up((size_t)N * 4);
        float *uacc = reinterpret_cast<float *>(p);
        p += up((size_t)N * 4);
        int32_t *ttok = reinterpret_cast<int32_t *>(p);
        p += up((size_t)N * 4);
        uint8_t *tcand = reinterpret_cast<uint8_t *>(p);
        p += up((size_t)N);
        int32_t *cid = reinterpret_cast<int32_t *>(p);
        p += up((size_t)K * k * 4);
        float *clog = reinterpret_cast<float *>(p);
        p += up((size_t)K * k * 4);
        uint16_t *pre = reinterpret_cast<uint16_t *>(p);
        for (int n = lane; n < N; n += 32) {
            rmax[n] = a.row_max[(size_t)b * N + n];
            rsum[n] = a.row_sum[(size_t)b * N + n];
            uacc[n] = a.u_acc[(size_t)b * N + n];
            ttok[n] = a.tree_tok[(size_t)b * N + n];
            tcand[n] = a.tree_cand[(size_t)b * N + n];
        }
        for (int e = lane; e < K * k; e += 32) {
            cid[e] = SR_CHECKED(a.cand_id[(size_t)b * K * k + e], a.V, b);
            clog[e] = a.cand_logit[(size_t)b * K * k + e];
        }
        for (int e = lane; e < N * k; e += 32) {
            const int u = e / k, j = e - u * k;
            if (topo.n_child[u] > 0) {  // (a node with children is at depth < K)
                const int t = SR_CHECKED(a.cand_id[((size_t)b * K + topo.depth[u]) * k + j], a.V, b);
                pre[e] = a.logits[((size_t)b * N + u) * a.V + t];
            }
        }
        __syncwarp();
        stage = WalkStage{rmax, rsum, uacc, ttok, tcand, cid, clog, pre, nullptr, nullptr, nullptr};
        sg = &stage;
    }
    WalkState st;
    walk_begin(a, b, lane, &st);
    int u = 0;
    for (;;) {
        if (topo.n_child[u] == 0) {
            st.kind = (u != 0) ? 1 : 0;
            st.have_residual = false;
            break;
        }
        const double M = sg ? (double)sg->rmax[u] : (double)a.row_max[(size_t)b * N + u];
        const double S = sg ? (double)sg->rsum[u] : (double)a.row_sum[(size_t)b * N + u];
        const int acc = walk_node(a, topo, b, u, M, S, 0u, lane, sm, &st, sg);
        if (acc < 0) {
            st.kind = 0;
            st.have_residual = true;
            break;
        }
        u = acc;
    }
    walk_end(a, b, u, sg ? (double)sg->rsum[u] : (double)a.row_sum[(size_t)b * N + u], lane, sm, &st);
}

// Maximum and sum of exponentials of one row by all NUC_THREADS threads of a CTA (same arithmetic as
// row_stats_kernel); every thread returns with the result.
__device__ void row_stats_row(const uint16_t *__restrict__ row_logits, int V, float c, float *sm_m, float *sm_s,
                              float *M_out, float *S_out) {
    const uint4 *p = reinterpret_cast<const uint4 *>(row_logits);
    const int nvec = V >> 3;
    float m = NEG_INF, nmc = 0.f, s = 0.f;
    int i = threadIdx.x;
    for (; i + 3 * NUC_THREADS < nvec; i += 4 * NUC_THREADS) {
        uint4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) v[u] = ld_nc_v4(p + i + u * NUC_THREADS);
#pragma unroll
        for (int u = 0; u < 4; ++u) online_update(v[u], c, m, nmc, s);
    }
    for (; i < nvec; i += NUC_THREADS) online_update(ld_nc_v4(p + i), c, m, nmc, s);
    const float mw = warp_max(m);
    s = (m == NEG_INF) ? 0.f : s * ex2_approx((m - mw) * c);
    s = warp_sum(s);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    __syncthreads();
    if (lane == 0) {
        sm_m[warp] = mw;
        sm_s[warp] = s;
    }
    __syncthreads();
    float mb = NEG_INF;
    for (int w = 0; w < NUC_THREADS / 32; ++w) mb = fmaxf(mb, sm_m[w]);
    float sb = 0.f;
    for (int w = 0; w < NUC_THREADS / 32; ++w)
        sb += (sm_m[w] == NEG_INF) ? 0.f : sm_s[w] * ex2_approx((sm_m[w] - mb) * c);
    *M_out = mb;
    *S_out = sb;
}

// One CTA per sequence, for the two variants in which something has to be computed per visited node before the
// node can be walked, and which nodes are visited is known only as the walk goes:
//   LAZY  the softmax statistics of a row are computed when the walk reaches it (at most K + 1 rows per
//         sequence instead of all N), and written to row_max / row_sum for those rows only;
//   NUC   the target distributions are their nuclei: the row's threshold is searched (nucleus_row) and left
//         in thr_key / keep_sum (the terminal draw reads those of the last node).
// Before each node all threads do that work, then warp 0 does the node.
template <bool LAZY, bool NUC>
__global__ void __launch_bounds__(NUC_THREADS)
walk_cta_kernel(WalkArgs a, Topo topo, float c, float top_p, float *__restrict__ row_max_w,
                float *__restrict__ row_sum_w, uint32_t *__restrict__ thr_key, float *__restrict__ keep_sum,
                float *__restrict__ out_thr, float *__restrict__ out_sum, int thr_ready) {
    extern __shared__ __align__(16) unsigned char nuc_raw[];  // NucleusSmem (NUC only): above the static limit
    NucleusSmem &nuc = *reinterpret_cast<NucleusSmem *>(nuc_raw);
    __shared__ WalkSmem sm;
    __shared__ float sm_m[NUC_THREADS / 32], sm_s[NUC_THREADS / 32];
    __shared__ int sh_next;  // next node, or -1 when the walk is over
    const int b = blockIdx.x, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    WalkState st;
    if (warp == 0) walk_begin(a, b, lane, &st);
    int u = 0;
    for (;;) {
        const size_t row = (size_t)b * a.N + u;
        float M, S;
        if constexpr (LAZY) {
            row_stats_row(a.logits + row * a.V, a.V, c, sm_m, sm_s, &M, &S);
            if (threadIdx.x == 0) {
                row_max_w[row] = M;
                row_sum_w[row] = S;
            }
        } else {
            M = a.row_max[row];
            S = a.row_sum[row];
        }
        uint32_t thr = 0u;
        float norm = S;
        if constexpr (NUC) {
            if (thr_ready && topo.n_child[u] > 0) {  // (left by nucleus_rows_kernel for every node with children)
                thr = thr_key[row];
                norm = keep_sum[row];
            } else {
                nucleus_row(a.logits + row * a.V, a.V, c, M, top_p * S, &nuc);
                thr = nuc.prefix;
                norm = nuc.keep;
            }
            if (threadIdx.x == 0 && !(thr_ready && topo.n_child[u] > 0)) {
                thr_key[row] = thr;
                keep_sum[row] = norm;
                if (out_sum) out_sum[row] = norm;
                if (out_thr) {  // the threshold as a logit: undo the key
                    const uint32_t bits = (thr & 0x8000u) ? (thr & 0x7fffu) : (~thr & 0xffffu);
                    out_thr[row] = __uint_as_float(bits << 16);
                }
            }
        }
        if (warp == 0) {
            int next = -1;
            if (topo.n_child[u] == 0) {
                st.kind = (u != 0) ? 1 : 0;
                st.have_residual = false;
            } else {
                next = walk_node(a, topo, b, u, (double)M, (double)norm, thr, lane, &sm, &st);
                if (next < 0) {
                    st.kind = 0;
                    st.have_residual = true;
                }
            }
            if (next < 0) walk_end(a, b, u, (double)norm, lane, &sm, &st);
            if (lane == 0) sh_next = next;
        }
        __syncthreads();
        const int next = sh_next;
        __syncthreads();
        if (next < 0) break;
        u = next;
    }
}

// The nucleus thresholds of every node with children, one CTA per (sequence, such node), all at once: which of
// them the walk visits is not known yet, but a row's threshold depends on the row alone, and one pass of all
// of them over the machine costs less than the visited ones one after the other inside a sequence's walk.  (A
// sequence that ends at a leaf still needs that leaf's threshold for its last token: the walk kernel finds it.)
#ifndef NUC_AHEAD_ROWS_PER_SM
#define NUC_AHEAD_ROWS_PER_SM 5
#endif
struct NodeList {
    int32_t n;
    int8_t node[SPECROLL_MAX_NODES];
};

__global__ void __launch_bounds__(NUC_THREADS)
nucleus_rows_kernel(const uint16_t *__restrict__ logits, int V, int N, NodeList nodes, float c, float top_p,
                    const float *__restrict__ row_max, const float *__restrict__ row_sum,
                    uint32_t *__restrict__ thr_key, float *__restrict__ keep_sum, float *__restrict__ out_thr,
                    float *__restrict__ out_sum) {
    extern __shared__ __align__(16) unsigned char nuc_raw[];
    NucleusSmem &nuc = *reinterpret_cast<NucleusSmem *>(nuc_raw);
    const int b = blockIdx.x / nodes.n, u = nodes.node[blockIdx.x - b * nodes.n];
    const size_t row = (size_t)b * N + u;
    const float M = row_max[row], S = row_sum[row];
    nucleus_row(logits + row * V, V, c, M, top_p * S, &nuc);
    if (threadIdx.x == 0) {
        const uint32_t thr = nuc.prefix;
        thr_key[row] = thr;
        keep_sum[row] = nuc.keep;
        if (out_sum) out_sum[row] = nuc.keep;
        if (out_thr) {  // the threshold as a logit: undo the key
            const uint32_t bits = (thr & 0x8000u) ? (thr & 0x7fffu) : (~thr & 0xffffu);
            out_thr[row] = __uint_as_float(bits << 16);
        }
    }
}

// ------------------------------------------------------------------------------ terminal draw

struct TermArgs {
    const uint16_t *logits;
    const float *u_fin;
    const float *row_max;
    const int32_t *n_acc, *term_node;
    const int32_t *ws_nov, *ws_ovid;
    const double *ws_ovm;
    const uint32_t *thr_key;  // nucleus threshold per row (NULL: no truncation)
    int32_t *out_tok;
    int32_t B, N, K, k, V;
    float c;  // log2(e) / T
    int32_t row_per_seq;  // logits holds one row per sequence (that of its terminal node) instead of [B, N, V]
};

// Plain softmax masses of eight tokens; tokens below the nucleus threshold (thr = 0: none) weigh nothing.
__device__ __forceinline__ void masses8(const uint4 &v, float M, float c, uint32_t thr, float (&e)[8]) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    if (thr == 0u) {  // (uniform over the CTA) no truncation: nothing to compare, a third of the instructions
        const float nm = -M * c;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            e[2 * i] = ex2_approx(fmaf(__uint_as_float(w[i] << 16), c, nm));
            e[2 * i + 1] = ex2_approx(fmaf(__uint_as_float(w[i] & 0xffff0000u), c, nm));
        }
        return;
    }
    // the order of the keys is the order of the values (-0 = +0): compare two logits at a time with the
    // threshold's value
    const uint32_t tb = (thr & 0x8000u) ? (thr & 0x7fffu) : (~thr & 0xffffu);  // the key undone
    const uint32_t tb2 = tb | (tb << 16);
    const __nv_bfloat162 t2 = *reinterpret_cast<const __nv_bfloat162 *>(&tb2);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float e0 = ex2_approx(fmaf(__uint_as_float(w[i] << 16), c, -M * c));
        const float e1 = ex2_approx(fmaf(__uint_as_float(w[i] & 0xffff0000u), c, -M * c));
        const uint32_t keep = __hge2_mask(*reinterpret_cast<const __nv_bfloat162 *>(&w[i]), t2);
        e[2 * i] = (keep & 0xffffu) ? e0 : 0.f;
        e[2 * i + 1] = (keep >> 16) ? e1 : 0.f;
    }
}
__device__ __forceinline__ float mass1(uint16_t bits, float M, float c, uint32_t thr) {
    return ord_key(bits) >= thr ? ex2_approx(fmaf(bf16_bits_to_float(bits), c, -M * c)) : 0.f;  // same form as masses8
}

__device__ __forceinline__ double warp_incl_scan(double v, int lane) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        double t = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += t;
    }
    return v;
}

// Pass 1 of the terminal draw by one warp: the plain softmax mass of every 32-vector slice of the segment
// [v_lo, v_hi) of a row, eight slices' loads in flight, left in out[0 .. n_sl).
__device__ __forceinline__ void term_slice_masses(const uint4 *__restrict__ p, int v_lo, int v_hi, int n_sl, float M, float c,
                                                  uint32_t thr, int lane, double *out) {
    for (int s0 = 0; s0 < n_sl; s0 += 8) {
        uint4 v[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int i = v_lo + (s0 + q) * 32 + lane;
            v[q] = (s0 + q < n_sl && i < v_hi) ? ld_nc_v4(p + i) : make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u);  // -inf: no mass
        }
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            float e[8];
            masses8(v[q], M, c, thr, e);
            // a slice's 256 masses are added pairwise in fp32 (relative error of a few 2^-24, the size of the
            // exponentials' own error); everything above a slice is fp64.  (Converting every mass to fp64 first
            // kept the conversion pipe busy for as long as the exponentials.)
            float acc = ((e[0] + e[1]) + (e[2] + e[3])) + ((e[4] + e[5]) + (e[6] + e[7]));
            acc = warp_sum(acc);
            if (lane == 0 && s0 + q < n_sl) out[s0 + q] = (double)acc;
        }
    }
}

// The masses of the eight tokens of vector i of a row (zero beyond v_hi), the residual entries in place of the
// plain masses of their tokens; returns their sum.
__device__ __forceinline__ double term_vector_masses(const uint4 *__restrict__ p, int i, int v_hi, float M, float c, uint32_t thr,
                                                     int nov, const int32_t *ovid, const double *ovm, double (&ms)[8]) {
    double lsum = 0.0;
    if (i < v_hi) {
        float e[8];
        masses8(ld_nc_v4(p + i), M, c, thr, e);
#pragma unroll
        for (int t = 0; t < 8; ++t) ms[t] = (double)e[t];
        for (int j = 0; j < nov; ++j) {
            const int off = ovid[j] - i * 8;
            if (off >= 0 && off < 8) {
#pragma unroll
                for (int t = 0; t < 8; ++t)
                    if (t == off) ms[t] = ovm[j];
            }
        }
#pragma unroll
        for (int t = 0; t < 8; ++t) lsum += ms[t];
    } else {
#pragma unroll
        for (int t = 0; t < 8; ++t) ms[t] = 0.0;
    }
    return lsum;
}

// The token inside a 32-vector slice, by the warp whose lanes hold the vectors' masses (ms, their sums lsum): the
// first token whose running mass, from base on, exceeds the target; take_last: the last one with positive mass.
__device__ __forceinline__ void term_pick_token(int i, const double (&ms)[8], double lsum, double base, double target,
                                                bool take_last, int v_hi, int32_t *dst, int lane) {
    const double incl = warp_incl_scan(lsum, lane);
    const unsigned hit = take_last ? 0u : __ballot_sync(0xffffffffu, base + incl > target);
    if (hit) {
        const int Lh = __ffs(hit) - 1;
        if (lane == Lh) {
            int tok = -1;
            double cum = base + (incl - lsum);
#pragma unroll
            for (int t = 0; t < 8; ++t) {
                cum += ms[t];
                if (tok < 0 && cum > target) tok = i * 8 + t;
            }
            if (tok < 0) {  // scan and sequential sums disagreed in the last bit
#pragma unroll
                for (int t = 0; t < 8; ++t)
                    if (ms[t] > 0.0) tok = i * 8 + t;
            }
            *dst = tok;
        }
    } else {
        // the lanes' scanned mass fell short of the slice's sum by rounding: last token with positive mass
        int last_pos = -1;
#pragma unroll
        for (int t = 0; t < 8; ++t)
            if (ms[t] > 0.0) last_pos = i * 8 + t;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) last_pos = max(last_pos, __shfl_xor_sync(0xffffffffu, last_pos, o));
        if (lane == 0) *dst = last_pos < 0 ? max(0, v_hi * 8 - 1) : last_pos;
    }
}

// Last step of the terminal draw by one warp, inside the segment [v_lo, v_hi) that holds the target mass: seg_slices =
// the segment's n_sl slice masses (residual entries applied), base = the mass before the segment; ovid / ovm = the nov
// residual entries.  Writes the token to *dst.
__device__ void term_pick(const uint4 *__restrict__ p, const double *seg_slices, int n_sl, int v_lo, int v_hi, double base,
                          double target, float M, float c, uint32_t thr, int nov, const int32_t *ovid, const double *ovm,
                          int32_t *dst, int lane) {
    // the slice inside the selected segment: first one whose running mass exceeds the target; if rounding made
    // the slices fall short of the segment's own sum, the last slice with positive mass
    int sl_sel = -1, sl_pos = -1;
    double base_pos = 0.0;
    for (int c0 = 0; c0 < n_sl && sl_sel < 0; c0 += 32) {
        const double v = (c0 + lane < n_sl) ? seg_slices[c0 + lane] : 0.0;
        const double incl = warp_incl_scan(v, lane);
        const unsigned hit = __ballot_sync(0xffffffffu, base + incl > target);
        const unsigned pos = __ballot_sync(0xffffffffu, v > 0.0);
        if (pos) {
            const int lp = 31 - __clz(pos);
            sl_pos = c0 + lp;
            base_pos = base + __shfl_sync(0xffffffffu, incl - v, lp);
        }
        if (hit) {
            const int lh = __ffs(hit) - 1;
            sl_sel = c0 + lh;
            base += __shfl_sync(0xffffffffu, incl - v, lh);
        } else {
            base += __shfl_sync(0xffffffffu, incl, 31);
        }
    }
    bool take_last = false;
    if (sl_sel < 0) {
        if (sl_pos < 0) {  // no mass at all in the segment (cannot be selected with positive total; keep a valid token)
            if (lane == 0) *dst = max(0, v_hi * 8 - 1);
            return;
        }
        sl_sel = sl_pos;
        base = base_pos;
        take_last = true;
    }
    // the token inside the slice
    const int i = v_lo + sl_sel * 32 + lane;
    double ms[8];
    const double lsum = term_vector_masses(p, i, v_hi, M, c, thr, nov, ovid, ovm, ms);
    term_pick_token(i, ms, lsum, base, target, take_last, v_hi, dst, lane);
}

// The vocabulary is cut into TERM_WARPS warp segments of vpw 8-token vectors, each walked in slices of 32 vectors (one per
// lane).  Pass 1 (all warps, independent loads) leaves the fp64 mass of every slice in shared memory; the walk's
// residual entries then replace the plain mass of their tokens; two scans pick the segment and the slice that
// hold u * total, and only that slice is read again to find the token.
__host__ __device__ inline int term_slices(int V) {
    const int nvec = V >> 3, vpw = (nvec + TERM_WARPS - 1) / TERM_WARPS;
    return (vpw + 31) / 32;
}

__global__ void __launch_bounds__(TERM_THREADS) terminal_kernel(TermArgs a) {
    extern __shared__ double sh_slice[];  // [TERM_WARPS][n_sl]
    __shared__ double sh_seg[32];
    __shared__ double sh_ovm[SPECROLL_MAX_TOPK];
    __shared__ int32_t sh_ovid[SPECROLL_MAX_TOPK];
    __shared__ int sh_pick[2];     // target warp, -1 if none
    __shared__ double sh_base[2];  // mass before the target warp's segment; target

    const int b = blockIdx.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int node = a.term_node[b];
    const int nov = a.ws_nov[b];
    const float M = a.row_max[(size_t)b * a.N + node];
    const uint32_t thr = a.thr_key ? a.thr_key[(size_t)b * a.N + node] : 0u;
    const uint16_t *lg = a.logits + (a.row_per_seq ? (size_t)b : (size_t)b * a.N + node) * a.V;
    const uint4 *p = reinterpret_cast<const uint4 *>(lg);
    const int nvec = a.V >> 3;
    const int vpw = (nvec + TERM_WARPS - 1) / TERM_WARPS;  // vectors per warp segment
    const int n_sl = (vpw + 31) / 32;                      // slices per segment
    const int v_lo = min(nvec, warp * vpw), v_hi = min(nvec, v_lo + vpw);

    if (threadIdx.x < nov) {
        sh_ovm[threadIdx.x] = a.ws_ovm[(size_t)b * a.k + threadIdx.x];
        sh_ovid[threadIdx.x] = a.ws_ovid[(size_t)b * a.k + threadIdx.x];
    }

    term_slice_masses(p, v_lo, v_hi, n_sl, M, a.c, thr, lane, sh_slice + warp * n_sl);
    __syncthreads();
    // the walk's residual entries replace the plain mass of their tokens (at most k of them: one thread)
    if (threadIdx.x == 0) {
        for (int j = 0; j < nov; ++j) {
            const int t = sh_ovid[j], vi = t >> 3;
            const int w = min(TERM_WARPS - 1, vi / vpw), sl = (vi - w * vpw) >> 5;
            sh_slice[w * n_sl + sl] += sh_ovm[j] - (double)mass1(lg[t], M, a.c, thr);
        }
    }
    __syncthreads();
    // segment masses
    {
        double acc = 0.0;
        for (int sl = lane; sl < n_sl; sl += 32) acc += sh_slice[warp * n_sl + sl];
        acc = warp_sum(acc);
        if (lane == 0) sh_seg[warp] = acc;
    }
    __syncthreads();
    if (warp == 0) {
        const double seg = lane < TERM_WARPS ? sh_seg[lane] : 0.0;
        const double incl = warp_incl_scan(seg, lane);
        const double total = __shfl_sync(0xffffffffu, incl, 31);
        const double target = (double)a.u_fin[b] * total;
        const unsigned hit = __ballot_sync(0xffffffffu, lane < TERM_WARPS && incl > target);
        const int wsel = hit ? (__ffs(hit) - 1) : -1;
        const double base = __shfl_sync(0xffffffffu, incl - seg, wsel < 0 ? 0 : wsel);
        if (lane == 0) {
            sh_pick[0] = wsel;
            sh_base[0] = base;
            sh_base[1] = target;
        }
    }
    __syncthreads();
    const int wsel = sh_pick[0];
    const int nacc = a.n_acc[b];
    int32_t *dst = a.out_tok + (size_t)b * (a.K + 1) + nacc;
    if (wsel < 0) {
        // u_fin * total reached the total through rounding: take the last token with positive mass
        if (threadIdx.x == 0) {
            int tok = a.V - 1;
            for (; tok > 0; --tok) {
                double ms = (double)mass1(lg[tok], M, a.c, thr);
                for (int j = 0; j < nov; ++j)
                    if (sh_ovid[j] == tok) ms = sh_ovm[j];
                if (ms > 0.0) break;
            }
            *dst = tok;
        }
        return;
    }
    if (warp != wsel) return;

    term_pick(p, sh_slice + warp * n_sl, n_sl, v_lo, v_hi, sh_base[0], sh_base[1], M, a.c, thr, nov, sh_ovid, sh_ovm, dst,
              lane);
}

// ------------------------------------------------------------------------------ walk + terminal draw in one launch
//
// The plain verification after the row statistics, one cluster of S CTAs per sequence (S = 1: plain CTAs).
//   (1) Everything a walk can read is staged in shared memory; what does not depend on the row statistics (the
//       candidates, the uniforms, the target logits at the candidates) is fetched before the wait for the previous
//       kernel in the stream, which this kernel is launched to overlap with (programmatic dependent launch).
//   (2) Which nodes the walk reaches depends on its decisions, but what happens AT a node does not: its children
//       are tried in slot order until one is accepted, each against the residual left by the rejections before it.
//       So every node with children is examined on its own, one warp per node, all at once: the first accepted
//       child (or none, and then the residual), and the smallest margin on the way.  The walk itself is then a
//       chain of at most K + 1 look-ups.  Every CTA of a cluster does (1) and (2) for itself: same inputs, same
//       arithmetic, same result, nothing to exchange.
//   (3) The terminal draw over the last node's row: the S * WT_WARPS warps of the cluster each take one segment of
//       the vocabulary; the slice masses of the other CTAs are read through distributed shared memory by the
//       cluster's first CTA, which finishes as terminal_kernel does.  (Letting the statistics pass leave the mass
//       of every slice of every row, so that this step reads a table and one slice, was tried: the table costs the
//       statistics kernel as much as it saves here.)
constexpr int WT_THREADS = 512;
constexpr int WT_WARPS = WT_THREADS / 32;

struct WtLayout {
    size_t stage, ovm, first, mm, slices, seg, par, e, p, total;
    int G, vpw, n_sl;
};
__host__ __device__ inline WtLayout wt_layout(int N, int K, int k, int V, int S) {
    WtLayout L;
    auto up = [](size_t x) { return (x + 15) / 16 * 16; };
    const int nvec = V >> 3;
    L.G = S * WT_WARPS;
    L.vpw = (nvec + L.G - 1) / L.G;
    L.n_sl = (L.vpw + 31) / 32;
    size_t o = 0;
    L.stage = o;
    o += up(walk_stage_bytes(N, K, k));
    L.ovm = o;
    o += up((size_t)N * k * sizeof(double));
    L.first = o;
    o += up((size_t)N * sizeof(int32_t));
    L.mm = o;
    o += up((size_t)N * sizeof(float));
    L.slices = o;
    o += up((size_t)L.G * L.n_sl * sizeof(double));
    L.seg = o;
    o += up((size_t)L.G * sizeof(double));
    L.par = o;
    o += up((size_t)N);
    L.e = o;
    o += up((size_t)K * k * sizeof(double));
    L.p = o;
    o += up((size_t)N * k * sizeof(double));
    L.total = o;
    return L;
}

__global__ void __launch_bounds__(WT_THREADS, 2) walk_term_kernel(WalkArgs a, Topo topo, const float *__restrict__ u_fin, float c,
                                                               int S, const float2 *__restrict__ run_tab) {
    __shared__ WalkSmem sh[WT_WARPS];
    extern __shared__ __align__(16) unsigned char sh_dyn[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int rank = S > 1 ? (int)cluster_ctarank() : 0;
    const int b = blockIdx.x / S;
    const int N = a.N, K = a.K, k = a.k;
    const WtLayout L = wt_layout(N, K, k, a.V, S);
    auto up = [](size_t x) { return (x + 15) / 16 * 16; };
    unsigned char *p0 = sh_dyn + L.stage;
    float *rmax = reinterpret_cast<float *>(p0);
    p0 += up((size_t)N * 4);
    float *rsum = reinterpret_cast<float *>(p0);
    p0 += up((size_t)N * 4);
    float *uacc = reinterpret_cast<float *>(p0);
    p0 += up((size_t)N * 4);
    int32_t *ttok = reinterpret_cast<int32_t *>(p0);
    p0 += up((size_t)N * 4);
    uint8_t *tcand = reinterpret_cast<uint8_t *>(p0);
    p0 += up((size_t)N);
    int32_t *cid = reinterpret_cast<int32_t *>(p0);
    p0 += up((size_t)K * k * 4);
    float *clog = reinterpret_cast<float *>(p0);
    p0 += up((size_t)K * k * 4);
    uint16_t *pre = reinterpret_cast<uint16_t *>(p0);
    double *ovm = reinterpret_cast<double *>(sh_dyn + L.ovm);
    int32_t *first = reinterpret_cast<int32_t *>(sh_dyn + L.first);
    float *mmin = reinterpret_cast<float *>(sh_dyn + L.mm);
    double *slices = reinterpret_cast<double *>(sh_dyn + L.slices);
    double *seg = reinterpret_cast<double *>(sh_dyn + L.seg);
    int8_t *par = reinterpret_cast<int8_t *>(sh_dyn + L.par);
    double *we = reinterpret_cast<double *>(sh_dyn + L.e);
    double *wp = reinterpret_cast<double *>(sh_dyn + L.p);
    const double inv_T = 1.0 / a.T;
    // (1) inputs of this call, none of them written by the kernel before this one
    for (int n = tid; n < N; n += WT_THREADS) {
        uacc[n] = a.u_acc[(size_t)b * N + n];
        ttok[n] = a.tree_tok[(size_t)b * N + n];
        tcand[n] = a.tree_cand[(size_t)b * N + n];
        par[n] = topo.parent[n];
    }
    for (int e = tid; e < K * k; e += WT_THREADS) {
        cid[e] = SR_CHECKED(a.cand_id[(size_t)b * K * k + e], a.V, b);
        clog[e] = a.cand_logit[(size_t)b * K * k + e];
    }
    for (int e = tid; e < N * k; e += WT_THREADS) {
        const int u = e / k, j = e - u * k;
        if (topo.n_child[u] > 0) {  // (a node with children is at depth < K)
            const int t = SR_CHECKED(a.cand_id[((size_t)b * K + topo.depth[u]) * k + j], a.V, b);
            pre[e] = a.logits[((size_t)b * N + u) * a.V + t];
        }
    }
    // the proposal weights of every head's candidates, relative to the head's largest logit
    __syncthreads();
    for (int e = tid; e < K * k; e += WT_THREADS) {
        const int hd = e / k;
        float mx = -INFINITY;
        for (int jj = 0; jj < k; ++jj) mx = fmaxf(mx, clog[hd * k + jj]);
        we[e] = exp(((double)clog[e] - (double)mx) * inv_T);
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");  // the row statistics are complete from here on
    for (int n = tid; n < N; n += WT_THREADS) {
        rmax[n] = a.row_max[(size_t)b * N + n];
        rsum[n] = a.row_sum[(size_t)b * N + n];
    }
    // the target probabilities of every walkable node's candidates (the statistics straight from global memory:
    // one round trip for everything)
    for (int e = tid; e < N * k; e += WT_THREADS) {
        const int u = e / k;
        if (topo.n_child[u] > 0) {
            const double M = (double)a.row_max[(size_t)b * N + u], S = (double)a.row_sum[(size_t)b * N + u];
            wp[e] = exp(((double)bf16_bits_to_float(pre[e]) - M) * inv_T) * (1.0 / S);
        }
    }
    __syncthreads();
    // (2) every node with children on its own
    {
        const WalkStage stage{rmax, rsum, uacc, ttok, tcand, cid, clog, pre, par, we, wp};
        int idx = 0;
        for (int u = 0; u < N; ++u) {
            if (topo.n_child[u] == 0) continue;
            if ((idx++ % WT_WARPS) != warp) continue;
            WalkState st;
            st.nacc = 0;
            st.kind = 0;
            st.sigma = 1.0;
            st.p_off = 0.0;
            st.mm = INFINITY;
            st.have_residual = false;
            const int acc = walk_node(a, topo, b, u, (double)rmax[u], (double)rsum[u], 0u, lane, &sh[warp], &st, &stage, false);
            if (acc < 0) {
                const double f = (double)rsum[u] / st.sigma;
                for (int j = lane; j < k; j += 32) ovm[u * k + j] = sh[warp].r[j] * f;
            }
            if (lane == 0) {
                first[u] = acc;
                mmin[u] = st.mm;
            }
            __syncwarp();
        }
    }
    __syncthreads();
    // the walk: every thread follows the same chain
    int u = 0, nacc = 0, kind = 0;
    bool resid = false;
    float mm = INFINITY;
    const bool writer = (rank == 0 && tid == 0);
    if (writer) {
        for (int i = 0; i <= K; ++i) a.path_node[(size_t)b * (K + 1) + i] = a.out_tok[(size_t)b * (K + 1) + i] = -1;
        a.path_node[(size_t)b * (K + 1)] = 0;
    }
    for (;;) {
        if (topo.n_child[u] == 0) {
            kind = (u != 0) ? 1 : 0;
            break;
        }
        mm = fminf(mm, mmin[u]);
        const int ch = first[u];
        if (ch < 0) {
            resid = true;
            break;
        }
        if (writer) {
            a.out_tok[(size_t)b * (K + 1) + nacc] = ttok[ch];
            a.path_node[(size_t)b * (K + 1) + nacc + 1] = ch;
        }
        ++nacc;
        u = ch;
    }
    if (writer) {
        a.n_acc[b] = nacc;
        a.term_node[b] = u;
        a.term_kind[b] = kind;
        if (a.min_margin) a.min_margin[b] = mm;
    }

    // (3) the terminal draw from row u: the residual (k entries over the plain masses) or the plain distribution
    const int nov = resid ? k : 0;
    const int32_t *ovid = cid + (resid ? topo.depth[u] : 0) * k;
    const double *ovm_u = ovm + u * k;
    const float M = rmax[u];
    const uint16_t *lg = a.logits + ((size_t)b * N + u) * a.V;
    const uint4 *p = reinterpret_cast<const uint4 *>(lg);
    const int nvec = a.V >> 3, G = L.G;
    // With the statistics kernel's table of the row's eight runs (run_tab; then S = 1): the run that holds the target
    // is found from the table and only that eighth of the row is read, cut into G segments like a whole row
    // otherwise.  v_base, nvec_r: the vectors the draw works on; base0: the mass before them.
    __shared__ int sh_run;
    __shared__ double sh_b0t[2];
    int v_base = 0, nvec_r = nvec;
    if (run_tab) {
        if (warp == 0) {
            const float2 e = lane < RS_WARPS ? run_tab[((size_t)b * N + u) * RS_WARPS + lane] : make_float2(-INFINITY, 0.f);
            double v = (lane < RS_WARPS && e.x != -INFINITY) ? (double)e.y * (double)ex2_approx((e.x - M) * c) : 0.0;
            for (int j = 0; j < nov; ++j)
                if (rs_run_of_vec(nvec, ovid[j] >> 3) == lane) v += ovm_u[j] - (double)mass1(pre[u * k + j], M, c, 0u);
            v = fmax(v, 0.0);  // (a run whose mass was all in overridden tokens, after rounding)
            const double incl = warp_incl_scan(v, lane);
            const double total = __shfl_sync(0xffffffffu, incl, 31);
            const double target = (double)u_fin[b] * total;
            const unsigned hit = __ballot_sync(0xffffffffu, lane < RS_WARPS && incl > target);
            const unsigned pos = __ballot_sync(0xffffffffu, v > 0.0);
            // (rounding kept the target at or above the total: the last run with mass; the draw inside it then ends
            // at its last token with mass)
            const int r = hit ? __ffs(hit) - 1 : (pos ? 31 - __clz(pos) : 0);
            const double b0 = __shfl_sync(0xffffffffu, incl - v, r);
            if (lane == 0) {
                sh_run = r;
                sh_b0t[0] = b0;
                sh_b0t[1] = target;
            }
        }
        __syncthreads();
        int v_end;
        rs_run(nvec, sh_run, &v_base, &v_end);
        nvec_r = v_end - v_base;
    }
    const int vpw = (nvec_r + G - 1) / G > 0 ? (nvec_r + G - 1) / G : 1;  // vectors per warp segment
    const int n_sl = (vpw + 31) / 32;                                     // slices per segment (<= the layout's)
    {
        {
            const int g = rank * WT_WARPS + warp;
            const int v_lo = v_base + min(nvec_r, g * vpw), v_hi = v_base + min(nvec_r, g * vpw + vpw);
            term_slice_masses(p, v_lo, v_hi, n_sl, M, c, 0u, lane, slices + (size_t)g * n_sl);
        }
        if (S > 1) {
            cluster_sync_all();  // every CTA's slice masses are in its shared memory
            if (rank == 0) {
                const int per = WT_WARPS * n_sl;
                for (int e = tid; e < (S - 1) * per; e += WT_THREADS) {
                    const int r = 1 + e / per, o = r * per + (e - (r - 1) * per);
                    slices[o] = ld_dsmem_f64(slices + o, r);
                }
            }
            cluster_sync_all();  // the other CTAs may leave
            if (rank != 0) return;
        }
        __syncthreads();
        if (tid == 0) {
            for (int j = 0; j < nov; ++j) {
                const int t = ovid[j], vi = (t >> 3) - v_base;
                if (vi < 0 || vi >= nvec_r) continue;  // (outside the run the draw works on)
                const int w = min(G - 1, vi / vpw), sl = (vi - w * vpw) >> 5;
                slices[w * n_sl + sl] += ovm_u[j] - (double)mass1(pre[u * k + j], M, c, 0u);  // (staged: lg[t])
            }
        }
        __syncthreads();
        for (int g = warp; g < G; g += WT_WARPS) {
            double acc = 0.0;
            for (int sl = lane; sl < n_sl; sl += 32) acc += slices[g * n_sl + sl];
            acc = warp_sum(acc);
            if (lane == 0) seg[g] = acc;
        }
        __syncthreads();
    }
    if (warp != 0) return;
    double target, base;
    if (run_tab) {
        base = sh_b0t[0];
        target = sh_b0t[1];
    } else {
        double total = 0.0;
        for (int g0 = 0; g0 < G; g0 += 32) total += warp_sum(g0 + lane < G ? seg[g0 + lane] : 0.0);
        target = (double)u_fin[b] * total;
        base = 0.0;
    }
    int wsel = -1;
    for (int g0 = 0; g0 < G && wsel < 0; g0 += 32) {
        const double v = g0 + lane < G ? seg[g0 + lane] : 0.0;
        const double incl = warp_incl_scan(v, lane);
        const unsigned hit = __ballot_sync(0xffffffffu, g0 + lane < G && base + incl > target);
        if (hit) {
            const int lh = __ffs(hit) - 1;
            wsel = g0 + lh;
            base += __shfl_sync(0xffffffffu, incl - v, lh);
        } else {
            base += __shfl_sync(0xffffffffu, incl, 31);
        }
    }
    int32_t *dst = a.out_tok + (size_t)b * (K + 1) + nacc;
    if (wsel < 0) {
        // the target reached the end of the masses through rounding: take the last token with positive mass (from the
        // end of the vectors the draw worked on, downwards)
        if (lane == 0) {
            int tok = (v_base + nvec_r) * 8 - 1;
            for (; tok > 0; --tok) {
                double ms = (double)mass1(lg[tok], M, c, 0u);
                for (int j = 0; j < nov; ++j)
                    if (ovid[j] == tok) ms = ovm_u[j];
                if (ms > 0.0) break;
            }
            *dst = tok;
        }
        return;
    }
    const int v_lo = v_base + min(nvec_r, wsel * vpw), v_hi = v_base + min(nvec_r, wsel * vpw + vpw);
    term_pick(p, slices + (size_t)wsel * n_sl, n_sl, v_lo, v_hi, base, target, M, c, 0u, nov, ovid, ovm_u, dst, lane);
}

// S CTAs per sequence: as many as keep the grid within about two CTAs per SM, a power of two up to the portable
// cluster size.
static int walk_term_split(int B) {
    int S = 8;
    while (S > 1 && (long long)B * S > 296) S >>= 1;
    return S;
}

static int launch_terminal(const TermArgs &ta, cudaStream_t st) {
    const size_t smem = (size_t)TERM_WARPS * term_slices(ta.V) * sizeof(double);
    if (smem > 200 * 1024) return SPECROLL_ELIMIT;
    if (smem > 40 * 1024)
        SR_CUDA_TRY(cudaFuncSetAttribute(terminal_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    terminal_kernel<<<ta.B, TERM_THREADS, smem, st>>>(ta);
    SR_LAUNCH_CHECK();
    return SPECROLL_OK;
}

}  // namespace specroll

// ------------------------------------------------------------------------------ entry points

using namespace specroll;

static int check_verify_desc(const specroll_verify_desc *d) {
    if (!d || d->B < 0 || d->N < 1 || d->N > SPECROLL_MAX_NODES || d->K < 1 || d->K > SPECROLL_MAX_HEADS ||
        d->k < 1 || d->k > SPECROLL_MAX_TOPK || d->V < 8 || (d->V % 8) || d->k > d->V ||
        !(d->temperature > 0.f) || (d->flags & ~SPECROLL_VERIFY_LAZY_STATS) != 0)
        return SPECROLL_EINVAL;
    return SPECROLL_OK;
}

static size_t verify_ws_base(const specroll_verify_desc *d) {
    size_t B = (size_t)d->B, k = (size_t)d->k;
    return align_up(B * k * sizeof(double), 256) + align_up(B * k * sizeof(int32_t), 256) +
           align_up(B * sizeof(int32_t), 256) + 256;
}

// The statistics kernel's table of every row's eight runs (plain verification with all rows' statistics).
static size_t verify_ws_runs(const specroll_verify_desc *d) {
    return align_up((size_t)d->B * d->N * RS_WARPS * sizeof(float2), 256);
}

extern "C" size_t specroll_verify_workspace_bytes(const specroll_verify_desc *d) {
    if (check_verify_desc(d) != SPECROLL_OK) return 0;
    return verify_ws_base(d) + ((d->flags & SPECROLL_VERIFY_LAZY_STATS) ? 0 : verify_ws_runs(d));
}

extern "C" size_t specroll_verify_nucleus_workspace_bytes(const specroll_verify_desc *d) {
    if (check_verify_desc(d) != SPECROLL_OK) return 0;
    const size_t rows = (size_t)d->B * d->N;
    return verify_ws_base(d) + align_up(rows * sizeof(uint32_t), 256) + align_up(rows * sizeof(float), 256);
}

// top_p in (0, 1): the target distributions are their nuclei; otherwise the plain softmax.
static int run_verify(const specroll_verify_desc *d, float top_p, const void *logits, const int32_t *parent_host,
                      const int32_t *tree_tok, const uint8_t *tree_cand, const int32_t *cand_id,
                      const float *cand_logit, const float *u_acc, const float *u_fin, int32_t *n_acc,
                      int32_t *path_node, int32_t *out_tok, int32_t *term_node, int32_t *term_kind, float *row_max,
                      float *row_sum, float *min_margin, float *nucleus_thr, float *nucleus_sum, void *workspace,
                      size_t workspace_bytes, void *cuda_stream, bool runs_optional = false) {
    if (check_verify_desc(d) != SPECROLL_OK) return SPECROLL_EINVAL;
    const bool truncate = top_p > 0.f && top_p < 1.f;
    Topo topo;
    if (build_topo(parent_host, d->N, d->K, d->k, &topo, nullptr) != SPECROLL_OK) return SPECROLL_EINVAL;
    if (d->B == 0) return SPECROLL_OK;  // (an empty batch has empty arrays: their pointers may be NULL)
    if (!logits || !tree_tok || !tree_cand || !cand_id || !cand_logit || !u_acc || !u_fin || !n_acc ||
        !path_node || !out_tok || !term_node || !term_kind || !row_max || !row_sum)
        return SPECROLL_EINVAL;
    if (!aligned16(logits)) return SPECROLL_EALIGN;
    const bool lazy = (d->flags & SPECROLL_VERIFY_LAZY_STATS) != 0;
    // the table of the rows' runs serves the plain verification with all rows' statistics; a caller with a fixed
    // scratch, or with the nucleus form's workspace, goes without it when it does not fit (the terminal draw then
    // reads the whole row, spread over a cluster for small batches)
    bool use_runs = !truncate && !lazy;
    if (use_runs && runs_optional && workspace_bytes < verify_ws_base(d) + verify_ws_runs(d)) use_runs = false;
    const size_t need = truncate ? specroll_verify_nucleus_workspace_bytes(d)
                                 : verify_ws_base(d) + (use_runs ? verify_ws_runs(d) : 0);
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) || workspace_bytes < need)
        return SPECROLL_EWORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const size_t B = (size_t)d->B, k = (size_t)d->k;
    char *ws = static_cast<char *>(workspace);
    double *ws_ovm = reinterpret_cast<double *>(ws);
    ws += align_up(B * k * sizeof(double), 256);
    int32_t *ws_ovid = reinterpret_cast<int32_t *>(ws);
    ws += align_up(B * k * sizeof(int32_t), 256);
    int32_t *ws_nov = reinterpret_cast<int32_t *>(ws);
    ws += align_up(B * sizeof(int32_t), 256) + 256;
    const size_t n_rows = B * (size_t)d->N;
    uint32_t *thr_key = truncate ? reinterpret_cast<uint32_t *>(ws) : nullptr;
    float *keep_sum = truncate ? reinterpret_cast<float *>(ws + align_up(n_rows * sizeof(uint32_t), 256)) : nullptr;

    const float c = (float)(1.4426950408889634 / (double)d->temperature);
    const int rows = d->B * d->N;
    float2 *run_tab = use_runs ? reinterpret_cast<float2 *>(ws) : nullptr;  // (behind the hand-over area; no nucleus arrays in this form)
    if (!lazy) {
        row_stats_kernel<<<rows, RS_THREADS, 0, st>>>(static_cast<const uint16_t *>(logits), d->V, c, row_max,
                                                      row_sum, run_tab);
        SR_LAUNCH_CHECK();
    }

    WalkArgs wa;
    wa.logits = static_cast<const uint16_t *>(logits);
    wa.cand_target = nullptr;
    wa.tree_tok = tree_tok;
    wa.tree_cand = tree_cand;
    wa.cand_id = cand_id;
    wa.cand_logit = cand_logit;
    wa.u_acc = u_acc;
    wa.row_max = row_max;
    wa.row_sum = row_sum;
    wa.n_acc = n_acc;
    wa.path_node = path_node;
    wa.out_tok = out_tok;
    wa.term_node = term_node;
    wa.term_kind = term_kind;
    wa.min_margin = min_margin;
    wa.ws_nov = ws_nov;
    wa.ws_ovid = ws_ovid;
    wa.ws_ovm = ws_ovm;
    wa.B = d->B;
    wa.N = d->N;
    wa.K = d->K;
    wa.k = d->k;
    wa.V = d->V;
    wa.T = (double)d->temperature;
    if (truncate) {
        int rc_ = device_setup(reinterpret_cast<const void *>(walk_cta_kernel<false, true>), (int)sizeof(NucleusSmem), nullptr);
        if (rc_ == SPECROLL_OK)
            rc_ = device_setup(reinterpret_cast<const void *>(walk_cta_kernel<true, true>), (int)sizeof(NucleusSmem), nullptr);
        if (rc_ != SPECROLL_OK) return rc_;
        if (lazy) {
            walk_cta_kernel<true, true><<<d->B, NUC_THREADS, sizeof(NucleusSmem), st>>>(
                wa, topo, c, top_p, row_max, row_sum, thr_key, keep_sum, nucleus_thr, nucleus_sum, 0);
        } else {
            NodeList nodes;
            nodes.n = 0;
            for (int u = 0; u < d->N; ++u)
                if (topo.n_child[u] > 0) nodes.node[nodes.n++] = (int8_t)u;
            // Worth it while those rows are few enough to be searched side by side (small batches, whose walks
            // would otherwise search three or four rows one after the other on a nearly empty machine); with
            // more rows than that, searching only the visited ones inside the walk is less work and faster.
            int n_sm = 0;
            rc_ = device_setup(reinterpret_cast<const void *>(nucleus_rows_kernel), (int)sizeof(NucleusSmem), &n_sm);
            if (rc_ != SPECROLL_OK) return rc_;
            const bool ahead = nodes.n > 0 && d->B * nodes.n <= NUC_AHEAD_ROWS_PER_SM * n_sm;
            if (ahead) {
                nucleus_rows_kernel<<<d->B * nodes.n, NUC_THREADS, sizeof(NucleusSmem), st>>>(
                    static_cast<const uint16_t *>(logits), d->V, d->N, nodes, c, top_p, row_max, row_sum, thr_key, keep_sum,
                    nucleus_thr, nucleus_sum);
                SR_LAUNCH_CHECK();
            }
            walk_cta_kernel<false, true><<<d->B, NUC_THREADS, sizeof(NucleusSmem), st>>>(
                wa, topo, c, top_p, row_max, row_sum, thr_key, keep_sum, nucleus_thr, nucleus_sum, ahead ? 1 : 0);
        }
    } else if (lazy) {
        walk_cta_kernel<true, false><<<d->B, NUC_THREADS, 0, st>>>(wa, topo, c, 1.0f, row_max, row_sum, nullptr, nullptr,
                                                                    nullptr, nullptr, 0);
    } else {
        // plain verification: the walk and the terminal draw in one launch, overlapping the statistics kernel's tail
        constexpr int WT_SMEM_LIMIT = 160 * 1024;
        const int S = use_runs ? 1 : walk_term_split(d->B);
        const WtLayout L = wt_layout(d->N, d->K, d->k, d->V, S);
        if (L.total > (size_t)WT_SMEM_LIMIT) return SPECROLL_ELIMIT;
        const int rc_ = device_setup(reinterpret_cast<const void *>(walk_term_kernel), WT_SMEM_LIMIT, nullptr);
        if (rc_ != SPECROLL_OK) return rc_;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(d->B * S));
        cfg.blockDim = dim3(WT_THREADS);
        cfg.dynamicSmemBytes = L.total;
        cfg.stream = st;
        cudaLaunchAttribute attrs[2];
        int na = 0;
        attrs[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attrs[na].val.programmaticStreamSerializationAllowed = 1;
        ++na;
        if (S > 1) {
            attrs[na].id = cudaLaunchAttributeClusterDimension;
            attrs[na].val.clusterDim.x = (unsigned)S;
            attrs[na].val.clusterDim.y = 1;
            attrs[na].val.clusterDim.z = 1;
            ++na;
        }
        cfg.attrs = attrs;
        cfg.numAttrs = na;
        SR_CUDA_TRY(cudaLaunchKernelEx(&cfg, walk_term_kernel, wa, topo, u_fin, c, S, (const float2 *)run_tab));
        return SPECROLL_OK;
    }
    SR_LAUNCH_CHECK();

    TermArgs ta;
    ta.logits = wa.logits;
    ta.u_fin = u_fin;
    ta.row_max = row_max;
    ta.n_acc = n_acc;
    ta.term_node = term_node;
    ta.ws_nov = ws_nov;
    ta.ws_ovid = ws_ovid;
    ta.ws_ovm = ws_ovm;
    ta.thr_key = thr_key;
    ta.out_tok = out_tok;
    ta.B = d->B;
    ta.N = d->N;
    ta.K = d->K;
    ta.k = d->k;
    ta.V = d->V;
    ta.c = c;
    ta.row_per_seq = 0;
    return launch_terminal(ta, st);
}

// The hand-over area between the walk and the terminal draw inside a workspace (the layout of run_verify).
static void carve_verify_ws(const specroll_verify_desc *d, void *workspace, double **ovm, int32_t **ovid, int32_t **nov) {
    const size_t B = (size_t)d->B, k = (size_t)d->k;
    char *ws = static_cast<char *>(workspace);
    *ovm = reinterpret_cast<double *>(ws);
    ws += align_up(B * k * sizeof(double), 256);
    *ovid = reinterpret_cast<int32_t *>(ws);
    ws += align_up(B * k * sizeof(int32_t), 256);
    *nov = reinterpret_cast<int32_t *>(ws);
}

namespace specroll {
// want_id[(b, u), j] = cand_id[b, depth(u), j]: the tokens whose target logit the walk reads at node u
__global__ void want_ids_kernel(Topo topo, int B, int N, int K, int k, const int32_t *__restrict__ cand_id,
                                int32_t *__restrict__ want_id) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (size_t)B * N * k) return;
    const int j = (int)(i % k), u = (int)((i / k) % N), b = (int)(i / ((size_t)k * N));
    const int hd = min((int)topo.depth[u], K - 1);  // (a node of the last level has no children; any valid token)
    want_id[i] = cand_id[((size_t)b * K + hd) * k + j];
}
}  // namespace specroll

extern "C" int specroll_verify_want_ids(const specroll_verify_desc *d, const int32_t *parent_host,
                                        const int32_t *cand_id, int32_t *want_id, void *cuda_stream) {
    if (check_verify_desc(d) != SPECROLL_OK || !cand_id || !want_id) return SPECROLL_EINVAL;
    Topo topo;
    if (build_topo(parent_host, d->N, d->K, d->k, &topo, nullptr) != SPECROLL_OK) return SPECROLL_EINVAL;
    const size_t n = (size_t)d->B * d->N * d->k;
    if (n == 0) return SPECROLL_OK;
    want_ids_kernel<<<(unsigned)((n + 255) / 256), 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        topo, d->B, d->N, d->K, d->k, cand_id, want_id);
    SR_LAUNCH_CHECK();
    return SPECROLL_OK;
}

extern "C" int specroll_verify_walk_sparse(const specroll_verify_desc *d, const void *cand_target,
                                           const float *row_max, const float *row_sum, const int32_t *parent_host,
                                           const int32_t *tree_tok, const uint8_t *tree_cand, const int32_t *cand_id,
                                           const float *cand_logit, const float *u_acc, int32_t *n_acc,
                                           int32_t *path_node, int32_t *out_tok, int32_t *term_node,
                                           int32_t *term_kind, float *min_margin, void *workspace,
                                           size_t workspace_bytes, void *cuda_stream) {
    if (check_verify_desc(d) != SPECROLL_OK || d->flags != 0) return SPECROLL_EINVAL;
    Topo topo;
    if (build_topo(parent_host, d->N, d->K, d->k, &topo, nullptr) != SPECROLL_OK) return SPECROLL_EINVAL;
    if (d->B == 0) return SPECROLL_OK;  // (an empty batch has empty arrays: their pointers may be NULL)
    if (!cand_target || !row_max || !row_sum || !tree_tok || !tree_cand || !cand_id || !cand_logit || !u_acc || !n_acc ||
        !path_node || !out_tok || !term_node || !term_kind)
        return SPECROLL_EINVAL;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) || workspace_bytes < verify_ws_base(d))
        return SPECROLL_EWORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    WalkArgs wa;
    wa.logits = nullptr;
    wa.cand_target = static_cast<const uint16_t *>(cand_target);
    wa.tree_tok = tree_tok;
    wa.tree_cand = tree_cand;
    wa.cand_id = cand_id;
    wa.cand_logit = cand_logit;
    wa.u_acc = u_acc;
    wa.row_max = row_max;
    wa.row_sum = row_sum;
    wa.n_acc = n_acc;
    wa.path_node = path_node;
    wa.out_tok = out_tok;
    wa.term_node = term_node;
    wa.term_kind = term_kind;
    wa.min_margin = min_margin;
    carve_verify_ws(d, workspace, &wa.ws_ovm, &wa.ws_ovid, &wa.ws_nov);
    wa.B = d->B;
    wa.N = d->N;
    wa.K = d->K;
    wa.k = d->k;
    wa.V = d->V;
    wa.T = (double)d->temperature;
    walk_kernel<<<(d->B + WALK_WARPS - 1) / WALK_WARPS, WALK_WARPS * 32, 0, st>>>(wa, topo);
    SR_LAUNCH_CHECK();
    return SPECROLL_OK;
}

extern "C" int specroll_verify_terminal_rows(const specroll_verify_desc *d, const void *term_logits,
                                             const float *row_max, const int32_t *n_acc, const int32_t *term_node,
                                             const float *u_fin, int32_t *out_tok, void *workspace,
                                             size_t workspace_bytes, void *cuda_stream) {
    if (check_verify_desc(d) != SPECROLL_OK || d->flags != 0) return SPECROLL_EINVAL;
    if (d->B == 0) return SPECROLL_OK;  // (an empty batch has empty arrays: their pointers may be NULL)
    if (!term_logits || !row_max || !n_acc || !term_node || !u_fin || !out_tok) return SPECROLL_EINVAL;
    if (!aligned16(term_logits)) return SPECROLL_EALIGN;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) || workspace_bytes < verify_ws_base(d))
        return SPECROLL_EWORKSPACE;
    TermArgs ta;
    double *ovm;
    int32_t *ovid, *nov;
    carve_verify_ws(d, workspace, &ovm, &ovid, &nov);
    ta.logits = static_cast<const uint16_t *>(term_logits);
    ta.u_fin = u_fin;
    ta.row_max = row_max;
    ta.n_acc = n_acc;
    ta.term_node = term_node;
    ta.ws_nov = nov;
    ta.ws_ovid = ovid;
    ta.ws_ovm = ovm;
    ta.thr_key = nullptr;
    ta.out_tok = out_tok;
    ta.B = d->B;
    ta.N = d->N;
    ta.K = d->K;
    ta.k = d->k;
    ta.V = d->V;
    ta.c = (float)(1.4426950408889634 / (double)d->temperature);
    ta.row_per_seq = 1;
    return launch_terminal(ta, static_cast<cudaStream_t>(cuda_stream));
}

extern "C" int specroll_verify(const specroll_verify_desc *d, const void *logits,
                               const int32_t *parent_host, const int32_t *tree_tok,
                               const uint8_t *tree_cand, const int32_t *cand_id,
                               const float *cand_logit, const float *u_acc, const float *u_fin,
                               int32_t *n_acc, int32_t *path_node, int32_t *out_tok,
                               int32_t *term_node, int32_t *term_kind, float *row_max,
                               float *row_sum, float *min_margin, void *workspace,
                               size_t workspace_bytes, void *cuda_stream) {
    return run_verify(d, 1.0f, logits, parent_host, tree_tok, tree_cand, cand_id, cand_logit, u_acc, u_fin, n_acc,
                      path_node, out_tok, term_node, term_kind, row_max, row_sum, min_margin, nullptr, nullptr,
                      workspace, workspace_bytes, cuda_stream);
}

extern "C" int specroll_verify_nucleus(const specroll_verify_desc *d, float top_p, const void *logits,
                                       const int32_t *parent_host, const int32_t *tree_tok,
                                       const uint8_t *tree_cand, const int32_t *cand_id,
                                       const float *cand_logit, const float *u_acc, const float *u_fin,
                                       int32_t *n_acc, int32_t *path_node, int32_t *out_tok,
                                       int32_t *term_node, int32_t *term_kind, float *row_max,
                                       float *row_sum, float *min_margin, float *nucleus_thr,
                                       float *nucleus_sum, void *workspace, size_t workspace_bytes,
                                       void *cuda_stream) {
    if (!(top_p > 0.f)) return SPECROLL_EINVAL;
    return run_verify(d, top_p, logits, parent_host, tree_tok, tree_cand, cand_id, cand_logit, u_acc, u_fin, n_acc,
                      path_node, out_tok, term_node, term_kind, row_max, row_sum, min_margin, nucleus_thr,
                      nucleus_sum, workspace, workspace_bytes, cuda_stream, /*runs_optional=*/true);
}

// ------------------------------------------------------------------------------ allocation-free variant
//
// Scratch of specroll_verify_static: lives in the library image, one copy per GPU that loads the
// library, held until the process exits.  Layout = the workspace layout of specroll_verify for the
// largest admitted problem (SPECROLL_STATIC_MAX_B sequences, SPECROLL_STATIC_MAX_BK residual entries).
namespace specroll {
constexpr size_t STATIC_SCRATCH_BYTES =
    (SPECROLL_STATIC_MAX_BK * sizeof(double) + 255) / 256 * 256 +
    (SPECROLL_STATIC_MAX_BK * sizeof(int32_t) + 255) / 256 * 256 +
    (SPECROLL_STATIC_MAX_B * sizeof(int32_t) + 255) / 256 * 256 + 256;
static __device__ __align__(256) unsigned char g_verify_scratch[STATIC_SCRATCH_BYTES];

constexpr int MAX_DEVICES = 64;
static void *g_scratch_addr[MAX_DEVICES];  // device address of g_verify_scratch, per device ordinal
static std::mutex g_scratch_mutex;
}  // namespace specroll

extern "C" int specroll_verify_static(const specroll_verify_desc *d, const void *logits,
                                      const int32_t *parent_host, const int32_t *tree_tok,
                                      const uint8_t *tree_cand, const int32_t *cand_id,
                                      const float *cand_logit, const float *u_acc, const float *u_fin,
                                      int32_t *n_acc, int32_t *path_node, int32_t *out_tok,
                                      int32_t *term_node, int32_t *term_kind, float *row_max,
                                      float *row_sum, float *min_margin, void *cuda_stream) {
    if (check_verify_desc(d) != SPECROLL_OK) return SPECROLL_EINVAL;
    if (d->B > SPECROLL_STATIC_MAX_B || (long long)d->B * d->k > SPECROLL_STATIC_MAX_BK) return SPECROLL_ELIMIT;
    if (verify_ws_base(d) > STATIC_SCRATCH_BYTES) return SPECROLL_ELIMIT;
    int dev = -1;
    SR_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= MAX_DEVICES) return SPECROLL_ELIMIT;
    void *scratch = nullptr;
    {
        // In host code the array's name is only a handle; the kernels need its device address,
        // which differs per GPU.  Looked up once per device, with that device current.
        std::lock_guard<std::mutex> lock(g_scratch_mutex);
        if (!g_scratch_addr[dev]) {
            void *p = nullptr;
            SR_CUDA_TRY(cudaGetSymbolAddress(&p, g_verify_scratch));
            g_scratch_addr[dev] = p;
        }
        scratch = g_scratch_addr[dev];
    }
    // (the table of the rows' runs is used when it fits the scratch beside the hand-over area, else the terminal draw
    // reads the whole row)
    return run_verify(d, 1.0f, logits, parent_host, tree_tok, tree_cand, cand_id, cand_logit, u_acc, u_fin, n_acc,
                      path_node, out_tok, term_node, term_kind, row_max, row_sum, min_margin, nullptr, nullptr, scratch,
                      STATIC_SCRATCH_BYTES, cuda_stream, /*runs_optional=*/true);
}
