// Exact target verification: softmax statistics of every tree node, the node-wise
// accept / resample walk, and the terminal (fallback or bonus) draw.
//
// Three launches per call:
//   row_stats_kernel    one CTA per (sequence, node) row: streams the bf16 logits once with
//                       128-bit loads and keeps an online (max, sum-exp) pair per thread.
//   walk_kernel         one warp per sequence.  The residual of the walk differs from p only
//                       on the <= k candidates of the current node (the proposal is zero
//                       elsewhere), so it is tracked as k numbers plus one scale for the
//                       rest of the vocabulary, all in fp64.
//   terminal_kernel     one CTA per sequence: inverse-CDF draw over the vocabulary in token
//                       order with fp64 segment sums; the walk's <= k residual entries override
//                       the plain softmax mass.
#include <math.h>

#include <mutex>

#include "common.cuh"

namespace specroll {

constexpr int RS_THREADS = 256;
constexpr int RS_UNROLL = 4;
constexpr int WALK_WARPS = 4;
constexpr int TERM_THREADS = 512;  // two CTAs per SM
constexpr int TERM_WARPS = TERM_THREADS / 32;
constexpr float NEG_INF = -INFINITY;

// ------------------------------------------------------------------------------ row statistics

__device__ __forceinline__ void online_update(const uint4 &v, float c, float &m, float &s) {
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
    }
    float acc = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) acc += ex2_approx((x[i] - m) * c);
    s += acc;
}

// logits[rows, V] bf16; c = log2(e) / T.  row_max = max_v l_v, row_sum = sum_v exp((l_v - max)/T).
__global__ void __launch_bounds__(RS_THREADS)
row_stats_kernel(const uint16_t *__restrict__ logits, int V, float c, float *__restrict__ row_max,
                 float *__restrict__ row_sum) {
    const size_t row = blockIdx.x;
    const uint4 *p = reinterpret_cast<const uint4 *>(logits + row * (size_t)V);
    const int nvec = V >> 3;
    float m = NEG_INF, s = 0.f;
    int i = threadIdx.x;
    for (; i + (RS_UNROLL - 1) * RS_THREADS < nvec; i += RS_UNROLL * RS_THREADS) {
        uint4 v[RS_UNROLL];
#pragma unroll
        for (int u = 0; u < RS_UNROLL; ++u) v[u] = ld_nc_v4(p + i + u * RS_THREADS);
#pragma unroll
        for (int u = 0; u < RS_UNROLL; ++u) online_update(v[u], c, m, s);
    }
    for (; i < nvec; i += RS_THREADS) online_update(ld_nc_v4(p + i), c, m, s);

    // warp, then block reduction of (m, s)
    float mw = warp_max(m);
    s = (m == NEG_INF) ? 0.f : s * ex2_approx((m - mw) * c);
    s = warp_sum(s);
    __shared__ float sm_m[RS_THREADS / 32], sm_s[RS_THREADS / 32];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) {
        sm_m[warp] = mw;
        sm_s[warp] = s;
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

// ------------------------------------------------------------------------------ walk

struct WalkArgs {
    const uint16_t *logits;
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

__global__ void __launch_bounds__(WALK_WARPS * 32) walk_kernel(WalkArgs a, Topo topo) {
    __shared__ double sh_r[WALK_WARPS][SPECROLL_MAX_TOPK];
    __shared__ double sh_w[WALK_WARPS][SPECROLL_MAX_TOPK];
    __shared__ float sh_cl[WALK_WARPS][SPECROLL_MAX_TOPK];
    __shared__ int32_t sh_id[WALK_WARPS][SPECROLL_MAX_TOPK];
    __shared__ double sh_bc[WALK_WARPS][2];  // broadcast slots: current max, accepted flag

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int b = blockIdx.x * WALK_WARPS + warp;
    if (b >= a.B) return;
    double *r = sh_r[warp], *w = sh_w[warp];
    float *cl = sh_cl[warp];
    int32_t *id = sh_id[warp];
    const int k = a.k, N = a.N, K = a.K;

    int u = 0, nacc = 0, kind = 0;
    double sigma = 1.0;  // residual of a token outside the candidate set = sigma * p(token)
    double p_off = 0.0;
    float mm = INFINITY;
    bool have_residual = false;
    if (lane == 0) {
        for (int i = 0; i <= K; ++i) a.path_node[(size_t)b * (K + 1) + i] = a.out_tok[(size_t)b * (K + 1) + i] = -1;
        a.path_node[(size_t)b * (K + 1)] = 0;
    }
    for (;;) {
        if (topo.n_child[u] == 0) {
            kind = (u != 0) ? 1 : 0;
            have_residual = false;
            break;
        }
        const int hd = topo.depth[u];
        const double M = (double)a.row_max[(size_t)b * N + u];
        const double S = (double)a.row_sum[(size_t)b * N + u];
        const uint16_t *lg = a.logits + ((size_t)b * N + u) * a.V;
        for (int j = lane; j < k; j += 32) {
            const int t = a.cand_id[((size_t)b * K + hd) * k + j];
            id[j] = t;
            cl[j] = a.cand_logit[((size_t)b * K + hd) * k + j];
            const double l = (double)bf16_bits_to_float(lg[t]);
            r[j] = exp((l - M) / a.T) / S;  // r = p_u on the candidates
        }
        __syncwarp();
        sigma = 1.0;
        if (lane == 0) {
            double pc = 0.0;
            for (int j = 0; j < k; ++j) pc += r[j];
            p_off = 1.0 - pc;
            if (p_off < 0.0) p_off = 0.0;
        }
        uint64_t taken = 0;
        int accepted = -1;
        for (int c = u + 1; c < N && accepted < 0; ++c) {
            if (topo.parent[c] != u) continue;
            // slot proposal q on the candidates not yet taken
            if (lane == 0) {
                double mx = -INFINITY;
                for (int j = 0; j < k; ++j)
                    if (!((taken >> j) & 1) && (double)cl[j] > mx) mx = (double)cl[j];
                sh_bc[warp][0] = mx;
            }
            __syncwarp();
            const double mx = sh_bc[warp][0];
            for (int j = lane; j < k; j += 32)
                w[j] = ((taken >> j) & 1) ? 0.0 : exp(((double)cl[j] - mx) / a.T);
            __syncwarp();
            const int jc = a.tree_cand[(size_t)b * N + c];
            if (lane == 0) {
                double s = 0.0;
                for (int j = 0; j < k; ++j) s += w[j];
                const double qy = w[jc] / s;
                double ratio;
                if (qy > 0.0)
                    ratio = r[jc] / qy;
                else
                    ratio = (r[jc] > 0.0) ? INFINITY : 0.0;
                const double uu = (double)a.u_acc[(size_t)b * N + c];
                const float mg = (float)fabs(uu - ratio);
                if (mg < mm) mm = mg;
                if (uu < (ratio < 1.0 ? ratio : 1.0)) {
                    sh_bc[warp][1] = (double)c;
                } else {
                    sh_bc[warp][1] = -1.0;
                    double Z = 0.0;
                    for (int j = 0; j < k; ++j) {
                        const double t = r[j] - w[j] / s;
                        w[j] = t > 0.0 ? t : 0.0;
                        Z += w[j];
                    }
                    Z += sigma * p_off;
                    if (Z > 1e-300) {
                        for (int j = 0; j < k; ++j) r[j] = w[j] / Z;
                        sigma /= Z;
                    }
                }
            }
            __syncwarp();
            accepted = (int)sh_bc[warp][1];
            taken |= 1ull << jc;
            __syncwarp();
        }
        if (accepted < 0) {
            kind = 0;
            have_residual = true;
            break;
        }
        if (lane == 0) {
            a.out_tok[(size_t)b * (K + 1) + nacc] = a.tree_tok[(size_t)b * N + accepted];
            a.path_node[(size_t)b * (K + 1) + nacc + 1] = accepted;
        }
        ++nacc;
        u = accepted;
    }
    // hand the residual over to the terminal draw
    if (have_residual) {
        const double S = (double)a.row_sum[(size_t)b * N + u];
        sigma = __shfl_sync(0xffffffffu, sigma, 0);
        for (int j = lane; j < k; j += 32) {
            a.ws_ovid[(size_t)b * k + j] = id[j];
            a.ws_ovm[(size_t)b * k + j] = r[j] * S / sigma;
        }
    }
    if (lane == 0) {
        a.ws_nov[b] = have_residual ? k : 0;
        a.n_acc[b] = nacc;
        a.term_node[b] = u;
        a.term_kind[b] = kind;
        if (a.min_margin) a.min_margin[b] = mm;
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
    int32_t *out_tok;
    int32_t B, N, K, k, V;
    float c;  // log2(e) / T
};

__device__ __forceinline__ void masses8(const uint4 &v, float M, float c, float (&e)[8]) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        e[2 * i] = ex2_approx((__uint_as_float(w[i] << 16) - M) * c);
        e[2 * i + 1] = ex2_approx((__uint_as_float(w[i] & 0xffff0000u) - M) * c);
    }
}

__device__ __forceinline__ double warp_incl_scan(double v, int lane) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        double t = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += t;
    }
    return v;
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
    const uint16_t *lg = a.logits + ((size_t)b * a.N + node) * a.V;
    const uint4 *p = reinterpret_cast<const uint4 *>(lg);
    const int nvec = a.V >> 3;
    const int vpw = (nvec + TERM_WARPS - 1) / TERM_WARPS;  // vectors per warp segment
    const int n_sl = (vpw + 31) / 32;                      // slices per segment
    const int v_lo = min(nvec, warp * vpw), v_hi = min(nvec, v_lo + vpw);

    if (threadIdx.x < nov) {
        sh_ovm[threadIdx.x] = a.ws_ovm[(size_t)b * a.k + threadIdx.x];
        sh_ovid[threadIdx.x] = a.ws_ovid[(size_t)b * a.k + threadIdx.x];
    }

    // pass 1: plain softmax mass of every slice, eight slices' loads in flight
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
            masses8(v[q], M, a.c, e);
            double acc = 0.0;
#pragma unroll
            for (int t = 0; t < 8; ++t) acc += (double)e[t];
            acc = warp_sum(acc);
            if (lane == 0 && s0 + q < n_sl) sh_slice[warp * n_sl + s0 + q] = acc;
        }
    }
    __syncthreads();
    // the walk's residual entries replace the plain mass of their tokens (at most k of them: one thread)
    if (threadIdx.x == 0) {
        for (int j = 0; j < nov; ++j) {
            const int t = sh_ovid[j], vi = t >> 3;
            const int w = min(TERM_WARPS - 1, vi / vpw), sl = (vi - w * vpw) >> 5;
            sh_slice[w * n_sl + sl] += sh_ovm[j] - (double)ex2_approx((bf16_bits_to_float(lg[t]) - M) * a.c);
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
                double ms = (double)ex2_approx((bf16_bits_to_float(lg[tok]) - M) * a.c);
                for (int j = 0; j < nov; ++j)
                    if (sh_ovid[j] == tok) ms = sh_ovm[j];
                if (ms > 0.0) break;
            }
            *dst = tok;
        }
        return;
    }
    if (warp != wsel) return;

    // the slice inside the selected segment: first one whose running mass exceeds the target; if rounding made
    // the slices fall short of the segment's own sum, the last slice with positive mass
    const double target = sh_base[1];
    double base = sh_base[0];
    int sl_sel = -1, sl_pos = -1;
    double base_pos = 0.0;
    for (int c0 = 0; c0 < n_sl && sl_sel < 0; c0 += 32) {
        const double v = (c0 + lane < n_sl) ? sh_slice[warp * n_sl + c0 + lane] : 0.0;
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
    double lsum = 0.0;
    if (i < v_hi) {
        float e[8];
        masses8(ld_nc_v4(p + i), M, a.c, e);
#pragma unroll
        for (int t = 0; t < 8; ++t) ms[t] = (double)e[t];
        for (int j = 0; j < nov; ++j) {
            const int off = sh_ovid[j] - i * 8;
            if (off >= 0 && off < 8) {
#pragma unroll
                for (int t = 0; t < 8; ++t)
                    if (t == off) ms[t] = sh_ovm[j];
            }
        }
#pragma unroll
        for (int t = 0; t < 8; ++t) lsum += ms[t];
    } else {
#pragma unroll
        for (int t = 0; t < 8; ++t) ms[t] = 0.0;
    }
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
        !(d->temperature > 0.f) || d->flags != 0)
        return SPECROLL_EINVAL;
    return SPECROLL_OK;
}

extern "C" size_t specroll_verify_workspace_bytes(const specroll_verify_desc *d) {
    if (check_verify_desc(d) != SPECROLL_OK) return 0;
    size_t B = (size_t)d->B, k = (size_t)d->k;
    return align_up(B * k * sizeof(double), 256) + align_up(B * k * sizeof(int32_t), 256) +
           align_up(B * sizeof(int32_t), 256) + 256;
}

extern "C" int specroll_verify(const specroll_verify_desc *d, const void *logits,
                               const int32_t *parent_host, const int32_t *tree_tok,
                               const uint8_t *tree_cand, const int32_t *cand_id,
                               const float *cand_logit, const float *u_acc, const float *u_fin,
                               int32_t *n_acc, int32_t *path_node, int32_t *out_tok,
                               int32_t *term_node, int32_t *term_kind, float *row_max,
                               float *row_sum, float *min_margin, void *workspace,
                               size_t workspace_bytes, void *cuda_stream) {
    if (check_verify_desc(d) != SPECROLL_OK) return SPECROLL_EINVAL;
    if (!logits || !tree_tok || !tree_cand || !cand_id || !cand_logit || !u_acc || !u_fin || !n_acc ||
        !path_node || !out_tok || !term_node || !term_kind || !row_max || !row_sum)
        return SPECROLL_EINVAL;
    Topo topo;
    if (build_topo(parent_host, d->N, d->K, d->k, &topo, nullptr) != SPECROLL_OK) return SPECROLL_EINVAL;
    if (!aligned16(logits)) return SPECROLL_EALIGN;
    if (d->B == 0) return SPECROLL_OK;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) ||
        workspace_bytes < specroll_verify_workspace_bytes(d))
        return SPECROLL_EWORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const size_t B = (size_t)d->B, k = (size_t)d->k;
    char *ws = static_cast<char *>(workspace);
    double *ws_ovm = reinterpret_cast<double *>(ws);
    ws += align_up(B * k * sizeof(double), 256);
    int32_t *ws_ovid = reinterpret_cast<int32_t *>(ws);
    ws += align_up(B * k * sizeof(int32_t), 256);
    int32_t *ws_nov = reinterpret_cast<int32_t *>(ws);

    const float c = (float)(1.4426950408889634 / (double)d->temperature);
    const int rows = d->B * d->N;
    row_stats_kernel<<<rows, RS_THREADS, 0, st>>>(static_cast<const uint16_t *>(logits), d->V, c, row_max,
                                                  row_sum);
    SR_LAUNCH_CHECK();

    WalkArgs wa;
    wa.logits = static_cast<const uint16_t *>(logits);
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
    walk_kernel<<<(d->B + WALK_WARPS - 1) / WALK_WARPS, WALK_WARPS * 32, 0, st>>>(wa, topo);
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
    ta.out_tok = out_tok;
    ta.B = d->B;
    ta.N = d->N;
    ta.K = d->K;
    ta.k = d->k;
    ta.V = d->V;
    ta.c = c;
    return launch_terminal(ta, st);
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
    if (specroll_verify_workspace_bytes(d) > STATIC_SCRATCH_BYTES) return SPECROLL_ELIMIT;
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
    return specroll_verify(d, logits, parent_host, tree_tok, tree_cand, cand_id, cand_logit, u_acc, u_fin, n_acc,
                           path_node, out_tok, term_node, term_kind, row_max, row_sum, min_margin, scratch,
                           STATIC_SCRATCH_BYTES, cuda_stream);
}
