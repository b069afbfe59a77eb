// Reliability side of the hidden-state correction (Sec. 3.4 "Reliability from delayed alignment", Eq.
// "reliability-score", the indicator of Eq. "reflex-correction"; App. "Implementation details", paragraph
// "Reflex configuration"): normalised random-projection sketches, realised alignments, exact online sample
// moments per (trajectory, horizon) slot, the conservative score and the gate that yields the correction ratio.
// Small, latency-bound kernels: a few thousand records and slots per call.
#include <math.h>

#include "common.cuh"

namespace specroll {

namespace gt {
constexpr int SK_THREADS = 256;
constexpr int MAX_RANK = 32;
}  // namespace gt

// One block per record: y = Pi x (rank dot products of length d), then y / ||y||.  A warp takes the ranks warp,
// warp + 8, ... (four at most) together, so x is read once per warp; with d % 4 == 0 and 16-byte aligned rows the
// loads are 128-bit and independent of the running sums, several in flight per lane.  (A record's x and Pi's rows
// are a few hundred KB fetched by one CTA: what bounds the kernel is how many bytes it keeps in flight.)
__global__ void __launch_bounds__(gt::SK_THREADS) sketch_kernel(int d, int rank, const float *__restrict__ X,
                                                                 const int32_t *__restrict__ rows,
                                                                 const float *__restrict__ Pi, float *__restrict__ sketch,
                                                                 int vec) {
    __shared__ float y[gt::MAX_RANK];
    constexpr int NW = gt::SK_THREADS / 32, RPW = gt::MAX_RANK / NW;
    const int r = blockIdx.x, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const float *x = X + (size_t)(rows ? rows[r] : r) * d;
    float acc[RPW];
#pragma unroll
    for (int q = 0; q < RPW; ++q) acc[q] = 0.f;
    if (vec) {
        const float4 *x4 = reinterpret_cast<const float4 *>(x);
        const float4 *p4 = reinterpret_cast<const float4 *>(Pi);
        const int d4 = d >> 2;
#pragma unroll 2
        for (int c = lane; c < d4; c += 32) {
            const float4 xv = x4[c];
#pragma unroll
            for (int q = 0; q < RPW; ++q) {
                const int i = warp + q * NW;
                if (i < rank) {
                    const float4 pv = p4[(size_t)i * d4 + c];
                    acc[q] = fmaf(pv.x, xv.x, fmaf(pv.y, xv.y, fmaf(pv.z, xv.z, fmaf(pv.w, xv.w, acc[q]))));
                }
            }
        }
    } else {
        for (int c = lane; c < d; c += 32) {
            const float xv = x[c];
#pragma unroll
            for (int q = 0; q < RPW; ++q) {
                const int i = warp + q * NW;
                if (i < rank) acc[q] = fmaf(Pi[(size_t)i * d + c], xv, acc[q]);
            }
        }
    }
#pragma unroll
    for (int q = 0; q < RPW; ++q) {
        const float t = warp_sum(acc[q]);
        if (lane == 0 && warp + q * NW < rank) y[warp + q * NW] = t;
    }
    __syncthreads();
    if (warp == 0) {
        const float v = lane < rank ? y[lane] : 0.f;
        const float nrm = sqrtf(warp_sum(v * v));
        if (lane < rank) sketch[(size_t)r * rank + lane] = nrm > 0.f ? v / nrm : 0.f;
    }
}

struct GateArgs {
    const float *s, *xi;
    const int32_t *slot;
    const uint8_t *keep;
    int32_t *n, *n_fb;
    float *mean, *M2;
    const float *m;
    const int32_t *horizon, *n_align_min, *n_fb_min;
    const float *alpha_lo, *alpha_hi;
    float *a, *rel, *alpha;
    int R, S, d, rank, H;
    float z_delta, mem_eps;
};

// Realised alignment of every record: a warp per record.
__global__ void __launch_bounds__(256) align_kernel(GateArgs g) {
    const int r = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (r >= g.R) return;
    if (g.keep && !g.keep[r]) {
        if (lane == 0 && g.a) g.a[r] = __int_as_float(0x7fc00000);
        return;
    }
    const float sv = lane < g.rank ? g.s[(size_t)r * g.rank + lane] : 0.f;
    const float xv = lane < g.rank ? g.xi[(size_t)r * g.rank + lane] : 0.f;
    const float dot = warp_sum(sv * xv), ns = sqrtf(warp_sum(sv * sv)), nx = sqrtf(warp_sum(xv * xv));
    if (lane == 0) g.a[r] = (ns > 0.f && nx > 0.f) ? dot / (ns * nx) : 0.f;
}

// A warp per slot: its records, in order, go into the running moments (lane 0 does the recurrences; the lanes
// look for the slot's records 32 at a time); then the score and the gate, with the RMS of the memory row.
__global__ void __launch_bounds__(256) gate_kernel(GateArgs g, const float *__restrict__ a) {
    const int j = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (j >= g.S) return;
    int n = g.n[j], nfb = g.n_fb[j];
    float mean = g.mean[j], M2 = g.M2[j];
    // the records in batches of 256: a lane's eight loads of a batch are independent of the recurrences
    for (int r0 = 0; r0 < g.R; r0 += 256) {
        unsigned mine = 0u;
        float av[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int r = r0 + q * 32 + lane;
            const bool mq = r < g.R && g.slot[r] == j && (!g.keep || g.keep[r]);
            mine |= (mq ? 1u : 0u) << q;
            av[q] = r < g.R ? a[r] : 0.f;
        }
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            unsigned bal = __ballot_sync(0xffffffffu, (mine >> q) & 1u);
            while (bal) {
                const int src = __ffs(bal) - 1;
                bal &= bal - 1;
                const float v = __shfl_sync(0xffffffffu, av[q], src);
                n += 1;
                const float delta = v - mean;
                mean += delta / (float)n;
                M2 += delta * (v - mean);
                nfb += 1;
            }
        }
    }
    float ss = 0.f;
    const float *mr = g.m + (size_t)j * g.d;
    if ((g.d % 4) == 0 && (reinterpret_cast<uintptr_t>(g.m) & 15u) == 0) {
        const float4 *m4 = reinterpret_cast<const float4 *>(mr);
        float s4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 4
        for (int c = lane; c < (g.d >> 2); c += 32) {
            const float4 v = m4[c];
            s4[0] = fmaf(v.x, v.x, s4[0]);
            s4[1] = fmaf(v.y, v.y, s4[1]);
            s4[2] = fmaf(v.z, v.z, s4[2]);
            s4[3] = fmaf(v.w, v.w, s4[3]);
        }
        ss = (s4[0] + s4[1]) + (s4[2] + s4[3]);
    } else {
        for (int c = lane; c < g.d; c += 32) ss = fmaf(mr[c], mr[c], ss);
    }
    ss = warp_sum(ss);
    if (lane == 0) {
        g.n[j] = n;
        g.n_fb[j] = nfb;
        g.mean[j] = mean;
        g.M2[j] = M2;
        const int h = g.horizon[j];
        float rel = -INFINITY;
        if (n >= 2) rel = mean - g.z_delta * sqrtf(M2 / (float)(n - 1)) / sqrtf((float)n);
        const bool open = h >= 0 && h < g.H && n >= g.n_align_min[h] && nfb >= g.n_fb_min[h] && rel > 0.f &&
                          sqrtf(ss / (float)g.d) > g.mem_eps;
        g.rel[j] = rel;
        g.alpha[j] = open ? g.alpha_lo[h] + (g.alpha_hi[h] - g.alpha_lo[h]) * fminf(rel, 1.f) : 0.f;
    }
}

}  // namespace specroll

using namespace specroll;

extern "C" int specroll_reflex_sketch(int32_t R, int32_t d, int32_t rank, const float *X, const int32_t *rows,
                                      const float *Pi, float *sketch, void *cuda_stream) {
    if (R < 0 || d < 1 || rank < 1 || rank > gt::MAX_RANK) return SPECROLL_EINVAL;
    if (R == 0) return SPECROLL_OK;
    if (!X || !Pi || !sketch) return SPECROLL_EINVAL;
    const int vec = (d % 4) == 0 && aligned16(X) && aligned16(Pi);
    sketch_kernel<<<R, gt::SK_THREADS, 0, static_cast<cudaStream_t>(cuda_stream)>>>(d, rank, X, rows, Pi, sketch, vec);
    SR_LAUNCH_CHECK();
    return SPECROLL_OK;
}

extern "C" int specroll_reflex_gate(const specroll_gate_desc *d, const float *s, const float *xi, const int32_t *slot,
                                    const uint8_t *keep, int32_t *n, float *mean, float *M2, int32_t *n_fb,
                                    const float *m, const int32_t *horizon, const int32_t *n_align_min,
                                    const int32_t *n_fb_min, const float *alpha_lo, const float *alpha_hi, float *a,
                                    float *rel, float *alpha, void *cuda_stream) {
    if (!d || d->R < 0 || d->S < 1 || d->d < 1 || d->rank < 1 || d->rank > gt::MAX_RANK || d->H < 1 ||
        !(d->z_delta >= 0.f) || !(d->mem_eps >= 0.f) || d->flags != 0)
        return SPECROLL_EINVAL;
    if (!n || !mean || !M2 || !n_fb || !m || !horizon || !n_align_min || !n_fb_min || !alpha_lo || !alpha_hi || !rel ||
        !alpha)
        return SPECROLL_EINVAL;
    // the alignments are needed by the second kernel: without the caller's array there is nowhere to keep them
    if (d->R > 0 && (!s || !xi || !slot || !a)) return SPECROLL_EINVAL;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    GateArgs g;
    g.s = s;
    g.xi = xi;
    g.slot = slot;
    g.keep = keep;
    g.n = n;
    g.n_fb = n_fb;
    g.mean = mean;
    g.M2 = M2;
    g.m = m;
    g.horizon = horizon;
    g.n_align_min = n_align_min;
    g.n_fb_min = n_fb_min;
    g.alpha_lo = alpha_lo;
    g.alpha_hi = alpha_hi;
    g.a = a;
    g.rel = rel;
    g.alpha = alpha;
    g.R = d->R;
    g.S = d->S;
    g.d = d->d;
    g.rank = d->rank;
    g.H = d->H;
    g.z_delta = d->z_delta;
    g.mem_eps = d->mem_eps;
    if (d->R > 0) {
        align_kernel<<<(d->R + 7) / 8, 256, 0, st>>>(g);
        SR_LAUNCH_CHECK();
    }
    gate_kernel<<<(d->S + 7) / 8, 256, 0, st>>>(g, a);
    SR_LAUNCH_CHECK();
    return SPECROLL_OK;
}
