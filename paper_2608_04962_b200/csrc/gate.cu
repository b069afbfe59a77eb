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

// One block per record: y = Pi x (rank dot products of length d, a warp each, round robin), then y / ||y||.
__global__ void __launch_bounds__(gt::SK_THREADS) sketch_kernel(int d, int rank, const float *__restrict__ X,
                                                                 const int32_t *__restrict__ rows,
                                                                 const float *__restrict__ Pi, float *__restrict__ sketch) {
    __shared__ float y[gt::MAX_RANK];
    const int r = blockIdx.x, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const float *x = X + (size_t)(rows ? rows[r] : r) * d;
    for (int i = warp; i < rank; i += gt::SK_THREADS / 32) {
        const float *p = Pi + (size_t)i * d;
        float acc = 0.f;
        for (int c = lane; c < d; c += 32) acc = fmaf(p[c], x[c], acc);
        acc = warp_sum(acc);
        if (lane == 0) y[i] = acc;
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
    for (int r0 = 0; r0 < g.R; r0 += 32) {
        const int r = r0 + lane;
        const bool mine = r < g.R && g.slot[r] == j && (!g.keep || g.keep[r]);
        unsigned bal = __ballot_sync(0xffffffffu, mine);
        while (bal) {
            const int src = __ffs(bal) - 1;
            bal &= bal - 1;
            const float av = a[r0 + src];
            n += 1;
            const float delta = av - mean;
            mean += delta / (float)n;
            M2 += delta * (av - mean);
            nfb += 1;
        }
    }
    float ss = 0.f;
    const float *mr = g.m + (size_t)j * g.d;
    for (int c = lane; c < g.d; c += 32) ss = fmaf(mr[c], mr[c], ss);
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
    sketch_kernel<<<R, gt::SK_THREADS, 0, static_cast<cudaStream_t>(cuda_stream)>>>(d, rank, X, rows, Pi, sketch);
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
