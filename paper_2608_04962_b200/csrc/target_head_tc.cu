// The target's vocabulary projection with the verification's row statistics fused into its epilogue, so that
// the target logits of the tree nodes never reach HBM (Sec. 3.2: "evaluate p_u for every unique tree prefix in one
// packed target forward"; App. B.2 needs, per node, the softmax normaliser and the probabilities of the node's
// candidate tokens only; the one full row per sequence that the terminal draw needs is produced afterwards by
// the same kernel in its storing form).
//
//   l[r, v] = bf16( H[r, :] . W[v, :] )         r < R rows (sequence, node),  v < V,  contraction over d
//   row_max[r] = max_v l[r, v],   row_sum[r] = sum_v exp((l[r, v] - row_max[r]) / T)
//   want_logit[r, q] = l[r, want_id[r, q]]      (the node's candidate tokens)
//
// The logits are rounded to bf16 before they are used, which is what a projection that stores them would have
// handed to the verification.  Same pipeline as the proposal's projection: persistent warp-specialised CTAs, TMA
// producer, one MMA-issuing thread (tcgen05, M=128, N=256, K=16, two accumulator buffers in TMEM), four epilogue
// warps with one thread per row.  A CTA owns a block of 128 rows and a contiguous range of vocabulary tiles; the
// per-(row, range) partial statistics are merged by a small kernel.
#include "tc05.cuh"

namespace specroll {

namespace thtc {
constexpr int BM = 128, BN = 256, BK = 64, STAGES = 4, UMMA_K = 16;
constexpr int A_BYTES = BM * BK * 2, B_BYTES = BN * BK * 2, STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int THREADS = 192;
constexpr int TMEM_COLS = 512;  // two 256-column accumulator buffers
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
constexpr int KW_MAX = 8;  // wanted tokens per row
}  // namespace thtc

// STORE = false: statistics and wanted logits;  STORE = true: the logits themselves, as bf16.
template <bool STORE>
__global__ void __launch_bounds__(thtc::THREADS, 1)
target_head_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, int M, int V,
                      int d, int n_mblocks, int n_groups, int tiles_per_group, float c_log2,
                      const int32_t *__restrict__ want_id, int kw, float *__restrict__ pm, float *__restrict__ ps,
                      uint16_t *__restrict__ want_logit, uint16_t *__restrict__ logits_out,
                      int32_t *__restrict__ status) {
    using namespace thtc;
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;  // 1024-byte alignment for the 128-byte swizzle atoms
    unsigned char *aligned = smem_raw + (base - raw);
    uint64_t *bars = reinterpret_cast<uint64_t *>(aligned + STAGES * STAGE_BYTES);
    // barrier slots: full[STAGES], empty[STAGES], tmem_full[2], tmem_empty[2]
    const uint32_t bar0 = base + STAGES * STAGE_BYTES;
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (STAGES + s); };
    auto tfull_bar = [&](int b) { return bar0 + 8u * (2 * STAGES + b); };
    auto tempty_bar = [&](int b) { return bar0 + 8u * (2 * STAGES + 2 + b); };
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * STAGES + 4);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int mb = blockIdx.x % n_mblocks, grp = blockIdx.x / n_mblocks;
    const int m0 = mb * BM;
    const int n_tiles = (V + BN - 1) / BN;
    const int t_lo = min(n_tiles, grp * tiles_per_group), t_hi = min(n_tiles, t_lo + tiles_per_group);
    const int KB = d / BK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(tfull_bar(b), 1);
            mbar_init(tempty_bar(b), 128);
        }
        *abort_flag = 0;
        fence_mbar_init();
        prefetch_tmap(&tmA);
        prefetch_tmap(&tmB);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            int issued[STAGES];
#pragma unroll
            for (int s = 0; s < STAGES; ++s) issued[s] = -1;
            bool ok = true;
            for (int tile = t_lo; tile < t_hi && ok; ++tile) {
                for (int kb = 0; kb < KB; ++kb) {
                    if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) {
                        ok = false;
                        break;
                    }
                    const uint32_t sa = base + stage * STAGE_BYTES, sb = sa + A_BYTES;
                    mbar_arrive_expect_tx(full_bar(stage), STAGE_BYTES);
                    tma_load_2d(sa, &tmA, kb * BK, m0, full_bar(stage));
                    tma_load_2d(sb, &tmB, kb * BK, tile * BN, full_bar(stage));
                    issued[stage] = (int)phase;
                    if (++stage == STAGES) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
            }
            if (!ok) {
                // aborting: let the copies already in flight land before the CTA goes away
#pragma unroll
                for (int s = 0; s < STAGES; ++s)
                    if (issued[s] >= 0) {
                        const unsigned long long t0 = globaltimer_ns();
                        while (!mbar_try_wait(full_bar(s), (uint32_t)issued[s]) &&
                               globaltimer_ns() - t0 < 100000000ull) {
                        }
                    }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = idesc_bf16(BM, BN, false, false);
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            int t = 0;
            for (int tile = t_lo; tile < t_hi && ok; ++tile, ++t) {
                const int buf = t & 1;
                const uint32_t acc_phase = (uint32_t)(t >> 1) & 1u;
                if (!mbar_wait(tempty_bar(buf), acc_phase ^ 1u, abort_flag)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * BN);
                for (int kb = 0; kb < KB; ++kb) {
                    if (!mbar_wait(full_bar(stage), phase, abort_flag)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t sa = base + stage * STAGE_BYTES, sb = sa + A_BYTES;
                    const uint64_t adesc = smem_desc_sw128(sa, 1024, 0), bdesc = smem_desc_sw128(sb, 1024, 0);
#pragma unroll
                    for (int kk = 0; kk < BK / UMMA_K; ++kk) {
                        // advancing K by 16 elements = 32 bytes = 2 descriptor address units
                        umma_ss(d_tmem, adesc + 2u * kk, bdesc + 2u * kk, idesc, (kb | kk) != 0 ? 1u : 0u);
                    }
                    umma_commit(empty_bar(stage));  // stage reusable once these MMAs have read it
                    if (++stage == STAGES) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
                if (ok) umma_commit(tfull_bar(buf));  // accumulator complete
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..5), thread = row
        const int lg = warp & 3;  // TMEM lane group this warp may read: lanes 32*lg .. 32*lg+31
        const int row = lg * 32 + lane;
        const bool row_ok = m0 + row < M;
        float m_run = -INFINITY, s_run = 0.f;  // online maximum (of the logits) and sum of exp((l - m) / T)
        int32_t want[KW_MAX];
#pragma unroll
        for (int q = 0; q < KW_MAX; ++q) want[q] = (!STORE && row_ok && q < kw) ? want_id[(size_t)(m0 + row) * kw + q] : -1;
        int t = 0;
        bool ok = true;
        for (int tile = t_lo; tile < t_hi && ok; ++tile, ++t) {
            const int buf = t & 1;
            const uint32_t acc_phase = (uint32_t)(t >> 1) & 1u;
            if (!mbar_wait(tfull_bar(buf), acc_phase, abort_flag)) break;
            tc_fence_after();
            const int n0 = tile * BN;
            const int ncol = min(BN, V - n0);
            const uint32_t taddr = tmem_base + ((uint32_t)(lg * 32) << 16) + (uint32_t)(buf * BN);
#pragma unroll 1
            for (int c = 0; c < BN; c += 32) {
                if (c >= ncol) break;  // (uniform) columns beyond the vocabulary
                uint32_t r[32];
                tmem_ld32(taddr + (uint32_t)c, r);
                tmem_ld_wait();
                // the logits as a storing projection would have left them: bf16
#pragma unroll
                for (int i = 0; i < 32; ++i)
                    r[i] = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(__uint_as_float(r[i]))) << 16;
                if constexpr (STORE) {
                    if (row_ok) {
                        uint16_t *dst = logits_out + (size_t)(m0 + row) * V + n0 + c;
                        if (c + 32 <= ncol) {
#pragma unroll
                            for (int i = 0; i < 32; i += 8) {
                                uint4 q4;
                                q4.x = (r[i] >> 16) | (r[i + 1] & 0xffff0000u);
                                q4.y = (r[i + 2] >> 16) | (r[i + 3] & 0xffff0000u);
                                q4.z = (r[i + 4] >> 16) | (r[i + 5] & 0xffff0000u);
                                q4.w = (r[i + 6] >> 16) | (r[i + 7] & 0xffff0000u);
                                *reinterpret_cast<uint4 *>(dst + i) = q4;
                            }
                        } else {
                            for (int i = 0; i < 32 && c + i < ncol; ++i) dst[i] = (uint16_t)(r[i] >> 16);
                        }
                    }
                } else {
                    const int nv = min(32, ncol - c);
                    float cm = -INFINITY;
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (i < nv) cm = fmaxf(cm, __uint_as_float(r[i]));
                    if (cm > m_run) {
                        s_run *= ex2_approx((m_run - cm) * c_log2);  // (0 * 2^-inf = 0 on the first chunk)
                        m_run = cm;
                    }
                    const float nm = -m_run * c_log2;
                    float s0 = 0.f, s1 = 0.f;
#pragma unroll
                    for (int i = 0; i < 32; i += 2) {
                        const float e0 = ex2_approx(fmaf(__uint_as_float(r[i]), c_log2, nm));
                        const float e1 = ex2_approx(fmaf(__uint_as_float(r[i + 1]), c_log2, nm));
                        s0 += (i < nv) ? e0 : 0.f;
                        s1 += (i + 1 < nv) ? e1 : 0.f;
                    }
                    s_run += s0 + s1;
                    // the row's wanted tokens that fall into these 32 columns (rare)
#pragma unroll
                    for (int q = 0; q < KW_MAX; ++q) {
                        const uint32_t off = (uint32_t)(want[q] - (n0 + c));
                        if (off < (uint32_t)nv) {
                            uint32_t val = 0;
#pragma unroll
                            for (int i = 0; i < 32; ++i)
                                if ((uint32_t)i == off) val = r[i];
                            want_logit[(size_t)(m0 + row) * kw + q] = (uint16_t)(val >> 16);
                        }
                    }
                }
            }
            tc_fence_before();
            mbar_arrive(tempty_bar(buf));
        }
        if (!STORE && row_ok && !*abort_flag) {
            pm[(size_t)(m0 + row) * n_groups + grp] = m_run;
            ps[(size_t)(m0 + row) * n_groups + grp] = s_run;
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

// row_max = max over the ranges, row_sum = sum of the ranges' sums brought to that maximum
__global__ void target_head_merge_kernel(const float *__restrict__ pm, const float *__restrict__ ps, int M, int n_groups,
                                         float c_log2, float *__restrict__ row_max, float *__restrict__ row_sum) {
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= M) return;
    float m = -INFINITY;
    for (int g = 0; g < n_groups; ++g) m = fmaxf(m, pm[(size_t)r * n_groups + g]);
    float s = 0.f;
    for (int g = 0; g < n_groups; ++g) {
        const float mg = pm[(size_t)r * n_groups + g];
        if (mg > -INFINITY) s += ps[(size_t)r * n_groups + g] * ex2_approx((mg - m) * c_log2);
    }
    row_max[r] = m;
    row_sum[r] = s;
}

}  // namespace specroll

using namespace specroll;

namespace {
struct HeadPlan {
    int n_mblocks, n_groups, tiles_per_group;
    size_t off_status, off_pm, off_ps, total;
};
int plan_head(int R, int V, HeadPlan *p) {
    using namespace thtc;
    p->n_mblocks = (R + BM - 1) / BM;
    const int n_tiles = (V + BN - 1) / BN;
    // Number of vocabulary ranges: the CTAs (row blocks x ranges) run in waves of one per SM; the estimate of a
    // plan is waves x (tiles per range + half a tile for a CTA's set-up and drain), and the candidate with the
    // lowest estimate wins (with 32 row blocks: 9 ranges in two full waves instead of 4 ranges on 128 SMs).
    int want = 1;
    double best = -1.0;
    for (int g = 1; g <= n_tiles && g <= 148; ++g) {
        const int tpg = (n_tiles + g - 1) / g, ng = (n_tiles + tpg - 1) / tpg;
        const long long ctas = (long long)(p->n_mblocks > 0 ? p->n_mblocks : 1) * ng;
        const double est = (double)((ctas + 147) / 148) * ((double)tpg + 0.5);
        if (best < 0.0 || est < best - 1e-9) {
            best = est;
            want = g;
        }
    }
    p->tiles_per_group = (n_tiles + want - 1) / want;
    p->n_groups = (n_tiles + p->tiles_per_group - 1) / p->tiles_per_group;
    size_t o = 0;
    p->off_status = o;
    o += 256;
    p->off_pm = o;
    o += align_up((size_t)R * p->n_groups * 4, 256);
    p->off_ps = o;
    o += align_up((size_t)R * p->n_groups * 4, 256);
    p->total = o + 256;
    return SPECROLL_OK;
}
bool head_shape_ok(int R, int d, int V) { return R >= 0 && d >= 64 && (d % 64) == 0 && V >= 8 && (V % 8) == 0; }
}  // namespace

extern "C" size_t specroll_target_head_stats_workspace_bytes(int32_t R, int32_t d, int32_t V) {
    if (!head_shape_ok(R, d, V)) return 0;
    HeadPlan p;
    plan_head(R, V, &p);
    return p.total;
}

extern "C" int specroll_target_head_stats(int32_t R, int32_t d, int32_t V, float temperature, const void *H, const void *W,
                                          const int32_t *want_id, int32_t kw, float *row_max, float *row_sum,
                                          void *want_logit, void *workspace, size_t workspace_bytes, void *cuda_stream) {
    using namespace thtc;
    if (!head_shape_ok(R, d, V) || !(temperature > 0.f) || kw < 0 || kw > KW_MAX) return SPECROLL_EINVAL;
    if (R == 0) return SPECROLL_OK;
    if (!H || !W || !row_max || !row_sum || (kw > 0 && (!want_id || !want_logit))) return SPECROLL_EINVAL;
    if (!aligned16(H) || !aligned16(W)) return SPECROLL_EALIGN;
    HeadPlan p;
    plan_head(R, V, &p);
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) || workspace_bytes < p.total) return SPECROLL_EWORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    unsigned char *ws = static_cast<unsigned char *>(workspace);
    int32_t *status = reinterpret_cast<int32_t *>(ws + p.off_status);
    float *pm = reinterpret_cast<float *>(ws + p.off_pm), *ps = reinterpret_cast<float *>(ws + p.off_ps);
    SR_CUDA_TRY(cudaMemsetAsync(status, 0, 256, st));
    CUtensorMap tmA, tmB;
    int rc = make_tmap_2d_bf16(&tmA, H, (uint64_t)R, (uint64_t)d, (uint64_t)d, BM);
    if (rc != SPECROLL_OK) return rc;
    rc = make_tmap_2d_bf16(&tmB, W, (uint64_t)V, (uint64_t)d, (uint64_t)d, BN);
    if (rc != SPECROLL_OK) return rc;
    if ((rc = device_setup(reinterpret_cast<const void *>(target_head_tc_kernel<false>), SMEM_BYTES, nullptr)) != SPECROLL_OK) return rc;
    const float c_log2 = 1.4426950408889634f / temperature;
    target_head_tc_kernel<false><<<p.n_mblocks * p.n_groups, THREADS, SMEM_BYTES, st>>>(
        tmA, tmB, R, V, d, p.n_mblocks, p.n_groups, p.tiles_per_group, c_log2, want_id, kw, pm, ps,
        static_cast<uint16_t *>(want_logit), nullptr, status);
    SR_LAUNCH_CHECK();
    target_head_merge_kernel<<<(R + 255) / 256, 256, 0, st>>>(pm, ps, R, p.n_groups, c_log2, row_max, row_sum);
    SR_LAUNCH_CHECK();
    return SPECROLL_OK;
}

extern "C" int specroll_target_head_rows(int32_t R, int32_t d, int32_t V, const void *H, const void *W, void *logits,
                                         int32_t *status, void *cuda_stream) {
    using namespace thtc;
    if (!head_shape_ok(R, d, V)) return SPECROLL_EINVAL;
    if (R == 0) return SPECROLL_OK;
    if (!H || !W || !logits || !status) return SPECROLL_EINVAL;
    if (!aligned16(H) || !aligned16(W) || !aligned16(logits)) return SPECROLL_EALIGN;
    HeadPlan p;
    plan_head(R, V, &p);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    SR_CUDA_TRY(cudaMemsetAsync(status, 0, 4, st));
    CUtensorMap tmA, tmB;
    int rc = make_tmap_2d_bf16(&tmA, H, (uint64_t)R, (uint64_t)d, (uint64_t)d, BM);
    if (rc != SPECROLL_OK) return rc;
    rc = make_tmap_2d_bf16(&tmB, W, (uint64_t)V, (uint64_t)d, (uint64_t)d, BN);
    if (rc != SPECROLL_OK) return rc;
    if ((rc = device_setup(reinterpret_cast<const void *>(target_head_tc_kernel<true>), SMEM_BYTES, nullptr)) != SPECROLL_OK) return rc;
    target_head_tc_kernel<true><<<p.n_mblocks * p.n_groups, THREADS, SMEM_BYTES, st>>>(
        tmA, tmB, R, V, d, p.n_mblocks, p.n_groups, p.tiles_per_group, 0.f, nullptr, 0, nullptr, nullptr, nullptr,
        static_cast<uint16_t *>(logits), status);
    SR_LAUNCH_CHECK();
    return SPECROLL_OK;
}
