// Shared vocabulary projection with fused per-row top-k on the 5th-generation tensor cores.
//
//   logits[r, v] = Zt[r, :] . W[v, :]      r < M = B*K rows,  v < V,  contraction over d
//
// Persistent warp-specialised kernel, one CTA per SM:
//   warp 0   TMA producer: 128x64 tile of Zt and 256x64 tile of W per stage, 128-byte swizzle
//   warp 1   allocates TMEM and issues tcgen05.mma (M=128, N=256, K=16), fp32 accumulators in
//            TMEM, two accumulator buffers so the epilogue of tile i overlaps the MMAs of tile i+1
//   warps 2-5 epilogue: tcgen05.ld, thread = row; each thread keeps the running top list of its row
//            in registers across all vocabulary tiles of the CTA, so logits never leave the SM
// A CTA owns one block of 128 rows and a contiguous range of vocabulary tiles; CTAs that share a
// vocabulary range run side by side, so each W tile is fetched from HBM once and re-read from L2.
// Partial lists go to pval/pid[M, n_groups, k] and are merged by topk_merge_kernel.
#include "tc05.cuh"

namespace specroll {

#ifdef SPECROLL_CHECK
// Debug build only: when armed (specroll_check_inject(1)), CTA 0 leaves out the signal "first accumulator complete"
// once.  The epilogue warps' wait for it then runs into its time limit, which is how the test reaches the path on
// which every role gives up, tensor memory is released and the kernel returns SPECROLL_ETIMEOUT.  Only an arrival
// on a barrier is left out: no copy or tensor operation is abandoned.
static __device__ int g_drop_one_signal;
int lm_head_arm_dropped_signal() {
    const int one = 1;
    return cudaMemcpyToSymbol(g_drop_one_signal, &one, sizeof(one)) == cudaSuccess ? SPECROLL_OK : SPECROLL_ECUDA;
}
#else
int lm_head_arm_dropped_signal() { return -1; }
#endif

namespace lmtc {
constexpr int BM = 128, BN = 256, BK = 64, STAGES = 4, UMMA_K = 16;
constexpr int A_BYTES = BM * BK * 2, B_BYTES = BN * BK * 2, STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int THREADS = 192;
constexpr int TMEM_COLS = 512;  // two 256-column accumulator buffers
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
constexpr int KMAX = 8;
}  // namespace lmtc

struct TopList8 {
    float v[lmtc::KMAX];
    int32_t id[lmtc::KMAX];
    __device__ __forceinline__ void init() {
#pragma unroll
        for (int i = 0; i < lmtc::KMAX; ++i) {
            v[i] = -INFINITY;
            id[i] = 0x7fffffff;
        }
    }
    // ids arrive in increasing order, so "strictly greater" keeps the lowest id on ties
    __device__ __forceinline__ void push(float x, int32_t t) {
#pragma unroll
        for (int i = lmtc::KMAX - 1; i > 0; --i) {
            if (x > v[i - 1]) {
                v[i] = v[i - 1];
                id[i] = id[i - 1];
            } else if (x > v[i]) {
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

__global__ void __launch_bounds__(lmtc::THREADS, 1)
lm_head_topk_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, int M,
                       int V, int d, int k, int n_mblocks, int n_groups, int tiles_per_group,
                       float *__restrict__ pval, int32_t *__restrict__ pid, int32_t *__restrict__ status) {
    using namespace lmtc;
    extern __shared__ unsigned char smem_raw[];
    pdl_launch_dependents();
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
    pdl_wait();  // set up under the tail of the kernel before; its outputs are read from here on

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
                bool signal = ok;
#ifdef SPECROLL_CHECK
                if (t == 0 && blockIdx.x == 0 && atomicExch(&g_drop_one_signal, 0) == 1) signal = false;
#endif
                if (signal) umma_commit(tfull_bar(buf));  // accumulator complete
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..5)
        const int lg = warp & 3;  // TMEM lane group this warp may read: lanes 32*lg .. 32*lg+31
        const int row = lg * 32 + lane;
        TopList8 top;
        top.init();
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
                uint32_t r[32];
                tmem_ld32(taddr + (uint32_t)c, r);
                tmem_ld_wait();
                if (c + 32 <= ncol) {
                    // Four at a time: one branch on their maximum, which is rarely above the list's last entry.
                    // (One branch per element made this loop, with a single warp per scheduler to hide nothing
                    // behind, slower than the MMAs of a tile: 16 k against 12 k cycles.)
#pragma unroll
                    for (int i = 0; i < 32; i += 4) {
                        const float x0 = __uint_as_float(r[i]), x1 = __uint_as_float(r[i + 1]);
                        const float x2 = __uint_as_float(r[i + 2]), x3 = __uint_as_float(r[i + 3]);
                        if (fmaxf(fmaxf(x0, x1), fmaxf(x2, x3)) > top.v[KMAX - 1]) {
                            if (x0 > top.v[KMAX - 1]) top.push(x0, n0 + c + i);
                            if (x1 > top.v[KMAX - 1]) top.push(x1, n0 + c + i + 1);
                            if (x2 > top.v[KMAX - 1]) top.push(x2, n0 + c + i + 2);
                            if (x3 > top.v[KMAX - 1]) top.push(x3, n0 + c + i + 3);
                        }
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        const float x = __uint_as_float(r[i]);
                        if (c + i < ncol && x > top.v[KMAX - 1]) top.push(x, n0 + c + i);
                    }
                }
            }
            tc_fence_before();
            mbar_arrive(tempty_bar(buf));
        }
        if (m0 + row < M && !*abort_flag) {
            const size_t o = ((size_t)(m0 + row) * n_groups + grp) * k;
#pragma unroll
            for (int i = 0; i < KMAX; ++i)
                if (i < k) {
                    pval[o + i] = top.v[i];
                    pid[o + i] = top.id[i];
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

// Host launcher.  Zt[M, d], W[V, d] bf16; partial lists [M, n_groups, k].
int launch_lm_head_tc(const void *Zt, const void *W, int M, int V, int d, int k, int n_mblocks, int n_groups,
                      int tiles_per_group, float *pval, int32_t *pid, int32_t *status, cudaStream_t st) {
    using namespace lmtc;
    CUtensorMap tmA, tmB;
    int rc = make_tmap_2d_bf16(&tmA, Zt, (uint64_t)M, (uint64_t)d, (uint64_t)d, BM);
    if (rc != SPECROLL_OK) return rc;
    rc = make_tmap_2d_bf16(&tmB, W, (uint64_t)V, (uint64_t)d, (uint64_t)d, BN);
    if (rc != SPECROLL_OK) return rc;
    if ((rc = device_setup(reinterpret_cast<const void *>(lm_head_topk_tc_kernel), SMEM_BYTES, nullptr)) != SPECROLL_OK) return rc;
    // (the dependent of the correction kernel in the stream)
    SR_CUDA_TRY(launch_dependent(true, lm_head_topk_tc_kernel, dim3(n_mblocks * n_groups), dim3(THREADS), SMEM_BYTES, st, tmA,
                                 tmB, M, V, d, k, n_mblocks, n_groups, tiles_per_group, pval, pid, status));
    return SPECROLL_OK;
}

}  // namespace specroll
