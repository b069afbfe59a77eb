// Head MLPs (Eq. "heads", Appendix on the proposal heads) on the 5th-generation tensor cores:
//
//   z[b, hd, o] = h[b, o] + SiLU( sum_i A[hd, o, i] * xhat[b, i] + bias[hd, o] )          (fp32 out)
//
// The contraction has only B rows on the activation side, so it is bound by streaming the weights
// (K d^2 2 bytes, each needed once).  The weights are therefore the M operand: a CTA owns 128
// output units of one head and the whole batch block (N = 64, 128 or 256 sequences), walks the
// d inputs in slices of 64, and every weight element crosses HBM -> shared memory exactly once;
// the (small) activation block is re-read from L2 by each CTA.  When that gives fewer CTAs than SMs the batch
// is cut into narrower blocks, whose CTAs share the weight tile through L2.
//   warp 0   TMA producer: 128 x 64 weight tile and BN x 64 activation tile per stage (128-byte swizzle)
//   warp 1   allocates BN TMEM columns and issues tcgen05.mma (M=128, N=BN, K=16), fp32 accumulator in TMEM
//   warps 2-5 epilogue: tcgen05.ld, thread = output unit; bias, SiLU and the residual are applied on the
//            way out, consecutive lanes write consecutive output units of one sequence
// One tile per CTA; stage counts are chosen so that two CTAs share an SM for N <= 128.
#include "tc05.cuh"

namespace specroll {

namespace hmtc {
constexpr int BM = 128, BK = 64, UMMA_K = 16, THREADS = 192;
constexpr int W_BYTES = BM * BK * 2;
// DEEP: for grids of at most one CTA per SM, where what a CTA keeps in flight is all the machine has in flight: a
// stage holds two 64-wide slices of the contraction side by side (two boxes per operand), so a weight row arrives as
// 256 contiguous bytes instead of 128 (the weights are row-major [d_out, d_in]: every row of a box is its own DRAM
// page) and the ring holds twice the bytes; one CTA per SM.  Needs d % 128 == 0.
template <int BN, bool DEEP>
struct Cfg {
    static constexpr int NBOX = DEEP ? 2 : 1;
    static constexpr int X_BYTES = BN * BK * 2;  // one box
    static constexpr int STAGE_BYTES = NBOX * (W_BYTES + X_BYTES);
    static constexpr int STAGES = BN == 64 ? 4 : (BN == 128 ? 3 : 4);
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
};
}  // namespace hmtc

template <int BN, bool DEEP>
__global__ void __launch_bounds__(hmtc::THREADS)
head_mlp_tc_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX, int KX,
                   const __nv_bfloat16 *__restrict__ bias, const __nv_bfloat16 *__restrict__ h,
                   float *__restrict__ z, int B, int K, int d, int32_t *__restrict__ status) {
    using namespace hmtc;
    using C = Cfg<BN, DEEP>;
    constexpr int STAGES = C::STAGES;
    extern __shared__ unsigned char smem_raw[];
    pdl_launch_dependents();
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;  // 1024-byte alignment for the 128-byte swizzle atoms
    unsigned char *aligned = smem_raw + (base - raw);
    uint64_t *bars = reinterpret_cast<uint64_t *>(aligned + STAGES * C::STAGE_BYTES);
    // barrier slots: full[STAGES], empty[STAGES], acc_full
    const uint32_t bar0 = base + STAGES * C::STAGE_BYTES;
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (STAGES + s); };
    const uint32_t acc_bar = bar0 + 8u * (2 * STAGES);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * STAGES + 1);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int o0 = blockIdx.x * BM, b0 = blockIdx.y * BN, hd = blockIdx.z;
    constexpr int NBOX = C::NBOX;
    const int KB = d / (BK * NBOX);

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
        }
        mbar_init(acc_bar, 1);
        *abort_flag = 0;
        fence_mbar_init();
        prefetch_tmap(&tmW);
        prefetch_tmap(&tmX);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), BN);
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
            const int w_row = hd * d + o0;                  // rows of A viewed as [K * d, d]
            const int x_row = (KX > 1 ? hd * B : 0) + b0;   // rows of xhat viewed as [KX * B, d]
            bool ok = true;
            int kb = 0;
            for (; kb < KB; ++kb) {
                const int stage = kb % STAGES;
                if (!mbar_wait(empty_bar(stage), ((uint32_t)(kb / STAGES) & 1u) ^ 1u, abort_flag)) {
                    ok = false;
                    break;
                }
                const uint32_t sw = base + stage * C::STAGE_BYTES, sx = sw + NBOX * W_BYTES;
                mbar_arrive_expect_tx(full_bar(stage), C::STAGE_BYTES);
#pragma unroll
                for (int bx = 0; bx < NBOX; ++bx) {
                    tma_load_2d(sw + bx * W_BYTES, &tmW, (kb * NBOX + bx) * BK, w_row, full_bar(stage));
                    tma_load_2d(sx + bx * C::X_BYTES, &tmX, (kb * NBOX + bx) * BK, x_row, full_bar(stage));
                }
            }
            if (!ok) {
                // aborting: let the copies already in flight land before the CTA goes away
                for (int j = max(0, kb - STAGES); j < kb; ++j) {
                    const unsigned long long t0 = globaltimer_ns();
                    while (!mbar_try_wait(full_bar(j % STAGES), (uint32_t)(j / STAGES) & 1u) &&
                           globaltimer_ns() - t0 < 100000000ull) {
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = idesc_bf16(BM, BN, false, false);
            bool ok = true;
            for (int kb = 0; kb < KB; ++kb) {
                const int stage = kb % STAGES;
                if (!mbar_wait(full_bar(stage), (uint32_t)(kb / STAGES) & 1u, abort_flag)) {
                    ok = false;
                    break;
                }
                tc_fence_after();
                const uint32_t sw = base + stage * C::STAGE_BYTES, sx = sw + NBOX * W_BYTES;
#pragma unroll
                for (int bx = 0; bx < NBOX; ++bx) {
                    const uint64_t adesc = smem_desc_sw128(sw + bx * W_BYTES, 1024, 0);
                    const uint64_t bdesc = smem_desc_sw128(sx + bx * C::X_BYTES, 1024, 0);
#pragma unroll
                    for (int kk = 0; kk < BK / UMMA_K; ++kk)  // 16 inputs further = 32 bytes = 2 descriptor address units
                        umma_ss(tmem_base, adesc + 2u * kk, bdesc + 2u * kk, idesc, (kb | bx | kk) != 0 ? 1u : 0u);
                }
                umma_commit(empty_bar(stage));  // stage reusable once these MMAs have read it
            }
            if (ok) umma_commit(acc_bar);  // accumulator complete
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..5)
        const int lg = warp & 3;  // TMEM lane group this warp may read: lanes 32*lg .. 32*lg+31
        const int o = o0 + lg * 32 + lane;  // this thread's output unit
        if (mbar_wait(acc_bar, 0u, abort_flag)) {
            tc_fence_after();
            const float bo = o < d ? __bfloat162float(bias[(size_t)hd * d + o]) : 0.f;
            const uint32_t taddr = tmem_base + ((uint32_t)(lg * 32) << 16);
#pragma unroll 1
            for (int c = 0; c < BN; c += 32) {
                if (b0 + c >= B) break;  // uniform: the rest of the block is padding
                uint32_t r[32];
                tmem_ld32(taddr + (uint32_t)c, r);
                tmem_ld_wait();
                if (o < d) {
                    // all residual loads first: taken one by one between the stores, each would cost a full
                    // round trip to L2 (that made the epilogue three quarters of the kernel)
                    float hv[32];
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        const int b = min(b0 + c + i, B - 1);
                        hv[i] = __bfloat162float(h[(size_t)b * d + o]);
                    }
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        const int b = b0 + c + i;
                        if (b < B) {
                            const float y = __uint_as_float(r[i]) + bo;
                            const float sl = y / (1.0f + __expf(-y));
                            z[((size_t)b * K + hd) * d + o] = hv[i] + sl;
                        }
                    }
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
        tmem_dealloc(tmem_base, BN);
    }
}

template <int BN, bool DEEP>
static int launch_bn2(const CUtensorMap &tmW, const CUtensorMap &tmX, int KX, const void *bias, const void *h, float *z,
                      int B, int K, int d, int32_t *status, cudaStream_t st, dim3 grid) {
    using namespace hmtc;
    using C = Cfg<BN, DEEP>;
    const int rc = device_setup(reinterpret_cast<const void *>(head_mlp_tc_kernel<BN, DEEP>), C::SMEM_BYTES, nullptr);
    if (rc != SPECROLL_OK) return rc;
    // (the dependent of the LayerNorm kernel in the stream)
    SR_CUDA_TRY(launch_dependent(true, head_mlp_tc_kernel<BN, DEEP>, grid, dim3(THREADS), C::SMEM_BYTES, st, tmW, tmX, KX,
                                 static_cast<const __nv_bfloat16 *>(bias), static_cast<const __nv_bfloat16 *>(h), z, B, K, d,
                                 status));
    return SPECROLL_OK;
}

template <int BN>
static int launch_bn(const CUtensorMap &tmW, const void *xhat, int KX, const void *bias, const void *h, float *z,
                     int B, int K, int d, int32_t *status, cudaStream_t st) {
    using namespace hmtc;
    CUtensorMap tmX;
    int rc = make_tmap_2d_bf16(&tmX, xhat, (uint64_t)KX * B, (uint64_t)d, (uint64_t)d, BN);
    if (rc != SPECROLL_OK) return rc;
    int n_sm = 0;
    if ((rc = device_setup(nullptr, 0, &n_sm)) != SPECROLL_OK) return rc;
    const dim3 grid((unsigned)((d + BM - 1) / BM), (unsigned)((B + BN - 1) / BN), (unsigned)K);
    if (BN < 256 && (d % (2 * BK)) == 0 && (long long)grid.x * grid.y * grid.z <= n_sm)
        return launch_bn2<BN, BN < 256>(tmW, tmX, KX, bias, h, z, B, K, d, status, st, grid);
    return launch_bn2<BN, false>(tmW, tmX, KX, bias, h, z, B, K, d, status, st, grid);
}

// Host launcher.  xhat[KX, B, d], A[K, d, d] (row = output unit), bias[K, d], h[B, d] bf16; z[B, K, d] fp32.
int launch_head_mlp_tc(const void *xhat, int KX, const void *A, const void *bias, const void *h, float *z, int B,
                       int K, int d, int32_t *status, cudaStream_t st) {
    CUtensorMap tmW;
    int rc = make_tmap_2d_bf16(&tmW, A, (uint64_t)K * d, (uint64_t)d, (uint64_t)d, hmtc::BM);
    if (rc != SPECROLL_OK) return rc;
    // the widest batch block that still gives every SM a CTA (a narrower block re-reads the weight tile, but from
    // L2: the CTAs of one weight tile run side by side)
    const long long tiles = (long long)K * ((d + hmtc::BM - 1) / hmtc::BM);
    if (B > 128 && tiles * ((B + 255) / 256) >= 148) return launch_bn<256>(tmW, xhat, KX, bias, h, z, B, K, d, status, st);
    if (B > 64 && tiles * ((B + 127) / 128) >= 148) return launch_bn<128>(tmW, xhat, KX, bias, h, z, B, K, d, status, st);
    return launch_bn<64>(tmW, xhat, KX, bias, h, z, B, K, d, status, st);
}

}  // namespace specroll
