// Baseline bf16 "TN" GEMM tile on legacy tensor-core instructions (mma.sync m16n8k16):
// C[BM x BN] += A[M, Kd] (row-major) * B[N, Kd]^T (row-major), fp32 accumulation.
// cp.async multi-stage pipeline, 128-byte rows with a 16-byte-chunk XOR swizzle, ldmatrix
// operand fetch.  Used where the tcgen05 path does not apply (small or oddly shaped problems).
#pragma once

#include "common.cuh"

namespace specroll {

template <int BM_, int BN_, int WM_, int WN_, int STAGES_>
struct MmaTile {
    static constexpr int BM = BM_, BN = BN_, WM = WM_, WN = WN_, STAGES = STAGES_;
    static constexpr int BK = 64;  // 128 bytes of bf16 per smem row
    static constexpr int THREADS = WM * WN * 32;
    static constexpr int WTM = BM / WM, WTN = BN / WN;  // warp tile
    static constexpr int MT = WTM / 16, NT = WTN / 8;
    static constexpr int A_BYTES = BM * BK * 2, B_BYTES = BN * BK * 2;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES;
    static_assert(WTM % 16 == 0 && WTN % 16 == 0, "warp tile must be a multiple of 16x16");

    // Copies rows [r0, r0+ROWS) x k-columns [k0, k0+64) of a row-major matrix into swizzled smem.
    template <int ROWS>
    static __device__ __forceinline__ void load_rows(uint32_t sbase, const __nv_bfloat16 *g, int ld,
                                                     int r0, int rmax, int k0) {
        constexpr int CHUNKS = ROWS * 8;
        for (int c = threadIdx.x; c < CHUNKS; c += THREADS) {
            const int row = c >> 3, ch = c & 7;
            const bool ok = (r0 + row) < rmax;
            const __nv_bfloat16 *src = g + (size_t)(ok ? r0 + row : 0) * ld + k0 + ch * 8;
            cp_async16(sbase + row * 128 + ((ch ^ (row & 7)) << 4), src, ok);
        }
    }

    static __device__ __forceinline__ void zero(float (&acc)[MT][NT][4]) {
#pragma unroll
        for (int i = 0; i < MT; ++i)
#pragma unroll
            for (int j = 0; j < NT; ++j)
#pragma unroll
                for (int t = 0; t < 4; ++t) acc[i][j][t] = 0.f;
    }

    // One full K loop for the tile at (m0, n0).  All threads of the CTA must call it.
    static __device__ __forceinline__ void run(unsigned char *smem, const __nv_bfloat16 *A, int lda,
                                               int m0, int M, const __nv_bfloat16 *Bm, int ldb, int n0,
                                               int Nn, int Kd, float (&acc)[MT][NT][4]) {
        const uint32_t s0 = smem_u32(smem);
        const int KT = Kd / BK;
        const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
        const int wm0 = (warp / WN) * WTM, wn0 = (warp % WN) * WTN;
        zero(acc);
#pragma unroll
        for (int s = 0; s < STAGES - 1; ++s) {
            if (s < KT) {
                load_rows<BM>(s0 + s * STAGE_BYTES, A, lda, m0, M, s * BK);
                load_rows<BN>(s0 + s * STAGE_BYTES + A_BYTES, Bm, ldb, n0, Nn, s * BK);
            }
            cp_async_commit();
        }
        for (int kt = 0; kt < KT; ++kt) {
            cp_async_wait<STAGES - 2>();
            __syncthreads();
            const int nx = kt + STAGES - 1;
            if (nx < KT) {
                const int st = nx % STAGES;
                load_rows<BM>(s0 + st * STAGE_BYTES, A, lda, m0, M, nx * BK);
                load_rows<BN>(s0 + st * STAGE_BYTES + A_BYTES, Bm, ldb, n0, Nn, nx * BK);
            }
            cp_async_commit();
            const uint32_t sa = s0 + (kt % STAGES) * STAGE_BYTES, sb = sa + A_BYTES;
#pragma unroll
            for (int kk = 0; kk < BK / 16; ++kk) {
                uint32_t af[MT][4], bfr[NT][2];
#pragma unroll
                for (int i = 0; i < MT; ++i) {
                    const int row = wm0 + i * 16 + (lane & 15), ch = kk * 2 + (lane >> 4);
                    ldmatrix_x4(af[i], sa + row * 128 + ((ch ^ (row & 7)) << 4));
                }
#pragma unroll
                for (int j = 0; j < NT / 2; ++j) {
                    const int row = wn0 + j * 16 + (lane & 7) + ((lane >> 4) << 3), ch = kk * 2 + ((lane >> 3) & 1);
                    uint32_t r[4];
                    ldmatrix_x4(r, sb + row * 128 + ((ch ^ (row & 7)) << 4));
                    bfr[2 * j][0] = r[0];
                    bfr[2 * j][1] = r[1];
                    bfr[2 * j + 1][0] = r[2];
                    bfr[2 * j + 1][1] = r[3];
                }
#pragma unroll
                for (int i = 0; i < MT; ++i)
#pragma unroll
                    for (int j = 0; j < NT; ++j) mma_bf16_16816(acc[i][j], af[i], bfr[j][0], bfr[j][1]);
            }
        }
        cp_async_wait<0>();
        __syncthreads();  // smem may be reused by the caller
    }
};

}  // namespace specroll
