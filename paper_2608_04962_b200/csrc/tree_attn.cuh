// Types shared by the two tree-attention kernels (legacy mma.sync and tcgen05).
#pragma once

#include "common.cuh"

namespace specroll {

struct AttnArgs {
    const __nv_bfloat16 *Q, *Kc, *Vc, *Kt, *Vt;
    const int32_t *kv_indptr;
    const int32_t *item_start;  // [B+1] exclusive prefix of the per-sequence chunk counts
    __nv_bfloat16 *O;
    float *lse;
    float *part_o;   // [items, Hkv, rows_pad, D]   un-normalised partial outputs of split sequences
    float *part_ml;  // [items, Hkv, rows_pad, 2]   (reference max in log2 units, sum)
    int32_t B, N, Hq, Hkv, G, rows, rows_pad, n_rb, rows_per_block, chunk_tiles;
    int32_t tile_tokens;  // KV tokens per tile: 64 (mma.sync kernel) or 128 (tcgen05 kernel)
    float scale_log2;     // scale * log2(e)
};

// tcgen05 kernel (tree_attn_tc.cu).  T_kv = total cached tokens.  Launches the main kernel only.
int launch_attn_tc(const AttnArgs &a, const TopoMask &mask, int D, int items, long long T_kv, int32_t *status,
                   cudaStream_t st);

}  // namespace specroll
