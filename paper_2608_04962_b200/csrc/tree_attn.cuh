// Types shared by the two tree-attention kernels (legacy mma.sync and tcgen05).
#pragma once

#include "common.cuh"

namespace specroll {

struct AttnArgs {
    const __nv_bfloat16 *Q, *Kc, *Vc, *Kt, *Vt;
    const int32_t *kv_indptr;
    const int32_t *item_start;  // [B+1] exclusive prefix of the per-sequence chunk counts (sequence order)
    __nv_bfloat16 *O;
    float *lse;
    float *part_o;   // [items, Hkv, rows_pad, D]   un-normalised partial outputs of split sequences
    float *part_ml;  // [items, Hkv, rows_pad, 2]   (reference max in log2 units, sum)
    int32_t B, N, Hq, Hkv, G, rows, rows_pad, n_rb, rows_per_block, chunk_tiles;
    int32_t tile_tokens;  // KV tokens per tile: 64 (mma.sync kernel) or 128 (tcgen05 kernel)
    float scale_log2;     // scale * log2(e)
    // ---- tcgen05 kernel only: work order and counters written by the prep kernel
    const int32_t *sorted_start;  // [B+1] exclusive prefix of the chunk counts in work order
    const int32_t *seq_at_rank;   // [B]   sequence at each position of the work order (longest chunks first)
    const int32_t *unit_tab;      // [items][8] per chunk in work order: b, chunk, n_chunks, first item, kv0, L, 0, 0
    int32_t *work_counter;        // next work unit to hand out
    int32_t *split_counters;      // [B, Hkv, n_rb] chunks of a (sequence, kv head, row block) that have finished
    int32_t total_work;           // items * Hkv * n_rb
    int32_t nodes_per_block;      // rows_per_block = nodes_per_block * G
    // paged cache (tcgen05 kernel only): pool page of every 128-token tile; a chunk table row then carries the
    // sequence's first slot in this table instead of its first token
    const int32_t *page_table;
    int early_cache;              // plan, cache and page table were complete before the preceding kernel was launched
    float *hand;                  // [ATTN_HAND_CTAS][4][128] per-CTA hand-over area between two groups of warps of the tcgen05 kernel
    int32_t merge_mode;           // chunks of a split sequence are merged 0: by the CTA that finishes last; 2: by a later kernel
    int32_t no_pdl;               // launch the attention kernel as an ordinary kernel, not as a programmatic dependent
};

constexpr int ATTN_HAND_CTAS = 256;  // CTAs the hand-over area is sized for (the grid is one CTA per SM)

// tcgen05 kernel (tree_attn_tc.cu).  T_kv = total cached tokens.  Launches the main kernel only.
int launch_attn_tc(const AttnArgs &a, const TopoMask &mask, int D, long long T_kv, int32_t *status, cudaStream_t st);
// Merges the chunks of split sequences after launch_attn_tc when a.merge_mode == 2.  items = chunks in the plan.
int launch_attn_merge_tc(const AttnArgs &a, int D, int items, cudaStream_t st);

}  // namespace specroll
