// What happens to the cache between two speculative steps (the paper lists accepted-path KV extraction among the
// contents of generation time; it gives no formula): the tree rows of the committed path - the anchor (node 0)
// and the accepted nodes - are appended to the sequence's paged cache, and the hidden state of the node whose
// distribution produced the step's last token becomes the next step's input.
#include "common.cuh"

namespace specroll {

constexpr int COMMIT_MAX_LAYERS = 64;  // layers one launch can serve (their pointers travel as kernel arguments)

struct CommitLayers {
    const uint4 *Kt[COMMIT_MAX_LAYERS], *Vt[COMMIT_MAX_LAYERS];
    uint4 *Kp[COMMIT_MAX_LAYERS], *Vp[COMMIT_MAX_LAYERS];
};

// grid = (B, K + 1, layers): block (b, i, l) copies tree row path_node[b, i] of layer l's K and V to cache
// position kv_len[b] + i of that layer's pool.
__global__ void __launch_bounds__(128)
commit_path_kernel(const __grid_constant__ CommitLayers lay, const int32_t *__restrict__ path_node,
                   const int32_t *__restrict__ n_acc, long long n_pages,
                   const int32_t *__restrict__ page_table, const int32_t *__restrict__ page_indptr,
                   const int32_t *__restrict__ kv_len, int N, int K, int row_vec, int32_t *__restrict__ status) {
    const int b = blockIdx.x, i = blockIdx.y;
    const uint4 *__restrict__ Kt = lay.Kt[blockIdx.z], *__restrict__ Vt = lay.Vt[blockIdx.z];
    uint4 *__restrict__ Kp = lay.Kp[blockIdx.z], *__restrict__ Vp = lay.Vp[blockIdx.z];
    const int na = n_acc[b];
    if (i > na || na < 0 || na > K) return;
    const int node = path_node[(size_t)b * (K + 1) + i];
    const long long pos = (long long)kv_len[b] + i;
    const long long slot = pos / SPECROLL_PAGE_TOKENS;
    const int own = page_indptr[b + 1] - page_indptr[b];
    int page = -1;
    if (node >= 0 && node < N && kv_len[b] >= 0 && slot < own) page = page_table[page_indptr[b] + slot];
    if (page < 0 || page >= n_pages) {
        // no room (or a bad table): nothing is written for this token, and the caller is told
        if (threadIdx.x == 0 && status) atomicExch(status, SPECROLL_ELIMIT);
        return;
    }
    const size_t src = ((size_t)b * N + node) * row_vec;
    const size_t dst = ((size_t)page * SPECROLL_PAGE_TOKENS + (size_t)(pos % SPECROLL_PAGE_TOKENS)) * row_vec;
    for (int v = threadIdx.x; v < row_vec; v += blockDim.x) {
        Kp[dst + v] = Kt[src + v];
        Vp[dst + v] = Vt[src + v];
    }
}

__global__ void commit_len_kernel(const int32_t *__restrict__ kv_len, const int32_t *__restrict__ n_acc, int B, int K,
                                  int32_t *__restrict__ kv_len_out) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    const int na = n_acc[b];
    kv_len_out[b] = kv_len[b] + ((na < 0 || na > K) ? 0 : na + 1);
}

// h_next[b, :] = hidden[b, term_node[b], :]
__global__ void __launch_bounds__(128)
gather_hidden_kernel(const uint4 *__restrict__ hidden, const int32_t *__restrict__ term_node, int N, int row_vec,
                     uint4 *__restrict__ h_next) {
    const int b = blockIdx.x;
    int node = term_node[b];
    if (node < 0 || node >= N) node = 0;
    const size_t src = ((size_t)b * N + node) * row_vec, dst = (size_t)b * row_vec;
    for (int v = threadIdx.x; v < row_vec; v += blockDim.x) h_next[dst + v] = hidden[src + v];
}

}  // namespace specroll

using namespace specroll;

static int commit_layers(int32_t B, int32_t N, int32_t K, int32_t Hkv, int32_t D, int32_t n_layers,
                         const void *const *Kt, const void *const *Vt, const int32_t *path_node, const int32_t *n_acc,
                         void *const *Kp, void *const *Vp, int64_t n_pages, const int32_t *page_table,
                         const int32_t *page_indptr, const int32_t *kv_len, int32_t *kv_len_out, int32_t *status,
                         void *cuda_stream) {
    if (B < 0 || N < 1 || N > SPECROLL_MAX_NODES || K < 1 || K > SPECROLL_MAX_HEADS || Hkv < 1 || (D != 64 && D != 128) ||
        n_pages < 0 || n_pages > (1LL << 24) || n_layers < 1)
        return SPECROLL_EINVAL;
    if (B == 0) return SPECROLL_OK;  // (an empty batch has empty arrays: their pointers may be NULL)
    if (!Kt || !Vt || !path_node || !n_acc || !Kp || !Vp || !page_table || !page_indptr || !kv_len) return SPECROLL_EINVAL;
    for (int l = 0; l < n_layers; ++l) {
        if (!Kt[l] || !Vt[l] || !Kp[l] || !Vp[l]) return SPECROLL_EINVAL;
        if (!aligned16(Kt[l]) || !aligned16(Vt[l]) || !aligned16(Kp[l]) || !aligned16(Vp[l])) return SPECROLL_EALIGN;
    }
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const int row_vec = Hkv * D / 8;  // 16-byte vectors per token row
    for (int l0 = 0; l0 < n_layers; l0 += COMMIT_MAX_LAYERS) {
        const int nl = n_layers - l0 < COMMIT_MAX_LAYERS ? n_layers - l0 : COMMIT_MAX_LAYERS;
        CommitLayers lay;
        for (int l = 0; l < nl; ++l) {
            lay.Kt[l] = static_cast<const uint4 *>(Kt[l0 + l]);
            lay.Vt[l] = static_cast<const uint4 *>(Vt[l0 + l]);
            lay.Kp[l] = static_cast<uint4 *>(Kp[l0 + l]);
            lay.Vp[l] = static_cast<uint4 *>(Vp[l0 + l]);
        }
        commit_path_kernel<<<dim3((unsigned)B, (unsigned)(K + 1), (unsigned)nl), 128, 0, st>>>(
            lay, path_node, n_acc, (long long)n_pages, page_table, page_indptr, kv_len, N, K, row_vec, status);
        SR_LAUNCH_CHECK();
    }
    if (kv_len_out) {
        // after the copies in stream order, so that the lengths may be updated in place
        commit_len_kernel<<<(B + 255) / 256, 256, 0, st>>>(kv_len, n_acc, B, K, kv_len_out);
        SR_LAUNCH_CHECK();
    }
    return SPECROLL_OK;
}

extern "C" int specroll_commit_path(int32_t B, int32_t N, int32_t K, int32_t Hkv, int32_t D, const void *Kt,
                                    const void *Vt, const int32_t *path_node, const int32_t *n_acc, void *Kp,
                                    void *Vp, int64_t n_pages, const int32_t *page_table,
                                    const int32_t *page_indptr, const int32_t *kv_len, int32_t *kv_len_out,
                                    int32_t *status, void *cuda_stream) {
    return commit_layers(B, N, K, Hkv, D, 1, &Kt, &Vt, path_node, n_acc, &Kp, &Vp, n_pages, page_table, page_indptr,
                         kv_len, kv_len_out, status, cuda_stream);
}

extern "C" int specroll_commit_path_layers(int32_t B, int32_t N, int32_t K, int32_t Hkv, int32_t D, int32_t n_layers,
                                           const void *const *Kt, const void *const *Vt, const int32_t *path_node,
                                           const int32_t *n_acc, void *const *Kp, void *const *Vp, int64_t n_pages,
                                           const int32_t *page_table, const int32_t *page_indptr,
                                           const int32_t *kv_len, int32_t *kv_len_out, int32_t *status,
                                           void *cuda_stream) {
    return commit_layers(B, N, K, Hkv, D, n_layers, Kt, Vt, path_node, n_acc, Kp, Vp, n_pages, page_table,
                         page_indptr, kv_len, kv_len_out, status, cuda_stream);
}

extern "C" int specroll_gather_hidden(int32_t B, int32_t N, int32_t d, const void *hidden, const int32_t *term_node,
                                      void *h_next, void *cuda_stream) {
    if (B < 0 || N < 1 || N > SPECROLL_MAX_NODES || d < 8 || (d % 8)) return SPECROLL_EINVAL;
    if (B == 0) return SPECROLL_OK;  // (an empty batch has empty arrays: their pointers may be NULL)
    if (!hidden || !term_node || !h_next) return SPECROLL_EINVAL;
    if (!aligned16(hidden) || !aligned16(h_next)) return SPECROLL_EALIGN;
    gather_hidden_kernel<<<(unsigned)B, 128, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        static_cast<const uint4 *>(hidden), term_node, N, d / 8, static_cast<uint4 *>(h_next));
    SR_LAUNCH_CHECK();
    return SPECROLL_OK;
}
