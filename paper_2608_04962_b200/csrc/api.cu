// Entry points that need no kernel: version, error strings, node budget; plus the host-side
// topology validation shared by the three steps.
#include <stdio.h>
#include <string.h>

#include <mutex>
#include <utility>
#include <vector>

#include "common.cuh"

namespace specroll {

static thread_local cudaError_t g_last_cuda = cudaSuccess;
static thread_local char g_msg[256];

int note_cuda_error(cudaError_t e) {
    g_last_cuda = e;
    return SPECROLL_ECUDA;
}

int device_setup(const void *kernel, int dynamic_smem_bytes, int *n_sm) {
    constexpr int MAX_DEV = 64;
    static std::mutex mu;
    static std::vector<std::pair<const void *, int>> done;  // (kernel, device) pairs whose limit has been raised
    static int sm_count[MAX_DEV];                           // 0 = not asked yet
    int dev = 0;
    SR_CUDA_TRY(cudaGetDevice(&dev));
    std::lock_guard<std::mutex> lock(mu);
    if (n_sm) {
        if (dev < 0 || dev >= MAX_DEV) {
            SR_CUDA_TRY(cudaDeviceGetAttribute(n_sm, cudaDevAttrMultiProcessorCount, dev));
        } else {
            if (sm_count[dev] == 0) SR_CUDA_TRY(cudaDeviceGetAttribute(&sm_count[dev], cudaDevAttrMultiProcessorCount, dev));
            *n_sm = sm_count[dev];
        }
    }
    if (!kernel) return SPECROLL_OK;
    for (const auto &e : done)
        if (e.first == kernel && e.second == dev) return SPECROLL_OK;
    SR_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, dynamic_smem_bytes));
    done.emplace_back(kernel, dev);
    return SPECROLL_OK;
}

// readers of the per-translation-unit check words (debug builds register them at load time)
static CheckReader *check_readers(int **n) {
    static CheckReader readers[16];
    static int count = 0;
    *n = &count;
    return readers;
}

void register_check_reader(CheckReader fn) {
    int *n = nullptr;
    CheckReader *r = check_readers(&n);
    if (*n < 16) r[(*n)++] = fn;
}

int lm_head_arm_dropped_signal();  // lm_head_tc.cu

int build_topo(const int32_t *parent_host, int N, int K, int k, Topo *t, TopoMask *m) {
    if (!parent_host || N < 1 || N > SPECROLL_MAX_NODES || parent_host[0] != -1) return SPECROLL_EINVAL;
    memset(t, 0, sizeof(*t));
    if (m) memset(m, 0, sizeof(*m));
    t->N = N;
    t->parent[0] = -1;
    if (m) m->anc[0] = 1ull;
    for (int n = 1; n < N; ++n) {
        int p = parent_host[n];
        if (p < 0 || p >= n) return SPECROLL_EINVAL;
        t->parent[n] = (int8_t)p;
        t->depth[n] = (int8_t)(t->depth[p] + 1);
        t->n_child[p]++;
        if (t->depth[n] > t->max_depth) t->max_depth = t->depth[n];
        if (K >= 0 && t->depth[n] > K) return SPECROLL_EINVAL;
        if (k >= 0 && t->n_child[p] > k) return SPECROLL_EINVAL;
        if (m) m->anc[n] = m->anc[p] | (1ull << n);
    }
    return SPECROLL_OK;
}

}  // namespace specroll

extern "C" {

int specroll_version(void) { return 100; }

const char *specroll_strerror(int code) {
    using namespace specroll;
    switch (code) {
        case SPECROLL_OK: return "ok";
        case SPECROLL_EINVAL: return "invalid argument (shape, limit, NULL pointer or malformed tree)";
        case SPECROLL_EALIGN: return "a tensor base pointer is not 16-byte aligned";
        case SPECROLL_EWORKSPACE: return "workspace too small or not 256-byte aligned";
        case SPECROLL_ETIMEOUT: return "a bounded device-side wait ran out";
        case SPECROLL_ELIMIT:
            return "problem exceeds the fixed size limit of this allocation-free entry point (use the "
                   "variant that takes a caller workspace)";
        case SPECROLL_EINDEX:
            return "an index read from a caller's device array is out of range (found by a build with index checks)";
        case SPECROLL_ECUDA:
            snprintf(g_msg, sizeof(g_msg), "CUDA error: %s", cudaGetErrorString(g_last_cuda));
            return g_msg;
        default: return "unknown error code";
    }
}

int specroll_check_status(int32_t *detail, int32_t reset) {
    using namespace specroll;
#ifndef SPECROLL_CHECK
    (void)reset;
    if (detail) *detail = 0;
    return -1;
#else
    int *n = nullptr;
    CheckReader *r = check_readers(&n);
    int first = SPECROLL_OK;
    for (int i = 0; i < *n; ++i) {
        int where = 0;
        const int rc = r[i](&where, reset);
        if (rc != SPECROLL_OK && first == SPECROLL_OK) {
            first = rc;
            if (detail) *detail = where;
        }
    }
    if (first == SPECROLL_OK && detail) *detail = 0;
    return first;
#endif
}

int specroll_check_inject(int32_t what) {
    if (what == 1) return specroll::lm_head_arm_dropped_signal();
    return SPECROLL_EINVAL;
}

int32_t specroll_node_budget(int32_t C_hw, int32_t B_active, int32_t N_min, int32_t N_max) {
    if (B_active < 1) return N_max;
    int32_t n = C_hw / B_active;
    if (n < N_min) n = N_min;
    if (n > N_max) n = N_max;
    return n;
}

}  // extern "C"
