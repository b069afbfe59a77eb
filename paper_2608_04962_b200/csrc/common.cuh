// Shared helpers of the sm_100a kernels: error plumbing, topology descriptor passed by value,
// small PTX wrappers (cp.async, ldmatrix, mma.sync) and warp utilities.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/specroll.h"

namespace specroll {

// Records the last CUDA error for specroll_strerror and returns SPECROLL_ECUDA.
int note_cuda_error(cudaError_t e);

#define SR_CUDA_TRY(expr)                                           \
    do {                                                            \
        cudaError_t _e = (expr);                                    \
        if (_e != cudaSuccess) return specroll::note_cuda_error(_e); \
    } while (0)

#define SR_LAUNCH_CHECK() SR_CUDA_TRY(cudaGetLastError())

#ifdef __CUDACC__
// Launch as the programmatic dependent of the kernel before it in the stream (pdl = false: an ordinary launch).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(bool pdl, void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                    Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}
#endif

// Raises a kernel's dynamic shared-memory limit the first time the kernel is launched on the current device
// (the attribute is per device), and optionally returns that device's SM count.  Thread-safe; later calls for
// the same (kernel, device) cost one table look-up.  Returns SPECROLL_OK or SPECROLL_ECUDA.
int device_setup(const void *kernel, int dynamic_smem_bytes, int *n_sm);

// ---- index checks of debug builds (-DSPECROLL_CHECK)
// No memory checker can be run on this code where it is developed, so a debug build makes the kernels check the
// indices they read from caller-supplied device arrays (token ids, candidate slots, record rows).  A bad index is
// never followed: the kernel notes the first one (a code and where) in a word of its translation unit and goes on
// with index 0, so the launch completes and the context stays usable.  specroll_check_status reads the words.
typedef int (*CheckReader)(int *detail, int reset);
void register_check_reader(CheckReader fn);
#ifdef SPECROLL_CHECK
#define SR_CHECK_TU()                                                                                      \
    static __device__ int sr_check_word[2];                                                                \
    static int sr_check_read(int *detail, int reset) {                                                     \
        int w_[2] = {0, 0};                                                                                \
        if (cudaMemcpyFromSymbol(w_, sr_check_word, sizeof(w_)) != cudaSuccess) return SPECROLL_ECUDA;     \
        if (reset) {                                                                                       \
            const int z_[2] = {0, 0};                                                                      \
            if (cudaMemcpyToSymbol(sr_check_word, z_, sizeof(z_)) != cudaSuccess) return SPECROLL_ECUDA;   \
        }                                                                                                  \
        if (detail) *detail = w_[1];                                                                       \
        return w_[0];                                                                                      \
    }                                                                                                      \
    static const int sr_check_registered = (specroll::register_check_reader(sr_check_read), 0);             \
    /* `index` if it lies in [0, n), else notes the failure and gives 0 */                                  \
    static __device__ __forceinline__ int sr_checked(int index, int n, int where) {                         \
        if (index >= 0 && index < n) return index;                                                          \
        if (atomicCAS(&sr_check_word[0], 0, SPECROLL_EINDEX) == 0) sr_check_word[1] = where;                \
        return 0;                                                                                           \
    }
#define SR_CHECK_FAIL(where)                                                        \
    do {                                                                            \
        if (atomicCAS(&sr_check_word[0], 0, SPECROLL_EINDEX) == 0) sr_check_word[1] = (where); \
    } while (0)
#define SR_CHECKED(index, n, where) sr_checked((index), (n), (where))
#else
#define SR_CHECK_TU()
#define SR_CHECKED(index, n, where) (index)
#endif

static inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Tree topology, validated on the host and handed to kernels by value (200 bytes).
struct Topo {
    int32_t N;
    int32_t max_depth;
    int8_t parent[SPECROLL_MAX_NODES];
    int8_t depth[SPECROLL_MAX_NODES];
    int8_t n_child[SPECROLL_MAX_NODES];
};

struct TopoMask {
    uint64_t anc[SPECROLL_MAX_NODES];  // bit j of anc[n]: node j is an ancestor of n, or n itself
};

// Returns SPECROLL_OK or SPECROLL_EINVAL.  K < 0 / k < 0 skip the depth / fan-out checks.
int build_topo(const int32_t *parent_host, int N, int K, int k, Topo *t, TopoMask *m);

// ------------------------------------------------------------------------------ device side
#ifdef __CUDACC__

__device__ __forceinline__ float bf16_bits_to_float(uint32_t bits16) {
    return __uint_as_float(bits16 << 16);
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// 16-byte streaming load that does not pollute L1.
__device__ __forceinline__ uint4 ld_nc_v4(const void *p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

__device__ __forceinline__ uint32_t smem_u32(const void *p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// Programmatic dependent launch: a kernel lets the next one in the stream start its prologue (pdl_launch_dependents)
// and waits for the one before it to complete, with its memory visible (pdl_wait; returns at once in a kernel that
// was launched the ordinary way).  Everything a kernel reads from, or writes to, global memory comes after its wait.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Thread-block clusters: this CTA's rank, a barrier over all threads of the cluster (release / acquire), and a
// load from the same shared-memory offset in another CTA of the cluster.
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ double ld_dsmem_f64(const void *own_smem_ptr, uint32_t cta_rank) {
    uint32_t remote;
    double v;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(smem_u32(own_smem_ptr)), "r"(cta_rank));
    asm volatile("ld.shared::cluster.f64 %0, [%1];" : "=d"(v) : "r"(remote) : "memory");
    return v;
}

__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, bool pred) {
    int sz = pred ? 16 : 0;  // src-size 0: destination is zero-filled
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N));
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}

// D(16x8, fp32) += A(16x16, bf16, row) * B(16x8, bf16, col)
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0,
                                               uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}

#endif  // __CUDACC__

}  // namespace specroll
