// Host-side construction of TMA tensor maps (driver entry point looked up at run time, so the
// library does not link against the driver).
#include <string.h>

#include <mutex>

#include "tc05.cuh"

namespace specroll {

// A tensor map is a pure function of (base pointer, extents, strides, box): the last few are remembered, so that
// the calls of a step (the same caches, weights and activations layer after layer, step after step) do not encode
// theirs again (encoding costs a few microseconds of host time per map, five maps per attention call).
namespace {
struct MapKey {
    const void *base;
    uint64_t a, b, c;
    uint32_t box1, box2, rank;
};
struct MapEntry {
    MapKey key;
    CUtensorMap map;
    bool used;
};
constexpr int MAP_CACHE = 128;
std::mutex map_mu;
MapEntry map_cache[MAP_CACHE];
unsigned map_next = 0;

bool map_lookup(const MapKey &k, CUtensorMap *out) {
    std::lock_guard<std::mutex> lock(map_mu);
    for (int i = 0; i < MAP_CACHE; ++i)
        if (map_cache[i].used && memcmp(&map_cache[i].key, &k, sizeof(MapKey)) == 0) {
            *out = map_cache[i].map;
            return true;
        }
    return false;
}
void map_store(const MapKey &k, const CUtensorMap &m) {
    std::lock_guard<std::mutex> lock(map_mu);
    MapEntry &e = map_cache[map_next++ % MAP_CACHE];
    e.key = k;
    e.map = m;
    e.used = true;
}
}  // namespace

// ------------------------------------------------------------------------------ tensor maps

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// 3-D bf16 tensor [n2, n1, n0] (n0 innermost, contiguous), box [box2, box1, 64], 128-byte swizzle.
int make_tmap_3d_bf16(CUtensorMap *map, const void *base, uint64_t n0, uint64_t n1, uint64_t n2, uint32_t box1,
                      uint32_t box2) {
    MapKey key;
    memset(&key, 0, sizeof(key));
    key.base = base;
    key.a = n0;
    key.b = n1;
    key.c = n2;
    key.box1 = box1;
    key.box2 = box2;
    key.rank = 3;
    if (map_lookup(key, map)) return SPECROLL_OK;
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return note_cuda_error(cudaErrorNotSupported);
    cuuint64_t dims[3] = {n0, n1, n2};
    cuuint64_t strides[2] = {n0 * 2, n0 * n1 * 2};
    cuuint32_t box[3] = {64, box1, box2};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return note_cuda_error(cudaErrorInvalidValue);
    map_store(key, *map);
    return SPECROLL_OK;
}

int make_tmap_2d_bf16(CUtensorMap *map, const void *base, uint64_t rows, uint64_t cols, uint64_t ld_elems,
                      uint32_t box_rows) {
    MapKey key;
    memset(&key, 0, sizeof(key));
    key.base = base;
    key.a = rows;
    key.b = cols;
    key.c = ld_elems;
    key.box1 = box_rows;
    key.rank = 2;
    if (map_lookup(key, map)) return SPECROLL_OK;
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return note_cuda_error(cudaErrorNotSupported);
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {ld_elems * 2};
    cuuint32_t box[2] = {64, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return note_cuda_error(cudaErrorInvalidValue);
    map_store(key, *map);
    return SPECROLL_OK;
}

}  // namespace specroll
