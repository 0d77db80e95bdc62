// Tiled tensor maps (TMA descriptors) for bf16 arrays whose innermost dimension is head_dim, with a
// small per-thread cache: a map depends only on the base pointer, the extents, the strides and the box,
// and a caller that scores the same cache layer after layer, or decodes step after step, asks for the
// same few maps every call.
#include "obc_common.cuh"
#include <cudaTypedefs.h>
#include <string.h>

namespace obc {
namespace {

PFN_cuTensorMapEncodeTiled get_encode() {
    static PFN_cuTensorMapEncodeTiled fn = nullptr;
    if (!fn) {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = (PFN_cuTensorMapEncodeTiled)ptr;
    }
    return fn;
}

struct MapKey {
    const void* base;
    int rank;
    uint32_t box_rows;
    uint64_t dims[4];
    uint64_t strides[3];
};
struct MapEntry { MapKey key; CUtensorMap map; bool used; };
constexpr int kCacheSlots = 16;

}  // namespace

bool make_map(CUtensorMap* map, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes,
              uint32_t box_rows) {
    thread_local MapEntry cache[kCacheSlots] = {};
    thread_local int next_slot = 0;
    MapKey key;
    memset(&key, 0, sizeof(key));
    key.base = base; key.rank = rank; key.box_rows = box_rows;
    for (int i = 0; i < rank; ++i) key.dims[i] = dims[i];
    for (int i = 0; i < rank - 1; ++i) key.strides[i] = strides_bytes[i];
    for (int i = 0; i < kCacheSlots; ++i)
        if (cache[i].used && memcmp(&cache[i].key, &key, sizeof(key)) == 0) { *map = cache[i].map; return true; }

    PFN_cuTensorMapEncodeTiled enc = get_encode();
    if (!enc) return false;
    cuuint64_t gdim[4]; cuuint64_t gstr[3]; cuuint32_t box[4] = {64, box_rows, 1, 1}; cuuint32_t estr[4] = {1, 1, 1, 1};
    for (int i = 0; i < rank; ++i) gdim[i] = dims[i];
    for (int i = 0; i < rank - 1; ++i) gstr[i] = strides_bytes[i];
    if (enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), gdim, gstr, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return false;
    MapEntry& e = cache[next_slot];
    next_slot = (next_slot + 1) % kCacheSlots;
    e.key = key; e.map = *map; e.used = true;
    return true;
}

}  // namespace obc
