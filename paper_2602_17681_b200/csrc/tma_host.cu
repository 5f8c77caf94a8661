// Host-side construction of TMA tensor maps through the driver entry point (no link-time libcuda dependency).
#include <cudaTypedefs.h>

#include <cstring>
#include <mutex>

#include "tc_common.cuh"

namespace latmix {

static PFN_cuTensorMapEncodeTiled_v12000 encode_fn() {
    static PFN_cuTensorMapEncodeTiled_v12000 fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &p, 12000, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(p);
    });
    return fn;
}

// A tensor map is a pure function of the arguments it is built from (address, extents, pitch, box), never of what the
// memory holds, so the last few are kept per host thread: a layer called again with the same buffers -- every decode
// step -- finds all its maps here instead of asking the driver for them (about a microsecond each, five or six per call).
namespace {
struct MapKey {
    const void* base;
    uint64_t d0, d1, d2;
    uint32_t b0, b1;
    int32_t kind;          // 0..2: 2-D map of that element kind; 3: scale tiles
    int32_t pad;
};
struct MapEntry { MapKey key; CUtensorMap map; bool valid; };
constexpr int kMapCacheEntries = 64;
thread_local MapEntry t_map_cache[kMapCacheEntries];

inline MapEntry& map_slot(const MapKey& k) {
    uint64_t h = reinterpret_cast<uint64_t>(k.base) >> 4;
    h ^= k.d0 * 0x9E3779B97F4A7C15ull; h ^= k.d1 * 0xC2B2AE3D27D4EB4Full; h ^= k.d2 * 0x165667B19E3779F9ull;
    h ^= ((uint64_t)k.b0 << 32 | k.b1) * 0x27D4EB2F165667C5ull; h ^= (uint64_t)(uint32_t)k.kind << 7;
    h ^= h >> 29;
    return t_map_cache[h % kMapCacheEntries];
}
inline bool map_lookup(const MapKey& k, CUtensorMap* out) {
    const MapEntry& e = map_slot(k);
    if (!e.valid || std::memcmp(&e.key, &k, sizeof(MapKey)) != 0) return false;
    std::memcpy(out, &e.map, sizeof(CUtensorMap));
    return true;
}
inline void map_store(const MapKey& k, const CUtensorMap* m) {
    MapEntry& e = map_slot(k);
    e.key = k; std::memcpy(&e.map, m, sizeof(CUtensorMap)); e.valid = true;
}
}  // namespace

bool make_tensor_map_2d(CUtensorMap* map, const void* base, int elem_kind, uint64_t cols, uint64_t rows,
                        uint64_t pitch_bytes, uint32_t box_cols, uint32_t box_rows) {
    MapKey key;
    std::memset(&key, 0, sizeof(key));
    key.base = base; key.d0 = cols; key.d1 = rows; key.d2 = pitch_bytes; key.b0 = box_cols; key.b1 = box_rows; key.kind = elem_kind;
    if (map_lookup(key, map)) return true;
    PFN_cuTensorMapEncodeTiled_v12000 fn = encode_fn();
    if (fn == nullptr) return false;
    CUtensorMapDataType dt = elem_kind == 0 ? CU_TENSOR_MAP_DATA_TYPE_UINT8
                             : elem_kind == 1 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {pitch_bytes};
    cuuint32_t box[2] = {box_cols, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, dt, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r == CUDA_SUCCESS) map_store(key, map);
    return r == CUDA_SUCCESS;
}

bool make_tensor_map_scale_tiles(CUtensorMap* map, const void* base, uint64_t k_tiles, uint64_t row_tiles,
                                 uint32_t box_k_tiles, uint32_t box_row_tiles) {
    MapKey key;
    std::memset(&key, 0, sizeof(key));
    key.base = base; key.d0 = k_tiles; key.d1 = row_tiles; key.b0 = box_k_tiles; key.b1 = box_row_tiles; key.kind = 3;
    if (map_lookup(key, map)) return true;
    PFN_cuTensorMapEncodeTiled_v12000 fn = encode_fn();
    if (fn == nullptr) return false;
    cuuint64_t dims[3] = {128, k_tiles, row_tiles};
    cuuint64_t strides[2] = {512, k_tiles * 512};
    cuuint32_t box[3] = {128, box_k_tiles, box_row_tiles};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT32, 3, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r == CUDA_SUCCESS) map_store(key, map);
    return r == CUDA_SUCCESS;
}

// cudaFuncSetAttribute(MaxDynamicSharedMemorySize) once per kernel and device instead of on every launch.
cudaError_t set_max_dynamic_smem(const void* kernel, int smem_bytes) {
    struct Entry { const void* kernel; int dev; int bytes; };
    static Entry cache[128];
    static int n_cached = 0;
    static std::mutex mu;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    std::lock_guard<std::mutex> lock(mu);
    for (int i = 0; i < n_cached; ++i)
        if (cache[i].kernel == kernel && cache[i].dev == dev && cache[i].bytes == smem_bytes) return cudaSuccess;
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
    if (e == cudaSuccess && n_cached < 128) cache[n_cached++] = Entry{kernel, dev, smem_bytes};
    return e;
}

// Number of SMs of the current device, asked once per device ordinal.
int sm_count() {
    static int cache[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    int n = cache[dev];
    if (n == 0) {
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return 148;
        cache[dev] = n;
    }
    return n;
}

// Number of CTA pairs (clusters of two) of `kernel` that can be resident at once on the current device; GPCs with
// an odd SM count leave an SM unpaired.  Cached per device ordinal and kernel.
int resident_cta_pairs(const void* kernel, int threads, int smem_bytes) {
    struct Entry { const void* kernel; int dev; int pairs; };
    static Entry cache[64];
    static int n_cached = 0;
    static std::mutex mu;
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    std::lock_guard<std::mutex> lock(mu);
    for (int i = 0; i < n_cached; ++i)
        if (cache[i].kernel == kernel && cache[i].dev == dev) return cache[i].pairs;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(sms / 2 * 2));
    cfg.blockDim = dim3((unsigned)threads);
    cfg.dynamicSmemBytes = (size_t)smem_bytes;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, kernel, &cfg) != cudaSuccess || n <= 0) {
        cudaGetLastError();
        n = sms / 2;
    }
    if (n_cached < 64) cache[n_cached++] = Entry{kernel, dev, n};
    return n;
}

}  // namespace latmix
