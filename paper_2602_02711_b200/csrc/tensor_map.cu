// Host-side tensor-map encoding for the TMA loads.
#include <cudaTypedefs.h>

#include <cstring>
#include <mutex>
#include <unordered_map>

#include <cstdlib>

#include "sm100.cuh"

namespace dmr {

namespace {
PFN_cuTensorMapEncodeTiled_v12000 g_encode = nullptr;
std::once_flag g_once;

void fetch_encode() {
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &fn, 12000, cudaEnableDefault, &qres);
    if (e == cudaSuccess && qres == cudaDriverEntryPointSuccess) g_encode = (PFN_cuTensorMapEncodeTiled_v12000)fn;
    else g_last_cuda_error = (int)(e != cudaSuccess ? e : cudaErrorUnknown);
}
}  // namespace

namespace {
// Encoded maps are kept by (address, geometry): a map is a pure function of these, so an entry never goes
// stale - a buffer that is freed and allocated again at the same address with the same shape gets the same
// map.  Decode-time calls are a few microseconds long, and encoding two maps per call was a visible share of them.
struct MapKey {
    uint64_t v[8];
    bool operator==(const MapKey &o) const { return memcmp(v, o.v, sizeof v) == 0; }
};
struct MapKeyHash {
    size_t operator()(const MapKey &k) const {
        uint64_t h = 1469598103934665603ull;
        for (uint64_t x : k.v) h = (h ^ x) * 1099511628211ull;
        return (size_t)h;
    }
};
std::mutex g_cache_mutex;
std::unordered_map<MapKey, CUtensorMap, MapKeyHash> g_cache;
constexpr size_t kMaxCachedMaps = 8192;
}  // namespace

bool make_tensor_map_2d(CUtensorMap *map, CUtensorMapDataType dtype, size_t elem_bytes, const void *base,
                        uint64_t rows, uint64_t cols, uint64_t row_stride_bytes, uint32_t box_rows,
                        uint32_t box_cols, TmaSwizzle swizzle) {
    std::call_once(g_once, fetch_encode);
    if (!g_encode) return false;
    const MapKey key = {{(uint64_t)(uintptr_t)base, (uint64_t)dtype, rows, cols, row_stride_bytes, box_rows, box_cols, (uint64_t)swizzle}};
    {
        std::lock_guard<std::mutex> lock(g_cache_mutex);
        auto it = g_cache.find(key);
        if (it != g_cache.end()) {
            *map = it->second;
            return true;
        }
    }
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {row_stride_bytes};
    cuuint32_t box[2] = {box_cols, box_rows};
    cuuint32_t estr[2] = {1, 1};
    (void)elem_bytes;
    CUresult r = g_encode(map, dtype, 2, const_cast<void *>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                          swizzle == TmaSwizzle::k128B ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        g_last_cuda_error = 10000 + (int)r;
        return false;
    }
    std::lock_guard<std::mutex> lock(g_cache_mutex);
    if (g_cache.size() >= kMaxCachedMaps) g_cache.clear();
    g_cache.emplace(key, *map);
    return true;
}


// cudaFuncSetAttribute(MaxDynamicSharedMemorySize) once per (kernel, device) instead of on every call.
bool ensure_dynamic_smem(const void *kernel, size_t bytes) {
    static std::mutex m;
    static std::unordered_map<uint64_t, size_t> done;  // (kernel address, device) -> bytes granted
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) dev = 0;
    const uint64_t key = ((uint64_t)(uintptr_t)kernel << 6) ^ (uint64_t)(dev & 63);
    std::lock_guard<std::mutex> lock(m);
    auto it = done.find(key);
    if (it != done.end() && it->second >= bytes) return true;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (e != cudaSuccess) {
        g_last_cuda_error = (int)e;
        (void)cudaGetLastError();
        return false;
    }
    done[key] = bytes;
    return true;
}

bool tc_pdl_enabled() {
    static int v = -1;
    if (v < 0) {
        const char *e = getenv("DMR_PDL");
        v = (e && e[0] == '0') ? 0 : 1;
    }
    return v != 0;
}

}  // namespace dmr
