// TMA tensor maps: encoded through the driver entry point (no link-time dependency on libcuda) and cached by key.
#include "tensormap.h"

#include <mutex>
#include <unordered_map>

namespace mpode {
namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    });
    return fn;
}

struct MapKey {
    const void* ptr; long long slots, rows, cols, slot_stride, ld; int box_rows, dt;
    bool operator==(const MapKey& o) const {
        return ptr == o.ptr && slots == o.slots && rows == o.rows && cols == o.cols && slot_stride == o.slot_stride &&
               ld == o.ld && box_rows == o.box_rows && dt == o.dt;
    }
};
struct MapKeyHash {
    size_t operator()(const MapKey& k) const {
        size_t h = (size_t)k.ptr;
        h = h * 1000003u ^ (size_t)k.slots;
        h = h * 1000003u ^ (size_t)k.rows;
        h = h * 1000003u ^ (size_t)k.cols;
        h = h * 1000003u ^ (size_t)k.slot_stride;
        h = h * 1000003u ^ (size_t)k.ld;
        h = h * 1000003u ^ (size_t)(k.box_rows * 4 + k.dt);
        return h;
    }
};

bool encode_cached(const MapKey& key, CUtensorMap* out) {
    static std::mutex mu;
    static std::unordered_map<MapKey, CUtensorMap, MapKeyHash> cache;
    std::lock_guard<std::mutex> lock(mu);
    auto it = cache.find(key);
    if (it != cache.end()) { *out = it->second; return true; }
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const bool three = key.slots > 0;
    cuuint64_t gdim[3] = {(cuuint64_t)key.cols, (cuuint64_t)key.rows, (cuuint64_t)(three ? key.slots : 1)};
    cuuint64_t gstr[2] = {(cuuint64_t)key.ld * 2, (cuuint64_t)key.slot_stride * 2};
    cuuint32_t box[3] = {(cuuint32_t)64, (cuuint32_t)key.box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUtensorMap m;
    CUresult r = fn(&m, key.dt == MPODE_BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16,
                    three ? 3 : 2, const_cast<void*>(key.ptr), gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return false;
    if (cache.size() > 4096) cache.clear();
    cache.emplace(key, m);
    *out = m;
    return true;
}

}  // namespace

bool get_tensor_map(const void* ptr, long long rows, long long cols, long long ld, int box_rows, mpode_dtype dt,
                    CUtensorMap* out) {
    return encode_cached(MapKey{ptr, 0, rows, cols, 0, ld, box_rows, (int)dt}, out);
}

bool get_tensor_map_3d(const void* ptr, long long slots, long long rows, long long cols, long long slot_stride,
                       long long ld, int box_rows, mpode_dtype dt, CUtensorMap* out) {
    if (slots < 1) return false;
    return encode_cached(MapKey{ptr, slots, rows, cols, slot_stride, ld, box_rows, (int)dt}, out);
}

bool get_tensor_map_nhwc(const void* ptr, int B, int H, int W, int C, int box_h, mpode_dtype dt, CUtensorMap* out) {
    static std::mutex mu;
    static std::unordered_map<MapKey, CUtensorMap, MapKeyHash> cache;
    MapKey key{ptr, -(long long)B, H, W, C, box_h, 0, (int)dt};     // negative slot count marks the 4-D kind
    std::lock_guard<std::mutex> lock(mu);
    auto it = cache.find(key);
    if (it != cache.end()) { *out = it->second; return true; }
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t gdim[4] = {(cuuint64_t)C, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)B};
    cuuint64_t gstr[3] = {(cuuint64_t)C * 2, (cuuint64_t)W * C * 2, (cuuint64_t)H * W * C * 2};
    cuuint32_t box[4] = {64u, (cuuint32_t)W, (cuuint32_t)box_h, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUtensorMap m;
    CUresult r = fn(&m, dt == MPODE_BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 4,
                    const_cast<void*>(ptr), gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return false;
    if (cache.size() > 4096) cache.clear();
    cache.emplace(key, m);
    *out = m;
    return true;
}

int current_device() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        cudaGetLastError();
        dev = 0;
    }
    return dev;
}

int sm_count() {
    static int n[kMaxDevices] = {0};
    const int dev = current_device();
    if (n[dev] == 0) {
        int v = 0;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) {
            cudaGetLastError();
            v = 148;        // no device (host-side size queries): the B200's count
        }
        n[dev] = v;
    }
    return n[dev];
}

}  // namespace mpode
