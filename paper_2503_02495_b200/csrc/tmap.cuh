// Host helpers: TMA tensor-map encoding through the driver entry point (no link against libcuda).
#pragma once
#include <cudaTypedefs.h>

#include <cstring>
#include <mutex>
#include <unordered_map>

#include "common.cuh"

namespace uoe {

inline PFN_cuTensorMapEncodeTiled_v12000 tensor_map_encoder() {
    static PFN_cuTensorMapEncodeTiled_v12000 fn = []() -> PFN_cuTensorMapEncodeTiled_v12000 {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess) return nullptr;
        if (q != cudaDriverEntryPointSuccess) return nullptr;
        return (PFN_cuTensorMapEncodeTiled_v12000)p;
    }();
    return fn;
}

// Encoded tensor maps are kept in a process-wide table keyed by everything that goes into the encoding (base
// address, extents, strides, box, type, swizzle), so a caller that reuses its buffers -- a training or serving loop
// on preallocated tensors -- encodes each map once and pays a table look-up per call afterwards.  The encoding is a
// pure function of the key, so a stale entry cannot exist; the table is emptied when it reaches kTmapCacheMax
// entries.  Thread-safe (one mutex).
struct TmapKey {
    uint64_t w[14];
    bool operator==(const TmapKey& o) const { return std::memcmp(w, o.w, sizeof(w)) == 0; }
};
struct TmapKeyHash {
    size_t operator()(const TmapKey& k) const {
        uint64_t h = 0x9E3779B97F4A7C15ull;
        for (uint64_t v : k.w) { h ^= v + 0x9E3779B97F4A7C15ull + (h << 6) + (h >> 2); }
        return (size_t)h;
    }
};
constexpr size_t kTmapCacheMax = 4096;
inline long long& tmap_encode_count() { static long long n = 0; return n; }     // encodings done (cache misses), for tests

// Tensor of `rank` dims (dims[0] innermost, contiguous), box of `box` elements, 128-byte swizzle.
// strides_bytes[i] is the stride of dim i+1.
inline bool make_tmap(CUtensorMap* out, const void* base, int rank, const uint64_t* dims,
                      const uint64_t* strides_bytes, const uint32_t* box,
                      CUtensorMapDataType dt = CU_TENSOR_MAP_DATA_TYPE_BFLOAT16,
                      CUtensorMapSwizzle swz = CU_TENSOR_MAP_SWIZZLE_128B) {
    static std::mutex mu;
    static std::unordered_map<TmapKey, CUtensorMap, TmapKeyHash> table;
    if (rank < 1 || rank > 4) return false;
    TmapKey key = {};
    key.w[0] = (uint64_t)(uintptr_t)base;
    key.w[1] = (uint64_t)rank | ((uint64_t)dt << 8) | ((uint64_t)swz << 24);
    for (int i = 0; i < rank; ++i) { key.w[2 + i] = dims[i]; key.w[6 + i] = box[i]; }
    for (int i = 0; i + 1 < rank; ++i) key.w[10 + i] = strides_bytes[i];
    {
        std::lock_guard<std::mutex> lock(mu);
        auto it = table.find(key);
        if (it != table.end()) { *out = it->second; return true; }
    }
    auto enc = tensor_map_encoder();
    if (!enc) return false;
    cuuint32_t elem_strides[5] = {1, 1, 1, 1, 1};
    cuuint64_t gdims[5], gstr[5];
    cuuint32_t gbox[5];
    for (int i = 0; i < rank; ++i) { gdims[i] = dims[i]; gbox[i] = box[i]; }
    for (int i = 0; i + 1 < rank; ++i) gstr[i] = strides_bytes[i];
    CUresult r = enc(out, dt, (cuuint32_t)rank, const_cast<void*>(base), gdims, gstr, gbox, elem_strides,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return false;
    std::lock_guard<std::mutex> lock(mu);
    ++tmap_encode_count();
    if (table.size() >= kTmapCacheMax) table.clear();
    table.emplace(key, *out);
    return true;
}

// SM count of the current device (cached per device).
inline int sm_count() {
    static DeviceValue cache;
    const int dev = current_device();
    if (cache.has(dev)) return cache.get(dev);
    int v = 148;
    if (dev >= 0) cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev);
    if (v <= 0) v = 148;
    if (dev >= 0) cache.set(dev, v);
    return v;
}

}  // namespace uoe
