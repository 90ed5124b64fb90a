// Host helpers: TMA tensor-map encoding through the driver entry point (no link against libcuda).
#pragma once
#include <cudaTypedefs.h>

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

// Tensor of `rank` dims (dims[0] innermost, contiguous), box of `box` elements, 128-byte swizzle.
// strides_bytes[i] is the stride of dim i+1.
inline bool make_tmap(CUtensorMap* out, const void* base, int rank, const uint64_t* dims,
                      const uint64_t* strides_bytes, const uint32_t* box,
                      CUtensorMapDataType dt = CU_TENSOR_MAP_DATA_TYPE_BFLOAT16,
                      CUtensorMapSwizzle swz = CU_TENSOR_MAP_SWIZZLE_128B) {
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
    return r == CUDA_SUCCESS;
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
