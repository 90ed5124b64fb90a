// Shared host/device helpers of the UoE library: derived sizes, workspace carving, status word,
// element conversions and activations.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "device_once.h"
#include "uoe.h"

namespace uoe {

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------

extern long long g_launch_count;   // kernels enqueued by this process (reported by uoe_launch_count)

#define UOE_CUDA_OK(expr)                                   \
    do {                                                    \
        cudaError_t _e = (expr);                            \
        if (_e != cudaSuccess) return UOE_ERR_CUDA;         \
    } while (0)

#define UOE_LAUNCHED()                                      \
    do {                                                    \
        ++uoe::g_launch_count;                              \
        if (cudaGetLastError() != cudaSuccess) return UOE_ERR_CUDA; \
    } while (0)

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Ordinal of the current device, or -1 (no device, or an ordinal beyond the per-device tables).
inline int current_device() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return -1;
    return dev;
}

// Opt-in of `kern` to `bytes` of dynamic shared memory, done once on every device the kernel is launched on
// (the attribute belongs to the device's copy of the function).
template <typename K>
inline uoe_status smem_opt_in(DeviceOnce& once, K kern, int bytes) {
    const int dev = current_device();
    if (dev < 0) return UOE_ERR_CUDA;
    if (once.needs(dev)) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return UOE_ERR_CUDA;
        once.mark(dev);
    }
    return UOE_OK;
}

// Every kernel is launched with programmatic stream serialization allowed: the next kernel in the stream may
// be scheduled, and run up to its pdl_wait(), while this one is still executing, which hides launch and
// prologue latency between the short kernels of a call.  Kernels call pdl_trigger() first (dependents may
// be launched once all CTAs of this grid have started) and pdl_wait() before touching global memory.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_k(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

// The same for a kernel of CTA pairs: clusters of two CTAs along x (the grid's x extent is even).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_k_pairs(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    at[1].id = cudaLaunchAttributeClusterDimension;
    at[1].val.clusterDim.x = 2;
    at[1].val.clusterDim.y = 1;
    at[1].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

// How many CTA pairs of a kernel can be resident on the device at once.
template <typename K>
inline cudaError_t max_resident_pairs(K kern, int threads, size_t smem, int* pairs) {
    int sms = 0, dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (err != cudaSuccess) return err;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(sms & ~1);
    cfg.blockDim = dim3(threads);
    cfg.dynamicSmemBytes = smem;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = 2;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    return cudaOccupancyMaxActiveClusters(pairs, kern, &cfg);
}

// While profiling is enabled (uoe_profile_enable), a ProfScope around a launch records a CUDA event
// before and after it on the launching stream; otherwise it does nothing.
struct ProfScope {
    ProfScope(const char* name, cudaStream_t s);
    ~ProfScope();
    int slot;
    cudaStream_t stream;
};

// Sizes derived from a problem (paper notation: l_p tokens per patch, l_a = c*l_p tokens per expert).
struct Dims {
    int B, L, Lv, d, n, k, m, c, l_p, l_a, d_e, H, d_h, d_g, d_rope;
    int esize;            // bytes per element of x / weights / y
    long long R;          // routed rows without padding = B*k*l_a
    long long Rmax;       // bound on expert_offsets[n]
    bool bf16;
};

// Validates the fields every op relies on; returns UOE_OK and fills `D`.
inline uoe_status make_dims(const uoe_problem* p, Dims& D) {
    if (!p) return UOE_ERR_INVALID_ARG;
    if (p->B < 1 || p->L < 1 || p->d < 1 || p->n < 1 || p->k < 1 || p->m < 1 || p->c < 1) return UOE_ERR_INVALID_ARG;
    if (p->k > p->n || p->c > p->m || p->L % p->m != 0) return UOE_ERR_INVALID_ARG;
    if (p->L_valid < 1 || p->L_valid > p->L) return UOE_ERR_INVALID_ARG;
    if (p->dtype != UOE_F32 && p->dtype != UOE_BF16) return UOE_ERR_INVALID_ARG;
    if (p->act < 0 || p->act > UOE_ACT_IDENTITY) return UOE_ERR_INVALID_ARG;
    if (p->d_e < 0 || p->H < 0 || p->d_h < 0) return UOE_ERR_INVALID_ARG;
    if (p->H > 0 && (p->H % p->n != 0 || p->d_h < 1)) return UOE_ERR_INVALID_ARG;
    if (p->d_rope < 0 || p->d_rope % 2 != 0 || (p->d_rope > 0 && p->d_rope > p->d_h)) return UOE_ERR_INVALID_ARG;
    D.B = p->B; D.L = p->L; D.Lv = p->L_valid; D.d = p->d; D.n = p->n; D.k = p->k; D.m = p->m; D.c = p->c;
    D.l_p = p->L / p->m; D.l_a = p->c * D.l_p; D.d_e = p->d_e; D.H = p->H; D.d_h = p->d_h;
    D.d_g = p->H > 0 ? (p->H / p->n) * p->d_h : 0;
    D.d_rope = p->d_rope;
    D.bf16 = p->dtype == UOE_BF16;
    D.esize = D.bf16 ? 2 : 4;
    D.R = (long long)p->B * p->k * D.l_a;
    D.Rmax = (D.R + (long long)p->n * (UOE_ROW_ALIGN - 1)) / UOE_ROW_ALIGN * UOE_ROW_ALIGN;
    if (D.R > (1ll << 30)) return UOE_ERR_UNSUPPORTED;
    if ((p->d * D.esize) % 16 != 0) return UOE_ERR_UNSUPPORTED;      // rows move in 16-byte pieces
    if (p->n > 32 || p->k > 32 || p->m > 1024) return UOE_ERR_UNSUPPORTED;   // selection runs in one warp
    return UOE_OK;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

// Workspace carving: every block starts on a 1024-byte boundary; block 0 is the status block
// (word 0: device status; the rest: small per-call counters).
struct WsCarver {
    size_t off = 0;
    size_t take(size_t bytes) { size_t o = off; off = align_up(off + bytes, 1024); return o; }
};
constexpr size_t kStatusBytes = 1024;
constexpr size_t kControlBytes = 1024 * 1024;    // what uoe_workspace_init zeroes: the status block and the counters after it

// ------------------------------------------------------------------------------------------------
// device side: programmatic dependent launch
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
// returns when every kernel this one depends on has completed and its writes are visible
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// ------------------------------------------------------------------------------------------------
// device side: elements
// ------------------------------------------------------------------------------------------------

__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }

template <typename T> struct Vec16;                       // elements per 16 bytes
template <> struct Vec16<float> { static constexpr int N = 4; };
template <> struct Vec16<__nv_bfloat16> { static constexpr int N = 8; };

template <typename T>
__device__ __forceinline__ void unpack16(const uint4& v, float* f) {
    if constexpr (sizeof(T) == 4) {
        f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y); f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
    } else {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            f[2 * i] = __uint_as_float(w[i] << 16);
            f[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
        }
    }
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&t);
}

template <typename T>
__device__ __forceinline__ uint4 pack16(const float* f) {
    uint4 v;
    if constexpr (sizeof(T) == 4) {
        v.x = __float_as_uint(f[0]); v.y = __float_as_uint(f[1]); v.z = __float_as_uint(f[2]); v.w = __float_as_uint(f[3]);
    } else {
        v.x = pack_bf16x2(f[0], f[1]); v.y = pack_bf16x2(f[2], f[3]);
        v.z = pack_bf16x2(f[4], f[5]); v.w = pack_bf16x2(f[6], f[7]);
    }
    return v;
}

__device__ __forceinline__ uint4 ld_stream16(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ void st_stream16(void* p, const uint4& v) {
    asm volatile("st.global.L1::no_allocate.v4.u32 [%0], {%1,%2,%3,%4};"
                 :: "l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// ------------------------------------------------------------------------------------------------
// activations phi (Eq. 1) and their derivatives, float32
// ------------------------------------------------------------------------------------------------

__device__ __forceinline__ float act_apply(float h, int act) {
    switch (act) {
        case UOE_ACT_GELU_ERF: return 0.5f * h * (1.0f + erff(h * 0.70710678118654752f));
        case UOE_ACT_GELU_TANH: {
            float u = 0.79788456080286536f * (h + 0.044715f * h * h * h);
            return 0.5f * h * (1.0f + tanhf(u));
        }
        case UOE_ACT_SILU: return h / (1.0f + expf(-h));
        default: return h;
    }
}

// 2^x on the special-function unit (relative error about 2^-22; the results here are rounded to bfloat16)
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ float tanh_fast(float x) {
    float y;
    asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// phi applied in place to N values with the selection made once (keeps unrolled epilogues small).  Used where the
// result is rounded to bfloat16: SiLU and the tanh GELU go through one hardware tanh per value
// (x sigmoid(x) = x/2 (1 + tanh(x/2)); relative error about 2^-11, below the bfloat16 rounding of the result).
template <int N>
__device__ __forceinline__ void act_apply_n(float* f, int act) {
    switch (act) {
        case UOE_ACT_GELU_ERF:
#pragma unroll
            for (int q = 0; q < N; ++q) f[q] = 0.5f * f[q] * (1.0f + erff(f[q] * 0.70710678118654752f));
            break;
        case UOE_ACT_GELU_TANH:
#pragma unroll
            for (int q = 0; q < N; ++q) {
                const float u = 0.79788456080286536f * (f[q] + 0.044715f * f[q] * f[q] * f[q]);
                f[q] = 0.5f * f[q] * (1.0f + tanh_fast(u));
            }
            break;
        case UOE_ACT_SILU:
#pragma unroll
            for (int q = 0; q < N; ++q) { const float hx = 0.5f * f[q]; f[q] = fmaf(hx, tanh_fast(hx), hx); }
            break;
        default: break;
    }
}

// phi(h) and phi'(h) for N values with the selection made once; sub-expressions are shared
// (SiLU: s = sigmoid(h), phi = h s, phi' = s (1 + h (1 - s))).
template <int N>
__device__ __forceinline__ void act_and_deriv_n(const float* h, float* a, float* d, int act) {
    switch (act) {
        case UOE_ACT_SILU:
#pragma unroll
            for (int q = 0; q < N; ++q) {
                const float s = __fdividef(1.0f, 1.0f + __expf(-h[q]));
                a[q] = h[q] * s;
                d[q] = s * (1.0f + h[q] * (1.0f - s));
            }
            break;
        case UOE_ACT_GELU_ERF:
#pragma unroll
            for (int q = 0; q < N; ++q) {
                const float cdf = 0.5f * (1.0f + erff(h[q] * 0.70710678118654752f));
                a[q] = h[q] * cdf;
                d[q] = cdf + h[q] * 0.39894228040143268f * __expf(-0.5f * h[q] * h[q]);
            }
            break;
        case UOE_ACT_GELU_TANH:
#pragma unroll
            for (int q = 0; q < N; ++q) {
                const float u = 0.79788456080286536f * (h[q] + 0.044715f * h[q] * h[q] * h[q]);
                const float t = tanhf(u);
                const float du = 0.79788456080286536f * (1.0f + 3.0f * 0.044715f * h[q] * h[q]);
                a[q] = 0.5f * h[q] * (1.0f + t);
                d[q] = 0.5f * (1.0f + t) + 0.5f * h[q] * (1.0f - t * t) * du;
            }
            break;
        default:
#pragma unroll
            for (int q = 0; q < N; ++q) { a[q] = h[q]; d[q] = 1.0f; }
            break;
    }
}

__device__ __forceinline__ float act_deriv(float h, int act) {
    switch (act) {
        case UOE_ACT_GELU_ERF: {
            float cdf = 0.5f * (1.0f + erff(h * 0.70710678118654752f));
            float pdf = 0.39894228040143268f * expf(-0.5f * h * h);
            return cdf + h * pdf;
        }
        case UOE_ACT_GELU_TANH: {
            float u = 0.79788456080286536f * (h + 0.044715f * h * h * h);
            float t = tanhf(u);
            float du = 0.79788456080286536f * (1.0f + 3.0f * 0.044715f * h * h);
            return 0.5f * (1.0f + t) + 0.5f * h * (1.0f - t * t) * du;
        }
        case UOE_ACT_SILU: {
            float s = 1.0f / (1.0f + expf(-h));
            return s * (1.0f + h * (1.0f - s));
        }
        default: return 1.0f;
    }
}

// ------------------------------------------------------------------------------------------------
// device status word (first word of the workspace)
// ------------------------------------------------------------------------------------------------

__device__ __forceinline__ void set_status(int* status, int code) {
    if (status) atomicCAS(status, 0, code);
}

}  // namespace uoe
