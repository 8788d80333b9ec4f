// Shared host/device helpers for the R3 kernels (argument checks, dtype helpers, launch checks).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "r3.h"

namespace r3 {

constexpr int kMaxExpertsPermute = 1024;
constexpr int kMaxExpertsCapture = 512;

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }
inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline size_t act_bytes(const r3_shape* s) { return s->act_dtype == R3_BF16 ? 2 : 4; }
inline size_t idx_bytes(const r3_shape* s) { return s->idx_type == R3_IDX_U8 ? 1 : 2; }

// Shape checks every entry point shares.  Returns R3_OK for T == 0 too (callers test T first).
inline r3_status check_shape(const r3_shape* s) {
    if (!s) return R3_ERR_INVALID_ARG;
    if (s->T < 0 || s->d <= 0 || s->E <= 0 || s->K <= 0 || s->F <= 0) return R3_ERR_INVALID_ARG;
    if (s->K > s->E) return R3_ERR_INVALID_ARG;
    if (s->act_dtype != R3_F32 && s->act_dtype != R3_BF16) return R3_ERR_INVALID_ARG;
    if (s->router_w_dtype != R3_F32 && s->router_w_dtype != R3_BF16) return R3_ERR_INVALID_ARG;
    if (s->idx_type != R3_IDX_U8 && s->idx_type != R3_IDX_I16) return R3_ERR_INVALID_ARG;
    if (s->idx_type == R3_IDX_U8 && s->E > 256) return R3_ERR_INVALID_ARG;
    if (s->E > 32767) return R3_ERR_INVALID_ARG;
    if ((s->d % 8) != 0 || (s->F % 8) != 0) return R3_ERR_INVALID_ARG;
    if ((long long)s->T * s->K > 0x7fffffffLL) return R3_ERR_INVALID_ARG;
    return R3_OK;
}

// Per-device "already done" flags for host-side set-up that CUDA keeps per device (function
// attributes, occupancy answers): a process that drives several devices repeats the set-up on
// each of them.  done() is false until mark() has been called with the same device current.
struct PerDevice {
    bool flag[64] = {};
    static int current() {
        int dev = 0;
        return (cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < 64) ? dev : 0;
    }
    bool done() const { return flag[current()]; }
    void mark() { flag[current()] = true; }
};

inline r3_status launch_status() {
    return cudaGetLastError() == cudaSuccess ? R3_OK : R3_ERR_CUDA;
}

__device__ __forceinline__ void report(int32_t* dev_status, int32_t code) {
    if (dev_status) atomicCAS(dev_status, 0, code);   // integer CAS: first error wins
}

// ---- element access by storage type -------------------------------------------------------
template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) {
    return __bfloat162float(v);
}
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) {
    return __float2bfloat16_rn(v);
}

// 16-byte vector of activations: 8 bf16 or 4 f32.
template <typename T> struct Vec16;
template <> struct Vec16<float> {
    static constexpr int N = 4;
    float4 v;
    __device__ __forceinline__ void unpack(float* f) const {
        f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w;
    }
    __device__ __forceinline__ void pack(const float* f) { v = make_float4(f[0], f[1], f[2], f[3]); }
};
template <> struct Vec16<__nv_bfloat16> {
    static constexpr int N = 8;
    uint4 v;
    __device__ __forceinline__ void unpack(float* f) const {
        const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float2 t = __bfloat1622float2(p[i]);
            f[2 * i] = t.x; f[2 * i + 1] = t.y;
        }
    }
    __device__ __forceinline__ void pack(const float* f) {
        __nv_bfloat162* p = reinterpret_cast<__nv_bfloat162*>(&v);
#pragma unroll
        for (int i = 0; i < 4; ++i) p[i] = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
    }
};

template <typename IdxT> __device__ __forceinline__ int idx_to_int(IdxT v);
template <> __device__ __forceinline__ int idx_to_int<uint8_t>(uint8_t v) { return v; }
template <> __device__ __forceinline__ int idx_to_int<int16_t>(int16_t v) { return v; }

}  // namespace r3

// Dispatch helpers: call `fn` with the C++ types that match the runtime dtype codes.
#define R3_DISPATCH_IDX(shape, IdxT, ...)                                         \
    do {                                                                          \
        if ((shape)->idx_type == R3_IDX_U8) { using IdxT = uint8_t; __VA_ARGS__; } \
        else { using IdxT = int16_t; __VA_ARGS__; }                               \
    } while (0)

#define R3_DISPATCH_ACT(shape, ActT, ...)                                              \
    do {                                                                               \
        if ((shape)->act_dtype == R3_BF16) { using ActT = __nv_bfloat16; __VA_ARGS__; } \
        else { using ActT = float; __VA_ARGS__; }                                      \
    } while (0)
