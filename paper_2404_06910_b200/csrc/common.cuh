// Shared host/device helpers of the library: error reporting, argument checks,
// storage-type loads.  Nothing here is used by (or shared with) the CPU oracle.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>

#include "../../include/sp.h"

namespace sp {

// ---- thread-local error message ---------------------------------------------------
char *error_buffer();                       // 512 bytes, thread local (api.cu)
int fail(int code, const char *fmt, ...);   // formats the message, returns code

#define SP_REQUIRE(cond, code, ...)                     \
    do {                                                \
        if (!(cond)) return ::sp::fail((code), __VA_ARGS__); \
    } while (0)

#define SP_CUDA(call)                                                                   \
    do {                                                                                \
        cudaError_t e__ = (call);                                                       \
        if (e__ != cudaSuccess)                                                         \
            return ::sp::fail(SP_ERR_CUDA, "%s failed: %s", #call, cudaGetErrorString(e__)); \
    } while (0)

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool aligned256(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 255u) == 0; }
inline int elt_bytes(int dtype) { return dtype == SP_F32 ? 4 : 2; }
__host__ __device__ constexpr size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

int check_layout(const sp_layout *lay);     // host-visible fields only (api.cu)

// Device status word codes (first 4 bytes of a workspace).
enum : uint32_t { STATUS_OK = 0, STATUS_TIMEOUT = 1, STATUS_BAD_LAYOUT = 2 };

#ifdef __CUDACC__
// One rotation (a, b) -> (a cos - b sin, a sin + b cos) with its roundings spelled out, so that every kernel that
// rotates the same pair with the same (cos, sin) stores the same bits.
__device__ __forceinline__ void rope_rotate(float a, float b, float c, float s, float &na, float &nb)
{
    na = __fmaf_rn(a, c, -__fmul_rn(b, s));
    nb = __fmaf_rn(a, s, __fmul_rn(b, c));
}
#endif
int num_sms();
// (cos, sin) of every (token, pair m < rot_dim / 2) at pos * base^(-2m / rot_dim), [n_tokens][rot_dim / 2] (rope.cu).
int launch_rope_table(const float *pos, int64_t n_tokens, int rot_dim, double base, float2 *out, cudaStream_t st);                              // multiprocessors of the current device (api.cu)

// ---- device helpers ----------------------------------------------------------------
#ifdef __CUDACC__
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// Loads 8 consecutive elements (bf16: one 16-byte load) or 4 (fp32) as floats.
template <typename T> struct Vec;
template <> struct Vec<__nv_bfloat16> {
    static constexpr int N = 8;
    __device__ __forceinline__ static void load(const __nv_bfloat16 *p, float (&f)[8]) {
        const uint4 w = *reinterpret_cast<const uint4 *>(p);
        f[0] = bf16_lo(w.x); f[1] = bf16_hi(w.x); f[2] = bf16_lo(w.y); f[3] = bf16_hi(w.y);
        f[4] = bf16_lo(w.z); f[5] = bf16_hi(w.z); f[6] = bf16_lo(w.w); f[7] = bf16_hi(w.w);
    }
};
template <> struct Vec<float> {
    static constexpr int N = 4;
    __device__ __forceinline__ static void load(const float *p, float (&f)[4]) {
        const float4 w = *reinterpret_cast<const float4 *>(p);
        f[0] = w.x; f[1] = w.y; f[2] = w.z; f[3] = w.w;
    }
};

__device__ __forceinline__ float to_float(float x) { return x; }
__device__ __forceinline__ float to_float(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ __forceinline__ void store_val(float *p, float x) { *p = x; }
__device__ __forceinline__ void store_val(__nv_bfloat16 *p, float x) { *p = __float2bfloat16_rn(x); }

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&t);
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
#endif  // __CUDACC__

}  // namespace sp
