// Shared device/host definitions of libsla (internal; the public interface is include/sla.h).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "sla.h"

namespace sla {

// Bits of the device status word (first int of the handle's workspace).
enum : int { kStatusTimeout = 1, kStatusBadIndex = 2 };

constexpr int kMaxTopK = 64;
constexpr int kMaxGroup = 16;

// Everything a kernel needs to know about one call, passed by value.
struct Call {
    int B, Hq, Hkv, D, G;
    long long q_sb, q_sh, q_st;     // strides of q_s / q / out, in elements
    long long kv_sb, kv_sh, kv_st;  // strides of k / v, in elements
    long long Lq, q_pos0, Lkv;
    int top_k, span_len, back, fwd;
    int window, mode;               // local window w (0 = none); sla_mode_t
    float search_scale, softmax_scale;
    int *status;                    // device status word
};

// floor(sqrt(x)) for 0 <= x < 2^62, exact.
__host__ __device__ inline long long isqrt_ll(long long x) {
    if (x <= 0) return 0;
    long long r = (long long)sqrt((double)x);
    while (r * r > x) --r;
    while ((r + 1) * (r + 1) <= x) ++r;
    return r;
}

// Base span length l(i) (Algorithm 1: l(i) = ceil(sqrt(i)) unless a fixed length is given).
__host__ __device__ inline long long base_len(long long i, int span_len) {
    if (span_len > 0) return span_len;
    if (i <= 0) return 0;
    long long r = isqrt_ll(i);
    return r * r < i ? r + 1 : r;
}

// ---- element loads: a 16-byte vector of T widened to fp32 ------------------------------------
template <typename T> struct Vec16;
template <> struct Vec16<float> {
    static constexpr int kElems = 4;
    __device__ static inline void load(const float *p, float (&f)[4]) {
        float4 v = __ldg(reinterpret_cast<const float4 *>(p));
        f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w;
    }
};
template <> struct Vec16<__nv_bfloat16> {
    static constexpr int kElems = 8;
    __device__ static inline void unpack(const uint4 &v, float (&f)[8]) {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            f[2 * j] = __uint_as_float(w[j] << 16);
            f[2 * j + 1] = __uint_as_float(w[j] & 0xffff0000u);
        }
    }
    __device__ static inline void load(const __nv_bfloat16 *p, float (&f)[8]) {
        uint4 v = __ldg(reinterpret_cast<const uint4 *>(p));
        unpack(v, f);
    }
};

template <typename T> __device__ inline T from_float(float x);
template <> __device__ inline float from_float<float>(float x) { return x; }
template <> __device__ inline __nv_bfloat16 from_float<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

}  // namespace sla
