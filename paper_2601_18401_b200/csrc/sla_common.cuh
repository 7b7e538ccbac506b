// Shared device/host definitions of libsla (internal; the public interface is include/sla.h).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "sla.h"

namespace sla {

// Bits of the device status word (first int of the handle's workspace).
enum : int { kStatusTimeout = 1, kStatusBadIndex = 2, kStatusOverrun = 4 };

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
    // Exponents other than 1/2 (Section "Span attention", general p; Section "Training"): the stride
    // offsets and the span-length steps come from tables the host builds (NULL: the exact integer
    // rules for p = 1/2).  off[s] = ceil((s+1)^(1/p_search)), ascending; len_first[v-1] = smallest i
    // with l(i) = ceil(i^p_span) >= v.  The *_host copies serve the host-side plans.
    const int *off, *off_host;
    int n_off;
    const int *len_first, *len_first_host;
    int n_len;
    // sequence-sharded decode: the key positions [shard_lo, shard_hi) this rank holds ([0, Lkv) otherwise)
    long long shard_lo, shard_hi;
};

// floor(sqrt(x)) for 0 <= x < 2^62, exact.
__host__ __device__ inline long long isqrt_ll(long long x) {
    if (x <= 0) return 0;
    long long r = (long long)sqrt((double)x);
    while (r * r > x) --r;
    while ((r + 1) * (r + 1) <= x) ++r;
    return r;
}

// Number of entries of the ascending table a[0..n) that are <= x.
__host__ __device__ inline int count_le(const int *a, int n, long long x) {
    int lo = 0, hi = n;
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (a[mid] <= x) lo = mid + 1; else hi = mid;
    }
    return lo;
}

// Base span length l(i) (Algorithm 1: l(i) = ceil(sqrt(i)) unless a fixed length is given; with a
// span exponent other than 1/2 the steps of ceil(i^p) come from the table).
__host__ __device__ inline long long base_len(long long i, int span_len, const int *len_first = nullptr,
                                              int n_len = 0) {
    if (span_len > 0) return span_len;
    if (i <= 0) return 0;
    if (len_first) return count_le(len_first, n_len, i);
    long long r = isqrt_ll(i);
    return r * r < i ? r + 1 : r;
}

// Stride pattern of a call.  In device code the device tables are read, in host code the host copies.
__host__ __device__ inline const int *pattern_off(const Call &c) {
#ifdef __CUDA_ARCH__
    return c.off;
#else
    return c.off_host;
#endif
}
__host__ __device__ inline const int *pattern_len(const Call &c) {
#ifdef __CUDA_ARCH__
    return c.len_first;
#else
    return c.len_first_host;
#endif
}
// Strides whose anchor exists for query position i: offsets <= i + 1.
__host__ __device__ inline int n_strides(const Call &c, long long i) {
    const int *off = pattern_off(c);
    return off ? count_le(off, c.n_off, i + 1) : (int)isqrt_ll(i + 1);
}
// Strides whose anchor lies inside the local window: offsets <= w.
__host__ __device__ inline int window_strides(const Call &c) {
    const int *off = pattern_off(c);
    return off ? count_le(off, c.n_off, c.window) : (int)isqrt_ll(c.window);
}
// Distance of the stride-s anchor from position i + 1.
__host__ __device__ inline int stride_offset(const Call &c, int s) {
    const int *off = pattern_off(c);
    return off ? off[s] : (s + 1) * (s + 1);
}
__host__ __device__ inline long long base_len(const Call &c, long long i) {
    return base_len(i, c.span_len, pattern_len(c), c.n_len);
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
