// Warp-cooperative top-k over anchor scores held in shared memory (Section "Span search": TopK over
// Anchors(i)); shared by the prefill search kernel and the decode step.  Internal to libsla.
#pragma once

#include <limits.h>
#include <math_constants.h>
#include <stdint.h>

namespace sla {
namespace topk {

constexpr int kCap = 64;   // candidate slots per warp in the selection

__device__ __forceinline__ uint32_t order_key(float x) {
    const uint32_t u = __float_as_uint(x);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Top-k of sc[0..n) for one head, sc[x] being the score of stride index s_base + x (the strides
// below s_base have their anchors inside the local window and are no candidates); writes
// anchors/scores.  All lanes of the warp take part.
__device__ inline void select_topk(float *sc, int n, int top_k, long long i, float *cand_v, int *cand_s,
                            int32_t *out_anchor, float *out_score, int lane, int s_base = 0) {
    const uint32_t kNegInfKey = order_key(-CUDART_INF_F);
    // A. lane maxima over the strided slots
    float lm = -CUDART_INF_F;
    for (int s = lane; s < n; s += 32) lm = fmaxf(lm, sc[s]);
    // B. threshold = top_k-th largest lane maximum (there are at least top_k scores >= it)
    uint32_t cur = order_key(lm), tau_key = kNegInfKey;
    if (n > top_k && top_k <= 32) {
        for (int j = 0; j < top_k; ++j) {
            const uint32_t mx = __reduce_max_sync(0xffffffffu, cur);
            tau_key = mx;
            if (mx == kNegInfKey) break;
            const uint32_t who = __ballot_sync(0xffffffffu, cur == mx);
            if (lane == __ffs(who) - 1) cur = kNegInfKey;
        }
    }
    // C. compact the candidates >= threshold
    int count = 0;
    for (int s0 = 0; s0 < n; s0 += 32) {
        const int s = s0 + lane;
        const float v = s < n ? sc[s] : 0.f;
        const bool take = s < n && order_key(v) >= tau_key;
        const uint32_t mask = __ballot_sync(0xffffffffu, take);
        if (take) {
            const int pos = count + __popc(mask & ((1u << lane) - 1u));
            if (pos < kCap) { cand_v[pos] = v; cand_s[pos] = s; }
        }
        count += __popc(mask);
    }
    __syncwarp();
    if (count <= kCap) {
        // D. k rounds of warp arg-max over the candidates (two per lane)
        float v0 = lane < count ? cand_v[lane] : -CUDART_INF_F, v1 = lane + 32 < count ? cand_v[lane + 32] : -CUDART_INF_F;
        int s0 = lane < count ? cand_s[lane] : INT_MAX, s1 = lane + 32 < count ? cand_s[lane + 32] : INT_MAX;
        for (int j = 0; j < top_k; ++j) {
            const bool first = v0 > v1 || (v0 == v1 && s0 <= s1);
            const float bv = first ? v0 : v1;
            const int bs = first ? s0 : s1;
            const uint32_t mx = __reduce_max_sync(0xffffffffu, order_key(bv));
            const int smin = __reduce_min_sync(0xffffffffu, (order_key(bv) == mx && bs != INT_MAX) ? bs : INT_MAX);
            if (smin == INT_MAX) {   // fewer candidates than slots: pad
                if (lane == 0) { out_anchor[j] = -1; out_score[j] = -CUDART_INF_F; }
                continue;
            }
            if (bs == smin && order_key(bv) == mx) {
                out_anchor[j] = (int32_t)(i + 1 - (long long)(s_base + bs + 1) * (s_base + bs + 1));
                out_score[j] = bv;
                if (first) { v0 = -CUDART_INF_F; s0 = INT_MAX; } else { v1 = -CUDART_INF_F; s1 = INT_MAX; }
            }
        }
    } else {
        // many equal scores at the threshold: plain k rounds over all scores
        for (int j = 0; j < top_k; ++j) {
            float bv = -CUDART_INF_F;
            int bs = INT_MAX;
            for (int s = lane; s < n; s += 32) {
                const float v = sc[s];
                if (v > bv) { bv = v; bs = s; }
            }
#pragma unroll
            for (int off = 16; off >= 1; off >>= 1) {
                const float ov = __shfl_xor_sync(0xffffffffu, bv, off);
                const int os = __shfl_xor_sync(0xffffffffu, bs, off);
                if (ov > bv || (ov == bv && os < bs)) { bv = ov; bs = os; }
            }
            if (lane == 0) {
                if (bs != INT_MAX) {
                    out_anchor[j] = (int32_t)(i + 1 - (long long)(s_base + bs + 1) * (s_base + bs + 1));
                    out_score[j] = bv;
                    sc[bs] = -CUDART_INF_F;
                } else {
                    out_anchor[j] = -1;
                    out_score[j] = -CUDART_INF_F;
                }
            }
            __syncwarp();
        }
    }
    __syncwarp();
}


}  // namespace topk
}  // namespace sla
