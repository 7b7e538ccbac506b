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
// anchors/scores.  `off`, when not NULL, is the table of stride offsets (else (s+1)^2).  All lanes of
// the warp take part.
__device__ inline void select_topk(float *sc, int n, int top_k, long long i, float *cand_v, int *cand_s,
                            int32_t *out_anchor, float *out_score, int lane, int s_base = 0,
                            const int *off = nullptr) {
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
        // D. rank of every candidate among the candidates (larger score first, smaller stride index on
        // ties: a strict total order on the order keys); ranks below top_k are the output slots
        uint32_t *cand_k = reinterpret_cast<uint32_t *>(cand_v);
        for (int cidx = lane; cidx < count; cidx += 32) cand_k[cidx] = order_key(cand_v[cidx]);
        __syncwarp();
        for (int cidx = lane; cidx < count; cidx += 32) {
            const uint32_t kc = cand_k[cidx];
            const int sc_ = cand_s[cidx];
            int rank = 0;
            for (int x = 0; x < count; ++x) {
                const uint32_t kx = cand_k[x];
                rank += (kx > kc) || (kx == kc && cand_s[x] < sc_);
            }
            if (rank < top_k) {
                const long long m = s_base + sc_ + 1;
                out_anchor[rank] = (int32_t)(i + 1 - (off ? (long long)off[m - 1] : m * m));
                out_score[rank] = __uint_as_float((kc & 0x80000000u) ? (kc & 0x7fffffffu) : ~kc);
            }
        }
        for (int j = count + lane; j < top_k; j += 32) {   // fewer candidates than slots: pad
            out_anchor[j] = -1;
            out_score[j] = -CUDART_INF_F;
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
                    out_anchor[j] = (int32_t)(i + 1 - (off ? (long long)off[s_base + bs]
                                                            : (long long)(s_base + bs + 1) * (s_base + bs + 1)));
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


// Top-k for HEADS heads at once (HEADS = 1, 2 or 4): the warp is split into HEADS groups of 32 / HEADS
// lanes and every group selects for its own head, so that the loop, vote and reduction instructions
// are issued once for all heads.  Same result as select_topk per head.
//   A. every lane keeps the T largest of its strided share of the head's n scores;
//   B. k rounds of a group-wide maximum over the lanes' current best give the k-th largest of those
//      T * lanes values: a threshold with at least k scores at or above it (needs k <= T * lanes);
//   C. the scores at or above the threshold are compacted into the head's candidate list;
//   D. every candidate's rank among the candidates (larger score first, smaller stride index on ties)
//      is its output slot.
// sc: scores of head x at sc[x * sc_stride + s]; cand_k / cand_s: HEADS * kCapG entries each; outputs of
// head x at out_*[x * out_stride + slot].  Returns false (for the whole warp, nothing written) when a
// head has more than kCapG candidates: the caller then falls back to select_topk.
constexpr int kCapG = 32;
template <int HEADS, int T>
__device__ inline bool select_topk_grouped(const float *sc, int sc_stride, int n, int top_k, long long i,
                                           uint32_t *cand_k, int *cand_s, int32_t *out_anchor, float *out_score,
                                           long long out_stride, int lane, int s_base, const int *off) {
    constexpr int LPH = 32 / HEADS;
    const int hh = lane / LPH, sub = lane % LPH;
    const uint32_t gmask = HEADS == 1 ? 0xffffffffu : (((1u << LPH) - 1u) << (hh * LPH));
    const float *my = sc + hh * sc_stride;
    // A. lane-local T largest keys (descending)
    uint32_t best[T];
#pragma unroll
    for (int t = 0; t < T; ++t) best[t] = 0u;
    for (int s = sub; s < n; s += LPH) {
        uint32_t kx = order_key(my[s]);
        kx = kx ? kx : 1u;   // 0 is "no entry"
#pragma unroll
        for (int t = 0; t < T; ++t) {
            const bool up = kx > best[t];
            const uint32_t lo_ = up ? best[t] : kx;
            best[t] = up ? kx : best[t];
            kx = lo_;
        }
    }
    // B. threshold: k-th largest of the group's lane-local bests
    uint32_t tau = 0u;
    const int rounds = n < top_k ? n : top_k;
    for (int j = 0; j < rounds; ++j) {
        const uint32_t mx = __reduce_max_sync(gmask, best[0]);
        tau = mx;
        const uint32_t who = __ballot_sync(0xffffffffu, best[0] == mx) & gmask;
        if (lane == __ffs(who) - 1) {
#pragma unroll
            for (int t = 0; t + 1 < T; ++t) best[t] = best[t + 1];
            best[T - 1] = 0u;
        }
    }
    if (rounds < top_k) tau = 1u;   // fewer scores than slots: everything is a candidate
    // C. compaction of the scores >= threshold, in stride order within each lane's share
    int count = 0;
    uint32_t *ck = cand_k + hh * kCapG;
    int *cs = cand_s + hh * kCapG;
    const int iters = (n + LPH - 1) / LPH;
    for (int it = 0; it < iters; ++it) {
        const int s = it * LPH + sub;
        uint32_t kx = 0u;
        if (s < n) {
            kx = order_key(my[s]);
            kx = kx ? kx : 1u;
        }
        const bool take = s < n && kx >= tau && tau != 0u;
        const uint32_t bits = __ballot_sync(0xffffffffu, take) & gmask;
        if (take) {
            const int pos = count + __popc(bits & ((1u << lane) - 1u));
            if (pos < kCapG) { ck[pos] = kx; cs[pos] = s; }
        }
        count += __popc(bits);
    }
    __syncwarp();
    if (__any_sync(0xffffffffu, count > kCapG)) return false;
    // D. rank among the candidates; pad the slots beyond them
    int32_t *oa = out_anchor + hh * out_stride;
    float *os = out_score + hh * out_stride;
    for (int cidx = sub; cidx < count; cidx += LPH) {
        const uint32_t kc = ck[cidx];
        const int sc_ = cs[cidx];
        int rank = 0;
        for (int x = 0; x < count; ++x) {
            const uint32_t kx = ck[x];
            rank += (kx > kc) || (kx == kc && cs[x] < sc_);
        }
        if (rank < top_k) {
            const long long m = s_base + sc_ + 1;
            oa[rank] = (int32_t)(i + 1 - (off ? (long long)off[m - 1] : m * m));
            os[rank] = __uint_as_float((kc & 0x80000000u) ? (kc & 0x7fffffffu) : ~kc);
        }
    }
    for (int j = count + sub; j < top_k; j += LPH) {
        oa[j] = -1;
        os[j] = -CUDART_INF_F;
    }
    __syncwarp();
    return true;
}


}  // namespace topk
}  // namespace sla
