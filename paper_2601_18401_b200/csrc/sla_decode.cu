// Decode step of libsla (Section "Kernel design", paragraph "Decoding path"): routing scores over
// the anchors of the single query position i = n_ctx-1, top-k, then attention over the routed spans
// read from the KV cache.  The step is bound by HBM reads of the selected K/V rows, so the attention
// kernel spreads each head's tokens evenly over many CTAs (split-K), streams whole rows with 16-byte
// loads, keeps a running (max, denominator, numerator) per lane group and merges at the end.
//
//   decode_score   grid (anchor chunks, B*Hkv, head tiles)   K anchor rows x G routing queries -> scores.  In
//                  the sequence-sharded step the CTA that finishes a (batch, KV head) last also selects this
//                  rank's k best candidates.
//   decode_attn    grid (n_splits, attention units)          every CTA first selects the k best anchors of its
//                  head from the scores (a threshold from the thread maxima, the candidates ranked), builds the
//                  spans of its unit and clips the overlaps -- redundantly per CTA, so that nothing waits for
//                  one CTA to do it for all -- then runs the online softmax over an even share of the tokens;
//                  the CTA that finishes a unit last merges the split results through their log-sum-exp.
//                  Union mode: one unit per head (its spans and the local window, clipped to disjoint pieces).
//                  Per-span mode (Algorithm 1 literally): one unit per selected anchor, J_t = S_t united with
//                  the window; the unit that finishes a head last applies the gate of Section "Combination" to
//                  the units' outputs.
// "Last" is decided by an atomic counter per unit / per head in the handle's header region; the last CTA puts
// the counter back to zero, so a step leaves them as it found them.
#include <limits.h>
#include <math_constants.h>

#include "sla_kernels.h"
#include "sla_topk.cuh"

namespace sla {

namespace {

constexpr int kScoreThreads = 256;
constexpr int kAttnThreads = 256;

template <int LPR> __device__ inline float reduce_sub(float x) {
#pragma unroll
    for (int off = LPR / 2; off >= 1; off >>= 1) x += __shfl_xor_sync(0xffffffffu, x, off);
    return x;
}

// ------------------------------------------------------------------------------------------------
template <typename T, int D, int GT>
__global__ void __launch_bounds__(kScoreThreads)
decode_score(const T *__restrict__ q_s, const T *__restrict__ k, Call c, long long n_ctx, int n, int s_min,
             float *__restrict__ scores, int *__restrict__ done, int *__restrict__ spans,
             int32_t *__restrict__ out_anchor, float *__restrict__ out_score) {
    extern __shared__ float dsm[];
    __shared__ int s_last;
    constexpr int E = Vec16<T>::kElems;
    constexpr int LPR = D / E;
    constexpr int RPI = 32 / LPR;
    constexpr int U = 2;
    constexpr int kWarps = kScoreThreads / 32;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int sub = lane % LPR, rsel = lane / LPR;
    const int g = blockIdx.y % c.Hkv, b = blockIdx.y / c.Hkv;
    const int h0 = g * c.G + blockIdx.z * GT;
    const long long i = n_ctx - 1;
    const T *kbase = k + b * c.kv_sb + g * c.kv_sh;

    // the attention kernel of this step may be scheduled now; it waits for this grid to finish before it
    // touches anything this kernel writes
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    float qv[GT][E];
#pragma unroll
    for (int t = 0; t < GT; ++t) Vec16<T>::load(q_s + b * c.q_sb + (long long)(h0 + t) * c.q_sh + sub * E, qv[t]);

    const int s_base = blockIdx.x * (kWarps * RPI * U);
    float part[U][GT];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const int s = s_base + (u * kWarps + warp) * RPI + rsel;
#pragma unroll
        for (int t = 0; t < GT; ++t) part[u][t] = 0.f;
        if (s < n) {
            // candidate x is stride s_min + x: the first s_min strides land inside the local window
            const long long tpos = i + 1 - stride_offset(c, s_min + s);
            float kv[E];
            Vec16<T>::load(kbase + tpos * c.kv_st + sub * E, kv);
#pragma unroll
            for (int t = 0; t < GT; ++t)
#pragma unroll
                for (int e = 0; e < E; ++e) part[u][t] = fmaf(qv[t][e], kv[e], part[u][t]);
        }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const int s = s_base + (u * kWarps + warp) * RPI + rsel;
#pragma unroll
        for (int t = 0; t < GT; ++t) {
            const float tot = reduce_sub<LPR>(part[u][t]);
            if (sub == 0 && s < n)
                scores[((long long)b * c.Hq + h0 + t) * n + s] = tot * c.search_scale;
        }
    }

    // the unsharded step selects in the attention kernel (every CTA for its own head): scores only
    if (!done) return;
    // ---- the CTA that completes this (batch, KV head) selects (sequence-sharded step: this rank's candidates)
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        const int total = gridDim.x * gridDim.z;
        const int prev = atomicAdd(done + blockIdx.y, 1);
        s_last = prev == total - 1;
        if (s_last) done[blockIdx.y] = 0;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    constexpr int kIv = kMaxTopK + 1;   // the spans and the window
    const int per_warp = n + 2 * topk::kCap + 4 * kIv;
    float *sc = dsm + (size_t)warp * per_warp;
    float *cand_v = sc + n;
    int *cand_s = reinterpret_cast<int *>(cand_v + topk::kCap);
    int *s_lo = cand_s + topk::kCap, *s_hi = s_lo + kIv, *p_lo = s_hi + kIv, *p_hi = p_lo + kIv;
    const long long ell = base_len(c, i);
    // span table of an attention unit: piece starts [pcap], cumulative token counts [pcap + 1], count
    const int pcap = c.mode == SLA_PER_SPAN ? 2 : c.top_k + 1, tstride = 2 * pcap + 2;
    for (int hg = warp; hg < c.G; hg += kWarps) {
        const long long bh = (long long)b * c.Hq + g * c.G + hg;
        const float *src = scores + bh * n;
        for (int s = lane; s < n; s += 32) sc[s] = __ldcg(src + s);   // written by other SMs: bypass L1
        __syncwarp();
        topk::select_topk(sc, n, c.top_k, i, cand_v, cand_s, out_anchor + bh * c.top_k, out_score + bh * c.top_k, lane,
                          s_min, c.off);
        __syncwarp();
        if (!spans) continue;   // sequence-sharded step: the spans are built after the global selection
        // intervals: the spans of the selected anchors (Algorithm 1: S_t = [max(0,t-b l), min(i,t+f l)])
        // and, last, the local window W = [max(0, i-w+1), i]
        const int n_iv = c.top_k + (c.window > 0 ? 1 : 0);
        const int w_lo = (int)(i - c.window + 1 > 0 ? i - c.window + 1 : 0);
        for (int j = lane; j < n_iv; j += 32) {
            int lo = INT_MAX, hi = -1;
            if (j == c.top_k) {
                lo = w_lo;
                hi = (int)i;
            } else {
                const long long t = out_anchor[bh * c.top_k + j];
                if (t >= 0) {
                    const long long a = t - (long long)c.back * ell, z = t + (long long)c.fwd * ell;
                    lo = (int)(a > 0 ? a : 0);
                    hi = (int)(z < i ? z : i);
                }
            }
            s_lo[j] = lo;
            s_hi[j] = hi;
        }
        __syncwarp();
        if (c.mode == SLA_PER_SPAN) {
            // one attention unit per selected anchor: the part of S_t left of the window, then the window
            if (lane == 0) {
                int n_sel = 0;
                for (int j = 0; j < c.top_k; ++j) n_sel += s_hi[j] >= 0;
                for (int j = 0; j < c.top_k; ++j) {
                    int *start = spans + (bh * c.top_k + j) * tstride;
                    int *cum = start + pcap;
                    int cnt = 0, total = 0;
                    cum[0] = 0;
                    // a head with nothing selected attends to the window alone: its first unit carries it
                    const bool sel = s_hi[j] >= 0, lone_w = n_sel == 0 && j == 0 && c.window > 0;
                    if (sel) {
                        const int hi_cut = c.window > 0 && s_hi[j] >= w_lo ? w_lo - 1 : s_hi[j];
                        if (s_lo[j] <= hi_cut) {
                            start[cnt] = s_lo[j];
                            total += hi_cut - s_lo[j] + 1;
                            cum[++cnt] = total;
                        }
                    }
                    if ((sel || lone_w) && c.window > 0) {
                        start[cnt] = w_lo;
                        total += (int)i - w_lo + 1;
                        cum[++cnt] = total;
                    }
                    start[2 * pcap + 1] = cnt;
                }
            }
            __syncwarp();
            continue;
        }
        // union mode: sort by (lo, hi), clip to disjoint pieces, cumulative token counts
        for (int j = lane; j < n_iv; j += 32) {
            const int lo = s_lo[j], hi = s_hi[j];
            int rank = 0;
            for (int m = 0; m < n_iv; ++m) {
                const int lm = s_lo[m], hm = s_hi[m];
                rank += (lm < lo) || (lm == lo && (hm < hi || (hm == hi && m < j)));
            }
            p_lo[rank] = lo;
            p_hi[rank] = hi;
        }
        __syncwarp();
        if (lane == 0) {
            int *start = spans + bh * tstride;
            int *cum = start + pcap;
            int cnt = 0;
            long long next_free = 0, total = 0;
            cum[0] = 0;
            for (int a = 0; a < n_iv; ++a) {
                const int lo = p_lo[a], hi = p_hi[a];
                if (hi < 0) break;
                const long long j0 = lo > next_free ? lo : next_free;
                if (j0 <= hi) {
                    start[cnt] = (int)j0;
                    total += hi - j0 + 1;
                    cum[cnt + 1] = (int)total;
                    ++cnt;
                }
                if ((long long)hi + 1 > next_free) next_free = (long long)hi + 1;
            }
            start[2 * pcap + 1] = cnt;
        }
        __syncwarp();
    }
}

// ------------------------------------------------------------------------------------------------
// Top-k of sc[0..n) by the whole CTA (Section "Span search": TopK over Anchors(i)); sc[x] is the score of
// stride index s_base + x.  Result in shared memory: sel_anchor[r] / sel_score[r], r = 0 .. top_k - 1, best
// first (larger score, then the nearer anchor, i.e. the smaller stride index), padded with (-1, -inf).
//   1. every thread takes the maximum of its contiguous run of scores;
//   2. the smallest of the maxima of k (rounded up to a power of two) groups of threads is a lower bound of the
//      k-th best score -- at least k scores lie at or above it -- and everything at or above it is a candidate;
//   3. the candidates are collected (typically a few more than k) and each one's rank among them is its slot.
// When more candidates turn up than the list holds (many equal scores), every warp selects the k best of its
// eighth of the scores with the warp routine of the prefill kernels instead, and the 8 k winners are ranked.
// May overwrite sc.
struct SelectSmem {
    static constexpr int kCand = 128;
    unsigned tmax[kAttnThreads];
    unsigned gmax[kMaxTopK];
    unsigned thr;
    int n_cand;
    unsigned cand_key[kCand];
    int cand_x[kCand];
    // fallback
    float cand_v[kAttnThreads / 32][topk::kCap];
    int cand_s[kAttnThreads / 32][topk::kCap];
    int32_t anchor[kAttnThreads / 32][kMaxTopK];
    float score[kAttnThreads / 32][kMaxTopK];
};

__device__ inline void cta_select_topk(float *sc, int n, int k, long long i, int s_base, const int *off, SelectSmem &m,
                                       int *sel_anchor, float *sel_score) {
    constexpr int kWarps = kAttnThreads / 32;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int per_t = (n + kAttnThreads - 1) / kAttnThreads;
    const int t0 = tid * per_t < n ? tid * per_t : n, t1 = t0 + per_t < n ? t0 + per_t : n;
    unsigned mx = 0u;   // below every order key of a real score
    for (int x = t0; x < t1; ++x) mx = max(mx, topk::order_key(sc[x]));
    m.tmax[tid] = mx;
    if (tid < k) {
        sel_anchor[tid] = -1;
        sel_score[tid] = -CUDART_INF_F;
    }
    if (tid == 0) m.n_cand = 0;
    __syncthreads();
    // Threshold: the threads form kp >= k groups (kp the next power of two); every group's maximum is a score
    // of its own, so at least k scores lie at or above the smallest group maximum: a lower bound of the k-th
    // best score that costs two short reductions instead of k rounds of a warp-wide maximum.
    int kp = 1;
    while (kp < k) kp <<= 1;
    const int gs = kAttnThreads / kp;   // threads per group (k <= 64: at least 4)
    if (tid < kp) {
        unsigned g = 0u;
        for (int j = 0; j < gs; ++j) g = max(g, m.tmax[tid * gs + j]);
        m.gmax[tid] = g;
    }
    __syncthreads();
    if (warp == 0) {
        unsigned lo = 0xffffffffu;
        int filled = 0;
        for (int j = lane; j < kp; j += 32) {
            const unsigned g = m.gmax[j];
            filled += g != 0u;
            lo = min(lo, g);
        }
        lo = __reduce_min_sync(0xffffffffu, lo);
        filled = __reduce_add_sync(0xffffffffu, filled);
        if (lane == 0) m.thr = filled >= k ? lo : 0u;   // fewer than k groups hold a score: everything is a candidate
    }
    __syncthreads();
    const unsigned thr = m.thr;
    for (int x = t0; x < t1; ++x) {
        const unsigned key = topk::order_key(sc[x]);
        if (key >= thr) {
            const int slot = atomicAdd(&m.n_cand, 1);
            if (slot < SelectSmem::kCand) {
                m.cand_key[slot] = key;
                m.cand_x[slot] = x;
            }
        }
    }
    __syncthreads();
    const int nc = m.n_cand;
    if (nc <= SelectSmem::kCand) {
        if (tid < nc) {
            const unsigned kc = m.cand_key[tid];
            const int xc = m.cand_x[tid];
            int rank = 0;
            for (int y = 0; y < nc; ++y) {
                const unsigned ky = m.cand_key[y];
                rank += (ky > kc) || (ky == kc && m.cand_x[y] < xc);
            }
            if (rank < k) {
                sel_anchor[rank] = (int)(i + 1 - (off ? (long long)off[s_base + xc] : (long long)(s_base + xc + 1) * (s_base + xc + 1)));
                sel_score[rank] = sc[xc];
            }
        }
        __syncthreads();
        return;
    }
    // ---- many equal scores: per-warp selection, then the warps' winners ranked
    const int per = (n + kWarps - 1) / kWarps;
    const int x0 = warp * per < n ? warp * per : n, x1 = x0 + per < n ? x0 + per : n;
    topk::select_topk(sc + x0, x1 - x0, k, i, m.cand_v[warp], m.cand_s[warp], m.anchor[warp], m.score[warp], lane,
                      s_base + x0, off);
    __syncthreads();
    for (int e = tid; e < kWarps * k; e += kAttnThreads) {
        const int w = e / k, j = e % k;
        const int a = m.anchor[w][j];
        if (a < 0) continue;
        const unsigned ka = topk::order_key(m.score[w][j]);
        int rank = 0;
        for (int w2 = 0; w2 < kWarps; ++w2)
            for (int j2 = 0; j2 < k; ++j2) {
                const int a2 = m.anchor[w2][j2];
                if (a2 < 0) break;   // a warp's winners come first, its padding last
                const unsigned k2 = topk::order_key(m.score[w2][j2]);
                rank += (k2 > ka) || (k2 == ka && a2 > a);
            }
        if (rank < k) {
            sel_anchor[rank] = a;
            sel_score[rank] = m.score[w][j];
        }
    }
    __syncthreads();
}

// Span table of one attention unit from the selected anchors (in shared memory: s_anchor[top_k], -1 = none),
// built by warp 0: piece starts in s_start, cumulative token counts in s_cum, returns the number of pieces.
// Union mode: the spans of the selected anchors (Algorithm 1: S_t = [max(0,t-b l), min(i,t+f l)]) and the local
// window W = [max(0, i-w+1), i], sorted by (lo, hi) and clipped to disjoint pieces.  Per-span mode: unit j is
// J_t of the j-th selected anchor, the part of S_t left of the window and then the window; a head with nothing
// selected attends to the window alone, carried by its first unit.
__device__ inline int build_unit_spans(const Call &c, long long i, int j_unit, const int *s_anchor, int *s_lo, int *s_hi,
                                       int *p_lo, int *p_hi, int *s_start, int *s_cum) {
    const int lane = threadIdx.x & 31;
    const long long ell = base_len(c, i);
    const int n_iv = c.top_k + (c.window > 0 ? 1 : 0);
    const int w_lo = (int)(i - c.window + 1 > 0 ? i - c.window + 1 : 0);
    for (int j = lane; j < n_iv; j += 32) {
        int lo = INT_MAX, hi = -1;
        if (j == c.top_k) {
            lo = w_lo;
            hi = (int)i;
        } else {
            const long long t = s_anchor[j];
            if (t >= 0) {
                const long long a = t - (long long)c.back * ell, z = t + (long long)c.fwd * ell;
                lo = (int)(a > 0 ? a : 0);
                hi = (int)(z < i ? z : i);
            }
        }
        s_lo[j] = lo;
        s_hi[j] = hi;
    }
    __syncwarp();
    int cnt = 0;
    if (c.mode == SLA_PER_SPAN) {
        if (lane == 0) {
            int n_sel = 0;
            for (int j = 0; j < c.top_k; ++j) n_sel += s_hi[j] >= 0;
            const int j = j_unit;
            int total = 0;
            s_cum[0] = 0;
            const bool sel = s_hi[j] >= 0, lone_w = n_sel == 0 && j == 0 && c.window > 0;
            if (sel) {
                const int hi_cut = c.window > 0 && s_hi[j] >= w_lo ? w_lo - 1 : s_hi[j];
                if (s_lo[j] <= hi_cut) {
                    s_start[cnt] = s_lo[j];
                    total += hi_cut - s_lo[j] + 1;
                    s_cum[++cnt] = total;
                }
            }
            if ((sel || lone_w) && c.window > 0) {
                s_start[cnt] = w_lo;
                total += (int)i - w_lo + 1;
                s_cum[++cnt] = total;
            }
        }
        return __shfl_sync(0xffffffffu, cnt, 0);
    }
    if (n_iv <= 32) {
        // a lane per interval, everything through shuffles: rank by (lo, hi), then, in sorted order, the running
        // maximum of the ends before an interval clips its start, a prefix sum of the lengths gives the
        // cumulative token counts and a ballot the slots of the pieces that are not empty
        const bool on = lane < n_iv;
        const int lo = on ? s_lo[lane] : INT_MAX, hi = on ? s_hi[lane] : -1;
        int rank = 0;
        for (int m = 0; m < n_iv; ++m) {
            const int lm = __shfl_sync(0xffffffffu, lo, m), hm = __shfl_sync(0xffffffffu, hi, m);
            rank += (lm < lo) || (lm == lo && (hm < hi || (hm == hi && m < lane)));
        }
        if (on) { p_lo[rank] = lo; p_hi[rank] = hi; }
        __syncwarp();
        const int slo = on ? p_lo[lane] : INT_MAX, shi = on ? p_hi[lane] : -1;   // sorted; absent intervals (hi < 0) last
        // exclusive running maximum of hi + 1 over the intervals before this one
        int end = shi + 1;   // 0 for an absent interval
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int y = __shfl_up_sync(0xffffffffu, end, off);
            if (lane >= off) end = max(end, y);
        }
        int prev_end = __shfl_up_sync(0xffffffffu, end, 1);
        if (lane == 0) prev_end = 0;
        const int j0 = max(slo, prev_end);
        const int len = (shi >= 0 && j0 <= shi) ? shi - j0 + 1 : 0;
        int incl = len;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int y = __shfl_up_sync(0xffffffffu, incl, off);
            if (lane >= off) incl += y;
        }
        const unsigned have = __ballot_sync(0xffffffffu, len > 0);
        if (len > 0) {
            const int idx = __popc(have & ((1u << lane) - 1u));
            s_start[idx] = j0;
            s_cum[idx + 1] = incl;
        }
        if (lane == 0) s_cum[0] = 0;
        return __popc(have);
    }
    for (int j = lane; j < n_iv; j += 32) {
        const int lo = s_lo[j], hi = s_hi[j];
        int rank = 0;
        for (int m = 0; m < n_iv; ++m) {
            const int lm = s_lo[m], hm = s_hi[m];
            rank += (lm < lo) || (lm == lo && (hm < hi || (hm == hi && m < j)));
        }
        p_lo[rank] = lo;
        p_hi[rank] = hi;
    }
    __syncwarp();
    if (lane == 0) {
        long long next_free = 0, total = 0;
        s_cum[0] = 0;
        for (int a = 0; a < n_iv; ++a) {
            const int lo = p_lo[a], hi = p_hi[a];
            if (hi < 0) break;
            const long long j0 = lo > next_free ? lo : next_free;
            if (j0 <= hi) {
                s_start[cnt] = (int)j0;
                total += hi - j0 + 1;
                s_cum[cnt + 1] = (int)total;
                ++cnt;
            }
            if ((long long)hi + 1 > next_free) next_free = (long long)hi + 1;
        }
    }
    return __shfl_sync(0xffffffffu, cnt, 0);
}

// `scores` [B*Hq][n_cand] (the unsharded step): every CTA selects the top-k of its head itself and builds its
// unit's spans -- nothing waits for a "last" CTA of the scoring kernel; the CTA of split 0 (of the head's first
// unit) writes the selection out.  `spans` (the sequence-sharded step): the table decode_shard_select built.
template <typename T, int D>
__global__ void __launch_bounds__(kAttnThreads)
decode_attn(const T *__restrict__ q, const T *__restrict__ k, const T *__restrict__ v, Call c,
            const int *__restrict__ spans, const float *__restrict__ scores, int n_cand, int s_min,
            float *__restrict__ partial, int *__restrict__ done,
            float *__restrict__ unit_out, int *__restrict__ done_head, int32_t *__restrict__ sel_anchor,
            float *__restrict__ sel_score, T *__restrict__ out, float *__restrict__ lse,
            float *__restrict__ shard_out) {
    extern __shared__ float s_scores[];   // [n_cand] (unsharded step)
    __shared__ int s_last;
    constexpr int E = Vec16<T>::kElems;
    constexpr int C = 2;                  // 16-byte chunks of a token row per lane: chunks sub and sub + LPR
    constexpr int LPR = D / (E * C);      // lanes per token row
    constexpr int RPI = 32 / LPR;
    constexpr int U = 4;
    constexpr int kWarps = kAttnThreads / 32;
    constexpr int kSlots = kWarps * RPI;  // token rows the CTA reads per load step
    constexpr int kIv = kMaxTopK + 1;
    __shared__ int s_start[kMaxTopK + 1], s_cum[kMaxTopK + 2];
    __shared__ float s_m[kSlots], s_l[kSlots];
    __shared__ float s_acc[kWarps][D];
    __shared__ SelectSmem s_sel;
    __shared__ int s_anchor[kMaxTopK], s_iv[4 * kIv], s_cnt;
    __shared__ float s_score[kMaxTopK];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int sub = lane % LPR, rsel = lane / LPR;
    // attention unit: a head (union mode) or one selected anchor of a head (per-span mode)
    const bool per_span = c.mode == SLA_PER_SPAN;
    const int units = per_span ? c.top_k : 1, pcap = per_span ? 2 : c.top_k + 1;
    const long long unit = blockIdx.y, bh = unit / units;
    const int h = (int)(bh % c.Hq), b = (int)(bh / c.Hq), g = h / c.G;
    const int n_splits = gridDim.x, split = blockIdx.x;

    // launched with programmatic stream serialization: everything above overlaps the tail of the
    // score kernel, whose results are read from here on
    asm volatile("griddepcontrol.wait;" ::: "memory");
    int cnt;
    if (scores) {
        const long long i = c.Lkv - 1;
        const float *src = scores + bh * n_cand;
        for (int x = tid; x < n_cand; x += kAttnThreads) s_scores[x] = __ldcg(src + x);
        __syncthreads();
        cta_select_topk(s_scores, n_cand, c.top_k, i, s_min, c.off, s_sel, s_anchor, s_score);
        if (tid < c.top_k && split == 0 && unit % units == 0) {
            sel_anchor[bh * c.top_k + tid] = s_anchor[tid];
            sel_score[bh * c.top_k + tid] = s_score[tid];
        }
        if (warp == 0) {
            const int n = build_unit_spans(c, i, (int)(unit % units), s_anchor, s_iv, s_iv + kIv, s_iv + 2 * kIv, s_iv + 3 * kIv,
                                           s_start, s_cum);
            if (lane == 0) s_cnt = n;
        }
        __syncthreads();
        cnt = s_cnt;
    } else {
        const int *sp = spans + unit * (2 * pcap + 2);
        cnt = sp[2 * pcap + 1];
        for (int j = tid; j < cnt; j += kAttnThreads) s_start[j] = sp[j];
        for (int j = tid; j <= cnt; j += kAttnThreads) s_cum[j] = sp[pcap + j];
        __syncthreads();
    }
    const long long total = cnt > 0 ? s_cum[cnt] : 0;
    const long long f_begin = total * split / n_splits, f_end = total * (split + 1) / n_splits;

    const T *kbase = k + b * c.kv_sb + g * c.kv_sh;
    const T *vbase = v + b * c.kv_sb + g * c.kv_sh;
    float qv[C][E];
    const float scale2 = c.softmax_scale * kLog2e;
#pragma unroll
    for (int ch = 0; ch < C; ++ch) {
        Vec16<T>::load(q + b * c.q_sb + (long long)h * c.q_sh + (ch * LPR + sub) * E, qv[ch]);
#pragma unroll
        for (int e = 0; e < E; ++e) qv[ch][e] *= scale2;
    }

    float m = -CUDART_INF_F, l = 0.f, acc[C][E];
#pragma unroll
    for (int ch = 0; ch < C; ++ch)
#pragma unroll
        for (int e = 0; e < E; ++e) acc[ch][e] = 0.f;
    int piece = 0;
    const int slot = warp * RPI + rsel;

    for (long long f0 = f_begin; f0 < f_end; f0 += kSlots * U) {
        uint4 kraw[U][C], vraw[U][C];
        bool ok[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const long long f = f0 + u * kSlots + slot;
            ok[u] = f < f_end;
            if (ok[u]) {
                while (f >= s_cum[piece + 1]) ++piece;
                const long long pos = s_start[piece] + (f - s_cum[piece]);
#pragma unroll
                for (int ch = 0; ch < C; ++ch) {
                    kraw[u][ch] = __ldg(reinterpret_cast<const uint4 *>(kbase + pos * c.kv_st + (ch * LPR + sub) * E));
                    vraw[u][ch] = __ldg(reinterpret_cast<const uint4 *>(vbase + pos * c.kv_st + (ch * LPR + sub) * E));
                }
            } else {
#pragma unroll
                for (int ch = 0; ch < C; ++ch) {
                    kraw[u][ch] = make_uint4(0, 0, 0, 0);
                    vraw[u][ch] = make_uint4(0, 0, 0, 0);
                }
            }
        }
        float x[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            x[u] = 0.f;
#pragma unroll
            for (int ch = 0; ch < C; ++ch) {
                float kv[E];
                if constexpr (sizeof(T) == 2) {
                    Vec16<__nv_bfloat16>::unpack(kraw[u][ch], kv);
                } else {
                    kv[0] = __uint_as_float(kraw[u][ch].x); kv[1] = __uint_as_float(kraw[u][ch].y);
                    kv[2] = __uint_as_float(kraw[u][ch].z); kv[3] = __uint_as_float(kraw[u][ch].w);
                }
#pragma unroll
                for (int e = 0; e < E; ++e) x[u] = fmaf(qv[ch][e], kv[e], x[u]);
            }
        }
        float m_new = m;
#pragma unroll
        for (int u = 0; u < U; ++u) {
            x[u] = reduce_sub<LPR>(x[u]);
            if (ok[u]) m_new = fmaxf(m_new, x[u]);
        }
        const float r = (m == -CUDART_INF_F) ? 0.f : exp2f(m - m_new);
        l *= r;
#pragma unroll
        for (int ch = 0; ch < C; ++ch)
#pragma unroll
            for (int e = 0; e < E; ++e) acc[ch][e] *= r;
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const float p = ok[u] ? exp2f(x[u] - m_new) : 0.f;
            l += p;
#pragma unroll
            for (int ch = 0; ch < C; ++ch) {
                float vv[E];
                if constexpr (sizeof(T) == 2) {
                    Vec16<__nv_bfloat16>::unpack(vraw[u][ch], vv);
                } else {
                    vv[0] = __uint_as_float(vraw[u][ch].x); vv[1] = __uint_as_float(vraw[u][ch].y);
                    vv[2] = __uint_as_float(vraw[u][ch].z); vv[3] = __uint_as_float(vraw[u][ch].w);
                }
#pragma unroll
                for (int e = 0; e < E; ++e) acc[ch][e] = fmaf(p, vv[e], acc[ch][e]);
            }
        }
        m = m_new;
    }

    // merge the lane groups of the warp, then the warps of the CTA
#pragma unroll
    for (int off = LPR; off < 32; off <<= 1) {
        const float om = __shfl_xor_sync(0xffffffffu, m, off);
        const float ol = __shfl_xor_sync(0xffffffffu, l, off);
        const float mn = fmaxf(m, om);
        const float a = (m == -CUDART_INF_F) ? 0.f : exp2f(m - mn);
        const float bb = (om == -CUDART_INF_F) ? 0.f : exp2f(om - mn);
        l = l * a + ol * bb;
#pragma unroll
        for (int ch = 0; ch < C; ++ch)
#pragma unroll
            for (int e = 0; e < E; ++e) {
                const float oa = __shfl_xor_sync(0xffffffffu, acc[ch][e], off);
                acc[ch][e] = acc[ch][e] * a + oa * bb;
            }
        m = mn;
    }
    if (rsel == 0) {
        if (sub == 0) { s_m[warp] = m; s_l[warp] = l; }
#pragma unroll
        for (int ch = 0; ch < C; ++ch)
#pragma unroll
            for (int e = 0; e < E; ++e) s_acc[warp][(ch * LPR + sub) * E + e] = acc[ch][e];
    }
    __syncthreads();
    if (tid < D) {
        float mm = -CUDART_INF_F;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) mm = fmaxf(mm, s_m[w]);
        float ll = 0.f, aa = 0.f;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) {
            const float sc = (s_m[w] == -CUDART_INF_F) ? 0.f : exp2f(s_m[w] - mm);
            ll += s_l[w] * sc;
            aa += s_acc[w][tid] * sc;
        }
        float *dst = partial + (unit * n_splits + split) * (D + 2);
        if (tid == 0) { dst[0] = mm; dst[1] = ll; }
        dst[2 + tid] = aa;
    }
    // ---- the CTA that completes this unit merges the split results
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const int prev = atomicAdd(done + unit, 1);
        s_last = prev == n_splits - 1;
        if (s_last) done[unit] = 0;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    float o_unit = 0.f, lse_unit = -CUDART_INF_F;
    if (tid < D) {
        const float *src = partial + unit * n_splits * (D + 2);
        float mm = -CUDART_INF_F;
        for (int s = 0; s < n_splits; ++s) mm = fmaxf(mm, __ldcg(src + s * (D + 2)));
        float ll = 0.f, aa = 0.f;
        for (int s = 0; s < n_splits; ++s) {
            const float ms = __ldcg(src + s * (D + 2));
            const float sc = (ms == -CUDART_INF_F) ? 0.f : exp2f(ms - mm);
            ll += __ldcg(src + s * (D + 2) + 1) * sc;
            aa += __ldcg(src + s * (D + 2) + 2 + tid) * sc;
        }
        o_unit = ll > 0.f ? aa / ll : 0.f;
        lse_unit = ll > 0.f ? (mm + log2f(ll)) * kLn2 : -CUDART_INF_F;
    }
    if (!per_span) {
        if (tid < D) {
            if (shard_out) {
                // sequence-sharded step: this rank's share of the head, merged with the others' later
                float *dst = shard_out + bh * (D + 2);
                dst[2 + tid] = o_unit;
                if (tid == 0) { dst[0] = lse_unit; dst[1] = 0.f; }
            } else {
                out[b * c.q_sb + (long long)h * c.q_sh + tid] = from_float<T>(o_unit);
                if (tid == 0) lse[bh] = lse_unit;
            }
        }
        return;
    }
    // ---- per-span mode: park A_t and its log-sum-exp; the unit that completes the head applies the gate
    if (tid < D) {
        float *dst = unit_out + unit * (D + 2);
        dst[2 + tid] = o_unit;
        if (tid == 0) dst[0] = lse_unit;
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const int prev = atomicAdd(done_head + bh, 1);
        s_last = prev == units - 1;
        if (s_last) done_head[bh] = 0;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    if (tid < D) {
        const int *an = s_anchor;      // every CTA of the head holds the head's selection
        const float *sc = s_score;
        const float *uo = unit_out + bh * units * (D + 2);
        float smax = -CUDART_INF_F;
        int n_sel = 0;
        for (int j = 0; j < c.top_k; ++j)
            if (an[j] >= 0) { smax = fmaxf(smax, sc[j]); ++n_sel; }
        float o = 0.f, l_first = -CUDART_INF_F;
        if (n_sel == 0) {
            // Algorithm 1, empty selection: the window alone (carried by the head's first unit)
            o = __ldcg(uo + 2 + tid);
            l_first = __ldcg(uo);
        } else {
            float sden = 0.f;
            for (int j = 0; j < c.top_k; ++j)
                if (an[j] >= 0) sden += expf(sc[j] - smax);
            bool first = true;
            for (int j = 0; j < c.top_k; ++j) {
                if (an[j] < 0) continue;
                o = fmaf(expf(sc[j] - smax) / sden, __ldcg(uo + j * (D + 2) + 2 + tid), o);
                if (first) { l_first = __ldcg(uo + j * (D + 2)); first = false; }
            }
        }
        out[b * c.q_sb + (long long)h * c.q_sh + tid] = from_float<T>(o);
        if (tid == 0) lse[bh] = l_first;
    }
}

// Dynamic shared memory above 48 KiB has to be allowed per kernel and device context.  The score kernel
// is given the largest size it can ever be launched with, once per (device, instantiation): later steps
// then launch without touching function attributes, whatever the context length.
constexpr int kScoreSmemMax = 200 * 1024;
template <typename K>
cudaError_t allow_score_smem(K kern, size_t smem) {
    static bool done[64] = {};
    if (smem <= 48 * 1024) return cudaSuccess;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return cudaErrorInvalidDevice;
    if (dev >= 0 && dev < 64 && done[dev]) return cudaSuccess;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kScoreSmemMax);
    if (e == cudaSuccess && dev >= 0 && dev < 64) done[dev] = true;
    return e;
}

template <typename T, int D>
cudaError_t decode_launch(const void *q_s, const void *q, const void *k, const void *v, const Call &c,
                          long long n_ctx, const DecodePlan &p, void *scratch, int *counters, void *out, float *lse,
                          int32_t *out_anchor, float *out_score, cudaStream_t st) {
    constexpr int E = Vec16<T>::kElems;
    constexpr int RPI = 32 / (D / E);
    char *base = (char *)scratch;
    float *scores = (float *)(base + p.off_scores);
    int *spans = (int *)(base + p.off_spans);
    float *partial = (float *)(base + p.off_partial);
    float *unit_out = (float *)(base + p.off_unit_out);
    const int units = c.mode == SLA_PER_SPAN ? c.top_k : 1;
    int *done_bg = counters, *done_unit = counters + c.B * c.Hkv, *done_head = done_unit + c.B * c.Hq * units;
    const int n = p.n_anchor, s_min = window_strides(c);
    const int rows_per_cta = (kScoreThreads / 32) * RPI * 2;
    const int gt = c.G % 8 == 0 ? 8 : c.G % 4 == 0 ? 4 : c.G % 2 == 0 ? 2 : 1;
    dim3 gs(n > 0 ? (n + rows_per_cta - 1) / rows_per_cta : 1, c.B * c.Hkv, c.G / gt);
    const T *qs = (const T *)q_s, *kk = (const T *)k;
    if ((size_t)n * sizeof(float) > 40 * 1024) return cudaErrorInvalidValue;   // the attention kernel holds a head's scores in shared memory
    cudaError_t e = cudaSuccess;
    // scores only (no completion counter, no shared memory): the attention kernel selects
#define SLA_LAUNCH_SCORE(GT)                                                                                         \
    decode_score<T, D, GT><<<gs, kScoreThreads, 0, st>>>(qs, kk, c, n_ctx, n, s_min, scores, (int *)nullptr,         \
                                                          (int *)nullptr, out_anchor, out_score)
    switch (gt) {
        case 8: SLA_LAUNCH_SCORE(8); break;
        case 4: SLA_LAUNCH_SCORE(4); break;
        case 2: SLA_LAUNCH_SCORE(2); break;
        default: SLA_LAUNCH_SCORE(1); break;
    }
#undef SLA_LAUNCH_SCORE
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    // programmatic dependent launch: the attention grid is set up while the score kernel drains
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(p.n_splits, c.B * c.Hq * units);
    cfg.blockDim = dim3(kAttnThreads);
    cfg.dynamicSmemBytes = (size_t)n * sizeof(float);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, decode_attn<T, D>, (const T *)q, kk, (const T *)v, c, (const int *)nullptr,
                              (const float *)scores, n, s_min, partial, done_unit, unit_out, done_head, out_anchor,
                              out_score, (T *)out, lse, (float *)nullptr);
}

// ------------------------------------------------------------------------------------------------
// Sequence-sharded decode step (the KV cache of one sequence split into contiguous position ranges, one
// per rank): every rank scores the anchors that fall into its range and keeps its k best
// (decode_score without a span table); the candidates of all ranks are gathered; every rank then picks
// the global k best, clips their spans to its own range (decode_shard_select), attends to that part
// (decode_attn with a partial result) and, after a second gather, all partial results are merged through
// their log-sum-exp (decode_shard_merge).  Union mode without a local window.

// One warp per (batch, query head): global top-k of the gathered candidates (larger score first, then the
// nearer anchor, i.e. the larger position: the order of the unsharded selection) and the table of this
// rank's pieces: the spans of the selected anchors, sorted, clipped to disjoint pieces and to
// [shard_lo, shard_hi).
__global__ void __launch_bounds__(32)
decode_shard_select(const int32_t *__restrict__ all_anchor, const float *__restrict__ all_score, int n_shards,
                    Call c, long long n_ctx, long long shard_lo, long long shard_hi, int32_t *__restrict__ out_anchor,
                    float *__restrict__ out_score, int *__restrict__ spans) {
    __shared__ int s_lo[kMaxTopK], s_hi[kMaxTopK];
    const int lane = threadIdx.x;
    const long long bh = blockIdx.x, n_bh = (long long)c.B * c.Hq;
    const int k = c.top_k, n = n_shards * k;
    const long long i = n_ctx - 1;
    for (int j = lane; j < k; j += 32) {
        out_anchor[bh * k + j] = -1;
        out_score[bh * k + j] = -CUDART_INF_F;
    }
    __syncwarp();
    for (int x = lane; x < n; x += 32) {
        const long long src = ((long long)(x / k) * n_bh + bh) * k + x % k;
        const int ax = all_anchor[src];
        if (ax < 0) continue;
        const uint32_t kx = topk::order_key(all_score[src]);
        int rank = 0;
        for (int y = 0; y < n; ++y) {
            const long long sy = ((long long)(y / k) * n_bh + bh) * k + y % k;
            const int ay = all_anchor[sy];
            if (ay < 0) continue;
            const uint32_t ky = topk::order_key(all_score[sy]);
            rank += (ky > kx) || (ky == kx && ay > ax);
        }
        if (rank < k) {
            out_anchor[bh * k + rank] = ax;
            out_score[bh * k + rank] = all_score[src];
        }
    }
    __syncwarp();
    if (lane == 0) {
        // spans of the selected anchors (Algorithm 1: S_t = [max(0,t-b l), min(i,t+f l)]), insertion-sorted
        const long long ell = base_len(c, i);
        int m = 0;
        for (int j = 0; j < k; ++j) {
            const long long t = out_anchor[bh * k + j];
            if (t < 0) continue;
            const long long a = t - (long long)c.back * ell, z = t + (long long)c.fwd * ell;
            const int l0 = (int)(a > 0 ? a : 0), h0 = (int)(z < i ? z : i);
            int pos = m;
            while (pos > 0 && (s_lo[pos - 1] > l0 || (s_lo[pos - 1] == l0 && s_hi[pos - 1] > h0))) {
                s_lo[pos] = s_lo[pos - 1];
                s_hi[pos] = s_hi[pos - 1];
                --pos;
            }
            s_lo[pos] = l0;
            s_hi[pos] = h0;
            ++m;
        }
        const int pcap = k + 1;
        int *start = spans + bh * (2 * pcap + 2);
        int *cum = start + pcap;
        int cnt = 0;
        long long next_free = 0, total = 0;
        cum[0] = 0;
        for (int a = 0; a < m; ++a) {
            long long j0 = s_lo[a] > next_free ? s_lo[a] : next_free;
            if ((long long)s_hi[a] + 1 > next_free) next_free = (long long)s_hi[a] + 1;
            // this rank's part of the piece
            long long j1 = s_hi[a];
            if (j0 < shard_lo) j0 = shard_lo;
            if (j1 > shard_hi - 1) j1 = shard_hi - 1;
            if (j0 <= j1) {
                start[cnt] = (int)j0;
                total += j1 - j0 + 1;
                cum[cnt + 1] = (int)total;
                ++cnt;
            }
        }
        start[2 * pcap + 1] = cnt;
    }
}

// One CTA per (batch, query head): merge of the ranks' partial results {lse, -, o[D]} (fp32).
template <typename T, int D>
__global__ void __launch_bounds__(D)
decode_shard_merge(const float *__restrict__ all_partial, int n_shards, Call c, T *__restrict__ out,
                   float *__restrict__ lse) {
    const long long bh = blockIdx.x, n_bh = (long long)c.B * c.Hq;
    const int h = (int)(bh % c.Hq), b = (int)(bh / c.Hq), tid = threadIdx.x;
    float mm = -CUDART_INF_F;
    for (int w = 0; w < n_shards; ++w) mm = fmaxf(mm, all_partial[((long long)w * n_bh + bh) * (D + 2)]);
    float den = 0.f, acc = 0.f;
    if (mm > -CUDART_INF_F) {
        for (int w = 0; w < n_shards; ++w) {
            const float *src = all_partial + ((long long)w * n_bh + bh) * (D + 2);
            if (src[0] == -CUDART_INF_F) continue;
            const float wt = expf(src[0] - mm);
            den += wt;
            acc = fmaf(wt, src[2 + tid], acc);
        }
    }
    out[b * c.q_sb + (long long)h * c.q_sh + tid] = from_float<T>(den > 0.f ? acc / den : 0.f);
    if (tid == 0) lse[bh] = den > 0.f ? mm + logf(den) : -CUDART_INF_F;
}

template <typename T, int D>
cudaError_t shard_search_launch(const void *q_s, const void *k_local, const Call &c, long long n_ctx, int s_first,
                                int n, void *scratch, int *counters, int32_t *cand_anchor, float *cand_score,
                                cudaStream_t st) {
    constexpr int E = Vec16<T>::kElems;
    constexpr int RPI = 32 / (D / E);
    float *scores = (float *)scratch;
    const int rows_per_cta = (kScoreThreads / 32) * RPI * 2;
    const int gt = c.G % 8 == 0 ? 8 : c.G % 4 == 0 ? 4 : c.G % 2 == 0 ? 2 : 1;
    dim3 gs(n > 0 ? (n + rows_per_cta - 1) / rows_per_cta : 1, c.B * c.Hkv, c.G / gt);
    // positions are global: the local slice starts at shard_lo
    const T *qs = (const T *)q_s, *kk = (const T *)k_local - c.shard_lo * c.kv_st;
    const size_t smem = (size_t)(kScoreThreads / 32) * (n + 2 * topk::kCap + 4 * (kMaxTopK + 1)) * sizeof(float);
    if (smem > (size_t)kScoreSmemMax) return cudaErrorInvalidValue;
    cudaError_t e = cudaSuccess;
#define SLA_LAUNCH_SCORE(GT)                                                                                         \
    do {                                                                                                             \
        auto kern = decode_score<T, D, GT>;                                                                          \
        e = allow_score_smem(kern, smem);                                                                            \
        if (e == cudaSuccess)                                                                                        \
            kern<<<gs, kScoreThreads, smem, st>>>(qs, kk, c, n_ctx, n, s_first, scores, counters, (int *)nullptr,    \
                                                  cand_anchor, cand_score);                                         \
    } while (0)
    switch (gt) {
        case 8: SLA_LAUNCH_SCORE(8); break;
        case 4: SLA_LAUNCH_SCORE(4); break;
        case 2: SLA_LAUNCH_SCORE(2); break;
        default: SLA_LAUNCH_SCORE(1); break;
    }
#undef SLA_LAUNCH_SCORE
    if (e != cudaSuccess) return e;
    return cudaGetLastError();
}

template <typename T, int D>
cudaError_t shard_attend_launch(const void *q, const void *k_local, const void *v_local, const Call &c, long long n_ctx,
                                const DecodePlan &p, void *scratch, int *counters, int n_shards,
                                const int32_t *all_anchor, const float *all_score, int32_t *out_anchor,
                                float *out_score, float *partial_out, cudaStream_t st) {
    char *base = (char *)scratch;
    int *spans = (int *)(base + p.off_spans);
    float *partial = (float *)(base + p.off_partial);
    int *done_unit = counters + c.B * c.Hkv, *done_head = done_unit + c.B * c.Hq;
    decode_shard_select<<<c.B * c.Hq, 32, 0, st>>>(all_anchor, all_score, n_shards, c, n_ctx, c.shard_lo, c.shard_hi,
                                                   out_anchor, out_score, spans);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const T *kk = (const T *)k_local - c.shard_lo * c.kv_st, *vv = (const T *)v_local - c.shard_lo * c.kv_st;
    decode_attn<T, D><<<dim3(p.n_splits, c.B * c.Hq), kAttnThreads, 0, st>>>(
        (const T *)q, kk, vv, c, spans, (const float *)nullptr, 0, 0, partial, done_unit, (float *)nullptr, done_head,
        out_anchor, out_score, (T *)nullptr, (float *)nullptr, partial_out);
    return cudaGetLastError();
}

}  // namespace

#define SLA_DISPATCH(fn, ...)                                                                    \
    (dtype == SLA_F32 ? (c.D == 64 ? fn<float, 64>(__VA_ARGS__) : fn<float, 128>(__VA_ARGS__))   \
                      : (c.D == 64 ? fn<__nv_bfloat16, 64>(__VA_ARGS__) : fn<__nv_bfloat16, 128>(__VA_ARGS__)))

cudaError_t launch_decode_shard_search(const void *q_s, const void *k_local, const Call &c, int dtype,
                                       long long n_ctx, int s_first, int n, void *scratch, int *counters,
                                       int32_t *cand_anchor, float *cand_score, cudaStream_t st) {
    return SLA_DISPATCH(shard_search_launch, q_s, k_local, c, n_ctx, s_first, n, scratch, counters, cand_anchor,
                        cand_score, st);
}

cudaError_t launch_decode_shard_attend(const void *q, const void *k_local, const void *v_local, const Call &c,
                                       int dtype, long long n_ctx, const DecodePlan &plan, void *scratch,
                                       int *counters, int n_shards, const int32_t *all_anchor,
                                       const float *all_score, int32_t *out_anchor, float *out_score,
                                       float *partial_out, cudaStream_t st) {
    return SLA_DISPATCH(shard_attend_launch, q, k_local, v_local, c, n_ctx, plan, scratch, counters, n_shards,
                        all_anchor, all_score, out_anchor, out_score, partial_out, st);
}

cudaError_t launch_decode_shard_merge(const float *all_partial, int n_shards, const Call &c, int dtype, void *out,
                                      float *lse, cudaStream_t st) {
    const unsigned grid = (unsigned)(c.B * c.Hq);
    if (dtype == SLA_F32) {
        if (c.D == 64) decode_shard_merge<float, 64><<<grid, 64, 0, st>>>(all_partial, n_shards, c, (float *)out, lse);
        else decode_shard_merge<float, 128><<<grid, 128, 0, st>>>(all_partial, n_shards, c, (float *)out, lse);
    } else {
        if (c.D == 64)
            decode_shard_merge<__nv_bfloat16, 64><<<grid, 64, 0, st>>>(all_partial, n_shards, c, (__nv_bfloat16 *)out, lse);
        else
            decode_shard_merge<__nv_bfloat16, 128><<<grid, 128, 0, st>>>(all_partial, n_shards, c, (__nv_bfloat16 *)out, lse);
    }
    return cudaGetLastError();
}
#undef SLA_DISPATCH


int decode_attn_blocks_per_sm(int dtype, int D) {
    // resident CTAs per SM with the shared memory a 16M-token context needs for a head's anchor scores
    constexpr size_t kOccSmem = 16 * 1024;
    static int cache[2][2] = {{0, 0}, {0, 0}};
    int &slot = cache[dtype == SLA_F32 ? 0 : 1][D == 64 ? 0 : 1];
    if (slot == 0) {
        int n = 0;
        cudaError_t e;
        if (dtype == SLA_F32)
            e = D == 64 ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, decode_attn<float, 64>, kAttnThreads, kOccSmem)
                        : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, decode_attn<float, 128>, kAttnThreads, kOccSmem);
        else
            e = D == 64 ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, decode_attn<__nv_bfloat16, 64>, kAttnThreads, kOccSmem)
                        : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, decode_attn<__nv_bfloat16, 128>, kAttnThreads, kOccSmem);
        slot = (e == cudaSuccess && n > 0) ? n : 1;
    }
    return slot;
}

DecodePlan plan_decode(const Call &c, long long n_ctx, int cta_slots, size_t gap) {
    DecodePlan p;
    // candidates: the strides whose anchor lies left of the local window
    const long long n_cand = n_strides(c, n_ctx - 1) - window_strides(c);
    p.n_anchor = (int)(n_cand > 0 ? n_cand : 0);
    const long long ell = base_len(c, n_ctx - 1);
    long long span_tokens = (long long)(c.back + c.fwd) * ell + 1;
    if (span_tokens > n_ctx) span_tokens = n_ctx;
    const bool per_span = c.mode == SLA_PER_SPAN;
    const int units = per_span ? c.top_k : 1, pcap = per_span ? 2 : c.top_k + 1;
    const long long win = c.window < n_ctx ? c.window : n_ctx;
    const long long max_tokens = per_span ? span_tokens + win : span_tokens * c.top_k + win;
    // one resident wave: as many splits per attention unit as fit the CTA slots of the device
    long long ns = (long long)cta_slots / ((long long)c.B * c.Hq * units);
    if (ns > max_tokens / 128) ns = max_tokens / 128;
    if (ns > 256) ns = 256;
    if (ns < 1) ns = 1;
    p.n_splits = (int)ns;
    const size_t bh = (size_t)c.B * c.Hq, n_units = bh * units;
    size_t off = 0;
    // a region of `size` bytes at the next 256-byte boundary, with a canary gap before it when asked for
    auto take = [&](size_t size) {
        if (gap) { p.canaries.add(off); off += gap; }
        const size_t at = off;
        off = (off + size + 255) & ~(size_t)255;
        return at;
    };
    p.off_scores = take(bh * (size_t)p.n_anchor * sizeof(float));
    p.off_spans = take(n_units * (size_t)(2 * pcap + 2) * sizeof(int));
    p.off_partial = take(n_units * (size_t)p.n_splits * (c.D + 2) * sizeof(float));
    p.off_unit_out = take(per_span ? n_units * (size_t)(c.D + 2) * sizeof(float) : 0);
    if (gap) { p.canaries.add(off); off += gap; }
    p.bytes = off;
    return p;
}

cudaError_t launch_decode(const void *q_s, const void *q, const void *k, const void *v, const Call &c,
                          int dtype, long long n_ctx, const DecodePlan &plan, void *scratch, int *counters,
                          void *out, float *lse, int32_t *out_anchor, float *out_score, cudaStream_t st) {
    if (dtype == SLA_F32) {
        return c.D == 64 ? decode_launch<float, 64>(q_s, q, k, v, c, n_ctx, plan, scratch, counters, out, lse, out_anchor, out_score, st)
                         : decode_launch<float, 128>(q_s, q, k, v, c, n_ctx, plan, scratch, counters, out, lse, out_anchor, out_score, st);
    }
    return c.D == 64 ? decode_launch<__nv_bfloat16, 64>(q_s, q, k, v, c, n_ctx, plan, scratch, counters, out, lse, out_anchor, out_score, st)
                     : decode_launch<__nv_bfloat16, 128>(q_s, q, k, v, c, n_ctx, plan, scratch, counters, out, lse, out_anchor, out_score, st);
}

// ------------------------------------------------------------------------------------------------
// Decode step for callers that cannot allocate device memory (declared in include/sla.h).
//
// Some hosts of this library run where cudaMalloc is off limits: inside a CUDA-graph capture or a
// stream-ordered region of a serving loop, in a process whose device memory is handed out in full to
// another allocator at start-up, or in a plug-in that is only lent a stream.  They cannot create an
// sla handle (its workspace is a cudaMalloc).  For them the decode step's scratch -- anchor scores,
// clipped spans, split results and the completion counters -- lives in the array below, which is
// part of the library image: every GPU that loads the library holds these 2 MiB until the process
// exits, whether or not the entry point is ever called.
namespace {

constexpr size_t kStaticScratchBytes = SLA_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_decode_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
// Device addresses of the array, one per device.  In host code the array's name is only a handle for
// the runtime: the address a kernel may use comes from cudaGetSymbolAddress, asked once per device
// with that device current.
unsigned char *g_decode_scratch_ptr[kMaxDevices] = {};
int g_cta_slots[kMaxDevices][2][2] = {};

}  // namespace
}  // namespace sla

extern "C" sla_status_t sla_decode_step_static(const void *q_s, const void *q, const void *k_cache,
                                               const void *v_cache, int64_t n_ctx, const sla_layout_t *l,
                                               const sla_params_t *p, void *out, float *lse, int32_t *out_anchor,
                                               float *out_score, void *stream) {
    sla::Call c;
    if (sla_status_t s = sla::check_decode_args(q_s, q, k_cache, v_cache, n_ctx, l, p, out, lse, out_anchor, out_score, &c))
        return s;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return SLA_ERR_CUDA;
    if (dev < 0 || dev >= sla::kMaxDevices) return SLA_ERR_UNSUPPORTED;
    if (!sla::g_decode_scratch_ptr[dev]) {
        // set-up, once per device (the current one): resolve the array's device address
        void *ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, sla::g_decode_scratch) != cudaSuccess || !ptr) return SLA_ERR_CUDA;
        sla::g_decode_scratch_ptr[dev] = static_cast<unsigned char *>(ptr);
    }
    int &slots = sla::g_cta_slots[dev][l->dtype == SLA_F32 ? 0 : 1][l->head_dim == 64 ? 0 : 1];
    if (slots == 0) {
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return SLA_ERR_CUDA;
        slots = sms * sla::decode_attn_blocks_per_sm(l->dtype, l->head_dim);
    }
    const sla::DecodePlan plan = sla::plan_decode(c, n_ctx, slots);
    const size_t counter_bytes = (((size_t)l->batch * (l->n_kv_heads + l->n_q_heads) * sizeof(int)) + 255) & ~(size_t)255;
    if (counter_bytes + plan.bytes > sla::kStaticScratchBytes) return SLA_ERR_WORKSPACE;   // beyond the fixed maximum
    if ((size_t)plan.n_anchor * sizeof(float) * 8 > 180 * 1024) return SLA_ERR_UNSUPPORTED;
    unsigned char *base = sla::g_decode_scratch_ptr[dev];
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // the array keeps whatever the previous call left; only the completion counters have to start at zero
    if (cudaMemsetAsync(base, 0, counter_bytes, st) != cudaSuccess) return SLA_ERR_CUDA;
    cudaError_t e = sla::launch_decode(q_s, q, k_cache, v_cache, c, l->dtype, n_ctx, plan, base + counter_bytes,
                                       reinterpret_cast<int *>(base), out, lse, out_anchor, out_score, st);
    return e == cudaSuccess ? SLA_OK : SLA_ERR_CUDA;
}
