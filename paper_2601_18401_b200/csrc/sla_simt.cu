// Generic SIMT kernels of libsla: exact-fp32 span-search and span-attention, one warp per query row.
//
// These kernels serve the fp32 path (where tensor-core inputs would lose the precision the 1e-4
// bound needs) and every shape or parameter set the tensor-core kernels do not cover.  A row of K or
// V is read by LPR = D*sizeof(T)/16 adjacent lanes, 16 bytes each, so a warp instruction always
// fetches whole, consecutive rows.
#include <limits.h>
#include <math_constants.h>

#include "sla_kernels.h"

namespace sla {

namespace {

constexpr int kWarpsPerBlock = 4;

// Decodes the flat row id used by both kernels.  Rows are ordered ((b*Hkv + g)*Lq + r)*G + hg so
// that the warps of a block are the query heads of one group at one position: they read the same
// key rows and hit in L1.
struct RowId {
    int b, g, h;
    long long r;
};
__device__ inline RowId decode_row(long long row, const Call &c) {
    RowId o;
    int hg = (int)(row % c.G);
    long long t1 = row / c.G;
    o.r = t1 % c.Lq;
    long long bg = t1 / c.Lq;
    o.g = (int)(bg % c.Hkv);
    o.b = (int)(bg / c.Hkv);
    o.h = o.g * c.G + hg;
    return o;
}

template <int LPR> __device__ inline float reduce_sub(float x) {
#pragma unroll
    for (int off = LPR / 2; off >= 1; off >>= 1) x += __shfl_xor_sync(0xffffffffu, x, off);
    return x;
}

// ------------------------------------------------------------------------------------------------
// Span-search (Section "Span search": s_{i,t} = <Q_s(i), K(t)> over Anchors(i), then TopK).
// Scores of all n(i) anchors go to shared memory; the k best are then pulled out one by one
// (largest score first, smaller stride index on ties).
// ------------------------------------------------------------------------------------------------
template <typename T, int D>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
search_rows_simt(const T *__restrict__ q_s, const T *__restrict__ k, Call c,
                 int32_t *__restrict__ out_anchor, float *__restrict__ out_score, int n_max) {
    constexpr int E = Vec16<T>::kElems;
    constexpr int LPR = D / E;
    constexpr int RPI = 32 / LPR;
    constexpr int U = 4;
    extern __shared__ float smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long row = (long long)blockIdx.x * kWarpsPerBlock + warp;
    if (row >= (long long)c.B * c.Hq * c.Lq) return;
    const RowId id = decode_row(row, c);
    const long long i = c.q_pos0 + id.r;
    // Algorithm 1: T = Anchors(i) without the window; t_s lies in W exactly when (s+1)^2 <= w
    const int s_min = window_strides(c);
    const int n = n_strides(c, i);
    float *sc = smem + (size_t)warp * n_max;
    const T *qrow = q_s + id.b * c.q_sb + id.h * c.q_sh + id.r * c.q_st;
    const T *kbase = k + id.b * c.kv_sb + id.g * c.kv_sh;
    const int sub = lane % LPR, rsel = lane / LPR;
    float qv[E];
    Vec16<T>::load(qrow + sub * E, qv);

    for (int s = lane; s < s_min && s < n; s += 32) sc[s] = -CUDART_INF_F;
    for (int s0 = s_min; s0 < n; s0 += RPI * U) {
        float part[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int s = s0 + u * RPI + rsel;
            part[u] = 0.f;
            if (s < n) {
                const long long t = i + 1 - stride_offset(c, s);
                float kv[E];
                Vec16<T>::load(kbase + t * c.kv_st + sub * E, kv);
#pragma unroll
                for (int e = 0; e < E; ++e) part[u] = fmaf(qv[e], kv[e], part[u]);
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const float tot = reduce_sub<LPR>(part[u]);
            const int s = s0 + u * RPI + rsel;
            if (sub == 0 && s < n) sc[s] = tot * c.search_scale;
        }
    }
    __syncwarp();

    const long long obase = ((((long long)id.b * c.Hq + id.h) * c.Lq) + id.r) * c.top_k;
    for (int j = 0; j < c.top_k; ++j) {
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
                out_anchor[obase + j] = (int32_t)(i + 1 - stride_offset(c, bs));
                out_score[obase + j] = bv;
                sc[bs] = -CUDART_INF_F;
            } else {
                out_anchor[obase + j] = -1;
                out_score[obase + j] = -CUDART_INF_F;
            }
        }
        __syncwarp();
    }
}

// ------------------------------------------------------------------------------------------------
// Span-attention (Section "Span attention", equation for A_{i,t}; Algorithm 1 span construction).
//   union mode     the selected spans of a row (and the local window W, if any) are sorted, overlaps
//                  are clipped away, and one online softmax runs over the remaining disjoint pieces;
//   per-span mode  Algorithm 1 literally: for every selected anchor t one softmax over
//                  J_t = S_t united with W, then O = sum_t alpha_t A_t with alpha = softmax of the
//                  search scores (Section "Combination"); an empty selection attends to W alone.
// ------------------------------------------------------------------------------------------------

// Online softmax of one row over n disjoint key intervals (base-2 exponentials).  On return every
// lane holds the warp's merged maximum m, denominator l and its E columns of the unnormalised output.
template <typename T, int D, int E>
__device__ inline void attend_intervals(const float (&qv)[E], const T *kbase, const T *vbase, long long kv_st,
                                        const int *iv_lo, const int *iv_hi, int n, int sub, int rsel,
                                        float &m, float &l, float (&acc)[E]) {
    constexpr int LPR = D / E;
    constexpr int RPI = 32 / LPR;
    constexpr int U = 2;
    m = -CUDART_INF_F;
    l = 0.f;
#pragma unroll
    for (int e = 0; e < E; ++e) acc[e] = 0.f;
    for (int pc = 0; pc < n; ++pc) {
        const int lo = iv_lo[pc], hi = iv_hi[pc];
        for (long long j0 = lo; j0 <= hi; j0 += RPI * U) {
            float x[U], vv[U][E];
            bool ok[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const long long j = j0 + u * RPI + rsel;
                ok[u] = j <= hi;
                x[u] = 0.f;
                if (ok[u]) {
                    float kv[E];
                    Vec16<T>::load(kbase + j * kv_st + sub * E, kv);
                    Vec16<T>::load(vbase + j * kv_st + sub * E, vv[u]);
#pragma unroll
                    for (int e = 0; e < E; ++e) x[u] = fmaf(qv[e], kv[e], x[u]);
                } else {
#pragma unroll
                    for (int e = 0; e < E; ++e) vv[u][e] = 0.f;
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
            for (int e = 0; e < E; ++e) acc[e] *= r;
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const float p = ok[u] ? exp2f(x[u] - m_new) : 0.f;
                l += p;
#pragma unroll
                for (int e = 0; e < E; ++e) acc[e] = fmaf(p, vv[u][e], acc[e]);
            }
            m = m_new;
        }
    }
    // merge the RPI sub-groups of the warp
#pragma unroll
    for (int off = LPR; off < 32; off <<= 1) {
        const float om = __shfl_xor_sync(0xffffffffu, m, off);
        const float ol = __shfl_xor_sync(0xffffffffu, l, off);
        const float mn = fmaxf(m, om);
        const float a = (m == -CUDART_INF_F) ? 0.f : exp2f(m - mn);
        const float b = (om == -CUDART_INF_F) ? 0.f : exp2f(om - mn);
        l = l * a + ol * b;
#pragma unroll
        for (int e = 0; e < E; ++e) {
            const float oa = __shfl_xor_sync(0xffffffffu, acc[e], off);
            acc[e] = acc[e] * a + oa * b;
        }
        m = mn;
    }
}

template <typename T, int D>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
attn_rows_simt(const T *__restrict__ q, const T *__restrict__ k, const T *__restrict__ v, Call c,
               const int32_t *__restrict__ anchor, const float *__restrict__ score, T *__restrict__ out,
               float *__restrict__ lse, float *__restrict__ lse_span) {
    constexpr int E = Vec16<T>::kElems;
    constexpr int LPR = D / E;
    constexpr int kIv = kMaxTopK + 1;   // the spans and the window
    __shared__ int s_lo[kWarpsPerBlock][kIv], s_hi[kWarpsPerBlock][kIv];
    __shared__ int p_lo[kWarpsPerBlock][kIv], p_hi[kWarpsPerBlock][kIv];
    __shared__ int p_cnt[kWarpsPerBlock];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long row = (long long)blockIdx.x * kWarpsPerBlock + warp;
    if (row >= (long long)c.B * c.Hq * c.Lq) return;
    const RowId id = decode_row(row, c);
    const long long i = c.q_pos0 + id.r;
    const long long ell = base_len(c, i);
    const long long orow_idx = (((long long)id.b * c.Hq + id.h) * c.Lq) + id.r;
    const long long abase = orow_idx * c.top_k;
    const int n_iv = c.top_k + (c.window > 0 ? 1 : 0);
    const int w_lo = (int)(i - c.window + 1 > 0 ? i - c.window + 1 : 0);   // W = [w_lo, i] when window > 0

    // 1. spans of the selected anchors; invalid entries become empty and sort last
    for (int j = lane; j < n_iv; j += 32) {
        int lo = INT_MAX, hi = -1;
        if (j == c.top_k) {
            lo = w_lo;
            hi = (int)i;
        } else {
            const long long t = anchor[abase + j];
            if (t > i) {
                atomicOr(c.status, kStatusBadIndex);
            } else if (t >= 0) {
                const long long a = t - (long long)c.back * ell, z = t + (long long)c.fwd * ell;
                lo = (int)(a > 0 ? a : 0);
                hi = (int)(z < i ? z : i);
            }
        }
        s_lo[warp][j] = lo;
        s_hi[warp][j] = hi;
    }
    __syncwarp();

    const T *qrow = q + id.b * c.q_sb + id.h * c.q_sh + id.r * c.q_st;
    const T *kbase = k + id.b * c.kv_sb + id.g * c.kv_sh;
    const T *vbase = v + id.b * c.kv_sb + id.g * c.kv_sh;
    const int sub = lane % LPR, rsel = lane / LPR;
    float qv[E];
    Vec16<T>::load(qrow + sub * E, qv);
    const float scale2 = c.softmax_scale * kLog2e;
#pragma unroll
    for (int e = 0; e < E; ++e) qv[e] *= scale2;
    T *orow = out + id.b * c.q_sb + id.h * c.q_sh + id.r * c.q_st + sub * E;
    float m, l, acc[E];

    if (c.mode == SLA_UNION) {
        // 2. rank sort by (lo, hi, index)
        for (int j = lane; j < n_iv; j += 32) {
            const int lo = s_lo[warp][j], hi = s_hi[warp][j];
            int rank = 0;
            for (int x = 0; x < n_iv; ++x) {
                const int lm = s_lo[warp][x], hm = s_hi[warp][x];
                rank += (lm < lo) || (lm == lo && (hm < hi || (hm == hi && x < j)));
            }
            p_lo[warp][rank] = lo;
            p_hi[warp][rank] = hi;
        }
        __syncwarp();
        // 3. clip overlaps: keep only the part of each span to the right of everything before it
        if (lane == 0) {
            int cnt = 0;
            long long next_free = 0;
            for (int a = 0; a < n_iv; ++a) {
                const int lo = p_lo[warp][a], hi = p_hi[warp][a];
                if (hi < 0) break;
                const long long j0 = lo > next_free ? lo : next_free;
                if (j0 <= hi) {
                    s_lo[warp][cnt] = (int)j0;
                    s_hi[warp][cnt] = hi;
                    ++cnt;
                }
                if (hi + 1 > next_free) next_free = (long long)hi + 1;
            }
            p_cnt[warp] = cnt;
        }
        __syncwarp();
        // 4. one online softmax over the pieces
        attend_intervals<T, D, E>(qv, kbase, vbase, c.kv_st, s_lo[warp], s_hi[warp], p_cnt[warp], sub, rsel, m, l, acc);
        if (rsel == 0) {
            const float inv = l > 0.f ? 1.f / l : 0.f;
#pragma unroll
            for (int e = 0; e < E; ++e) orow[e] = from_float<T>(acc[e] * inv);
            if (sub == 0) lse[orow_idx] = l > 0.f ? (m + log2f(l)) * kLn2 : -CUDART_INF_F;
        }
        return;
    }

    // per-span mode: gate weights from the search scores of the selected (valid) anchors
    float smax = -CUDART_INF_F;
    int n_sel = 0;
    for (int j = 0; j < c.top_k; ++j)
        if (s_hi[warp][j] >= 0) {
            smax = fmaxf(smax, score[abase + j]);
            ++n_sel;
        }
    float sden = 0.f;
    for (int j = 0; j < c.top_k; ++j)
        if (s_hi[warp][j] >= 0) sden += expf(score[abase + j] - smax);
    float o[E];
#pragma unroll
    for (int e = 0; e < E; ++e) o[e] = 0.f;
    float lse_first = -CUDART_INF_F;
    bool first = true;
    if (n_sel == 0) {
        if (c.window > 0) {   // Algorithm 1, empty selection: the window alone
            attend_intervals<T, D, E>(qv, kbase, vbase, c.kv_st, &s_lo[warp][c.top_k], &s_hi[warp][c.top_k], 1, sub, rsel, m, l, acc);
            const float inv = l > 0.f ? 1.f / l : 0.f;
#pragma unroll
            for (int e = 0; e < E; ++e) o[e] = acc[e] * inv;
            lse_first = l > 0.f ? (m + log2f(l)) * kLn2 : -CUDART_INF_F;
        }
    }
    for (int j = 0; j < c.top_k; ++j) {
        const bool sel = s_hi[warp][j] >= 0;
        float l_t = -CUDART_INF_F;
        if (sel) {
            // J_t = S_t united with W: the part of S_t left of the window, then the window
            int n = 0;
            if (lane == 0) {
                const int hi_cut = c.window > 0 && s_hi[warp][j] >= w_lo ? w_lo - 1 : s_hi[warp][j];
                int cnt = 0;
                if (s_lo[warp][j] <= hi_cut) {
                    p_lo[warp][cnt] = s_lo[warp][j];
                    p_hi[warp][cnt] = hi_cut;
                    ++cnt;
                }
                if (c.window > 0) {
                    p_lo[warp][cnt] = w_lo;
                    p_hi[warp][cnt] = (int)i;
                    ++cnt;
                }
                p_cnt[warp] = cnt;
            }
            __syncwarp();
            n = p_cnt[warp];
            attend_intervals<T, D, E>(qv, kbase, vbase, c.kv_st, p_lo[warp], p_hi[warp], n, sub, rsel, m, l, acc);
            __syncwarp();
            const float alpha = expf(score[abase + j] - smax) / sden;
            const float wgt = l > 0.f ? alpha / l : 0.f;
#pragma unroll
            for (int e = 0; e < E; ++e) o[e] = fmaf(wgt, acc[e], o[e]);
            l_t = l > 0.f ? (m + log2f(l)) * kLn2 : -CUDART_INF_F;
            if (first) {
                lse_first = l_t;
                first = false;
            }
        }
        if (lse_span && lane == 0) lse_span[abase + j] = l_t;
    }
    if (rsel == 0) {
#pragma unroll
        for (int e = 0; e < E; ++e) orow[e] = from_float<T>(o[e]);
        if (sub == 0) lse[orow_idx] = lse_first;
    }
}

template <typename T, int D>
cudaError_t search_launch(const void *q_s, const void *k, const Call &c, int32_t *oa, float *os,
                          cudaStream_t st) {
    const long long rows = (long long)c.B * c.Hq * c.Lq;
    const int n_max = n_strides(c, c.q_pos0 + c.Lq - 1) + 1;
    const size_t smem = (size_t)kWarpsPerBlock * n_max * sizeof(float);
    if (smem > 200 * 1024) return cudaErrorInvalidValue;
    auto kern = search_rows_simt<T, D>;
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    const long long blocks = (rows + kWarpsPerBlock - 1) / kWarpsPerBlock;
    kern<<<(unsigned)blocks, kWarpsPerBlock * 32, smem, st>>>((const T *)q_s, (const T *)k, c, oa, os, n_max);
    return cudaGetLastError();
}

template <typename T, int D>
cudaError_t attn_launch(const void *q, const void *k, const void *v, const Call &c, const int32_t *anchor,
                        const float *score, void *out, float *lse, float *lse_span, cudaStream_t st) {
    const long long rows = (long long)c.B * c.Hq * c.Lq;
    const long long blocks = (rows + kWarpsPerBlock - 1) / kWarpsPerBlock;
    attn_rows_simt<T, D><<<(unsigned)blocks, kWarpsPerBlock * 32, 0, st>>>(
        (const T *)q, (const T *)k, (const T *)v, c, anchor, score, (T *)out, lse, lse_span);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_search_simt(const void *q_s, const void *k, const Call &c, int dtype, int32_t *oa,
                               float *os, cudaStream_t st) {
    if (dtype == SLA_F32) {
        return c.D == 64 ? search_launch<float, 64>(q_s, k, c, oa, os, st)
                         : search_launch<float, 128>(q_s, k, c, oa, os, st);
    }
    return c.D == 64 ? search_launch<__nv_bfloat16, 64>(q_s, k, c, oa, os, st)
                     : search_launch<__nv_bfloat16, 128>(q_s, k, c, oa, os, st);
}

cudaError_t launch_attn_simt(const void *q, const void *k, const void *v, const Call &c, int dtype,
                             const int32_t *anchor, const float *score, void *out, float *lse, float *lse_span,
                             cudaStream_t st) {
    if (dtype == SLA_F32) {
        return c.D == 64 ? attn_launch<float, 64>(q, k, v, c, anchor, score, out, lse, lse_span, st)
                         : attn_launch<float, 128>(q, k, v, c, anchor, score, out, lse, lse_span, st);
    }
    return c.D == 64 ? attn_launch<__nv_bfloat16, 64>(q, k, v, c, anchor, score, out, lse, lse_span, st)
                     : attn_launch<__nv_bfloat16, 128>(q, k, v, c, anchor, score, out, lse, lse_span, st);
}

}  // namespace sla
