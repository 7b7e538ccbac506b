// Span-search for bf16, head_dim 128 and groups of four query heads per KV head (Section "Span
// search": s_{i,t} = <Q_s(i), K(t)> over the anchors t_s = i + 1 - offset(s), then TopK), with the
// selection folded into the scoring loop.
//
// The fixed stride pattern makes the keys of one stride contiguous over consecutive queries: query
// i0 + j scores key t0 + j at stride s (Section "Span search": "the fixed stride pattern allows us to
// calculate the search scores in a more efficient manner").  A warp owns four consecutive query
// positions of one (batch, KV head).  Its routing queries -- 4 positions x 4 heads -- are the 16 rows
// of the A operand of an m16n8k16 tensor-core MMA and stay in registers for the whole row of strides;
// the 8 columns of the B operand are the keys of two strides for the four positions, fetched with
// plain 32-byte loads (every key row is needed by exactly one position per stride, so there is
// nothing to share through shared memory; K stays in L2).  Of the 16 x 8 products of an MMA the
// 4 x 4 x 2 diagonal blocks are scores -- exactly one per lane: lane (row group r8, quad index q)
// receives the score of (position 2(q&1) + (r8>>2), head r8&3) at stride s0 + (q>>1).  So every lane
// owns one (position, head) pair on every other stride and keeps that pair's running top-k itself:
//   - the K best values so far, sorted, in registers (a branch-free insertion of two min/max per slot);
//   - every score that beat the K-th best when it arrived is appended with its stride index to the
//     lane's list in shared memory -- the final selection is a subset of that list.  When a list runs
//     full, the warp's lanes drop the entries that have fallen below their K-th best since.
// At the end each lane sorts out the stride indices of its K best, the two lanes of a pair merge their
// lists through shuffles (larger score first, smaller stride index on ties) and write the slots.
// The dims are assigned to the MMA's k slots in a permuted order (identical for A and B, which leaves
// the dot product unchanged) so that each lane loads 32 contiguous bytes of a row and a quad a whole
// 128-byte line.
#include <limits.h>
#include <math_constants.h>

#include "sla_kernels.h"

namespace sla {

namespace {

using bf16 = __nv_bfloat16;
constexpr int kWarps = 8;
constexpr int kQW = 4;   // query positions per warp
constexpr int kG = 4;    // query heads per KV head

template <int K> struct ListCap { static constexpr int value = 2 * K + 8; };

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// 32 bytes per lane in one load: the four lanes of a quad cover a whole 128-byte line of a row, so a warp's
// load touches eight full lines (with 16-byte loads it would touch the same eight lines for half the bytes)
struct Words8 { uint32_t w[8]; };
__device__ __forceinline__ Words8 ldg256(const void *p) {
    Words8 r;
    asm volatile("ld.global.nc.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r.w[0]), "=r"(r.w[1]), "=r"(r.w[2]), "=r"(r.w[3]), "=r"(r.w[4]), "=r"(r.w[5]), "=r"(r.w[6]), "=r"(r.w[7])
                 : "l"(p));
    return r;
}

__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// Descending order of (score, stride): larger score first, smaller stride index on ties.
__device__ __forceinline__ bool beats(float xa, int sa, float xb, int sb) { return xa > xb || (xa == xb && sa < sb); }

// Batcher's odd-even merge sort of K (a power of two) register-resident (score, stride) pairs, best first.
template <int K>
__device__ __forceinline__ void sort_pairs(float (&x)[K], int (&s)[K]) {
#pragma unroll
    for (int p = 1; p < K; p <<= 1)
#pragma unroll
        for (int k = p; k >= 1; k >>= 1)
#pragma unroll
            for (int a = 0; a < K; ++a) {
                // a is the upper element of a comparator (a, a + k) of this stage of the network
                const int j0 = k % p, b = a + k;
                if (a >= j0 && (a - j0) % (2 * k) < k && b < K && a / (2 * p) == b / (2 * p)) {
                    const bool sw = beats(x[b], s[b], x[a], s[a]);
                    const float xa = sw ? x[b] : x[a], xb = sw ? x[a] : x[b];
                    const int sa = sw ? s[b] : s[a], sb = sw ? s[a] : s[b];
                    x[a] = xa; x[b] = xb; s[a] = sa; s[b] = sb;
                }
            }
}

template <int K>
__global__ void __launch_bounds__(kWarps * 32, 2)
search_diag(const bf16 *__restrict__ q_s, const bf16 *__restrict__ k, Call c, int32_t *__restrict__ out_anchor,
            float *__restrict__ out_score) {
    constexpr int CAP = ListCap<K>::value;
    extern __shared__ float smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int r8 = lane >> 2, q = lane & 3;
    // the tiles with the most strides (the last positions) start first
    const long long r0 = ((long long)(gridDim.x - 1 - blockIdx.x) * kWarps + warp) * kQW;
    if (r0 >= c.Lq) return;
    const int bg = blockIdx.y, g = bg % c.Hkv, b = bg / c.Hkv;
    float *lx = smem + (size_t)warp * (2 * CAP * 32) + lane;                  // list entry e: lx[32 e], ls[32 e]
    int *ls = reinterpret_cast<int *>(smem + (size_t)warp * (2 * CAP * 32) + CAP * 32) + lane;

    const long long last = c.Lq - 1;
    // ---- A operand: rows r8 and r8 + 8 = (position r8>>2, head r8&3) and (position 2 + (r8>>2), head r8&3)
    Words8 qa[2], qb[2];
    {
        const long long ra = r0 + (r8 >> 2) < last ? r0 + (r8 >> 2) : last;
        const long long rb = r0 + 2 + (r8 >> 2) < last ? r0 + 2 + (r8 >> 2) : last;
        const bf16 *base = q_s + b * c.q_sb + (long long)(g * kG + (r8 & 3)) * c.q_sh + 16 * q;
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            qa[j] = ldg256(base + ra * c.q_st + 64 * j);
            qb[j] = ldg256(base + rb * c.q_st + 64 * j);
        }
    }
    // strides of the warp's positions: one integer square root per warp (quadratic pattern), the other
    // positions have as many strides or one more
    const int i0 = (int)(c.q_pos0 + r0);   // positions fit 31 bits
    const int n0 = n_strides(c, i0);
    auto n_at = [&](int i) -> int {
        if (c.off) return n_strides(c, i);
        return n0 + ((long long)(n0 + 1) * (n0 + 1) <= (long long)i + 1);
    };
    // ---- loader role: column r8 of the B operand = key of position jc at stride s0 + u_ld
    const int jc = r8 & 3, u_ld = r8 >> 2;
    const bool row_ld = r0 + jc <= last;
    const int i_ld = row_ld ? i0 + jc : (int)(c.q_pos0 + last);
    const int n_ld = row_ld ? n_at(i_ld) : 0;
    // ---- owner role: the score this lane receives
    const int jq = ((q & 1) << 1) | (r8 >> 2), hh = r8 & 3, u_own = q >> 1;
    const bool row_own = r0 + jq <= last;
    const int i_own = row_own ? i0 + jq : (int)(c.q_pos0 + last);
    const int n_own = row_own ? n_at(i_own) : 0;
    // Algorithm 1: anchors inside the local window are no candidates; t_s lies in W iff offset(s) <= w
    const int s_min = c.window > 0 ? window_strides(c) : 0;
    const bool full_group = r0 + kQW - 1 <= last;
    const int n_max = full_group ? n_at(i0 + kQW - 1) : n_at((int)(c.q_pos0 + last));
    const int n_all = full_group ? n0 : s_min;   // strides below n_all exist for every position of the warp

    const bf16 *kbase = k + b * c.kv_sb + g * c.kv_sh + 16 * q;
    const int kv_st = (int)c.kv_st;
    auto fetch = [&](int s0, bool check, Words8 (&kb)[2]) {
        const int s = s0 + u_ld;
        int t = i_ld + 1 - stride_offset(c, s < c.n_off || !c.off ? s : 0);
        if (check && s >= n_ld) t = i_ld;   // a valid row either way
        const bf16 *row = kbase + (long long)t * kv_st;
        kb[0] = ldg256(row);
        kb[1] = ldg256(row + 64);
    };

    float v[K];
#pragma unroll
    for (int j = 0; j < K; ++j) v[j] = -CUDART_INF_F;
    int cnt = 0;

    // Drops the list entries that can no longer be among the K best (all lanes, each its own list):
    // what is left are the entries above the K-th best value and the earliest of those equal to it,
    // at most K in all, still in stride order.
    auto compact = [&]() {
        const float vk = v[K - 1];
        int allow_eq = K;
#pragma unroll
        for (int j = 0; j < K; ++j) allow_eq -= v[j] > vk;
        int w = 0;
        for (int e = 0; e < cnt; ++e) {
            const float x = lx[32 * e];
            const int s = ls[32 * e];
            const bool eq = x == vk;
            if (x > vk || (eq && allow_eq > 0)) {
                allow_eq -= eq;
                lx[32 * w] = x;
                ls[32 * w] = s;
                ++w;
            }
        }
        cnt = w;
    };

    // Two new scores at a time.  Each one that beats the K-th best so far goes to the list; the sorted
    // values take both in one pass: with hi >= lo the new j-th best is
    // max(v[j], min(v[j-1], hi), min(v[j-2], lo)).
    auto offer2 = [&](int sa, float xa, int sb, float xb) {
        const float vk = v[K - 1];
        if (xa > vk) {
            lx[32 * cnt] = xa;
            ls[32 * cnt] = sa;
            ++cnt;
        }
        if (xb > vk) {
            lx[32 * cnt] = xb;
            ls[32 * cnt] = sb;
            ++cnt;
        }
        const float hi = fmaxf(xa, xb), lo = fminf(xa, xb);
#pragma unroll
        for (int j = K - 1; j >= 2; --j) v[j] = max3(v[j], fminf(v[j - 1], hi), fminf(v[j - 2], lo));
        if (K >= 2) v[1] = max3(v[1], fminf(v[0], hi), lo);
        v[0] = fmaxf(v[0], hi);
    };
    // scores of one B tile (two strides): two independent accumulation chains, added at the end
    auto score = [&](const Words8 (&kb)[2]) -> float {
        float a0[4] = {0.f, 0.f, 0.f, 0.f}, a1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int x = 0; x < 4; ++x) {
            mma_bf16_16816(a0, qa[0].w[2 * x], qb[0].w[2 * x], qa[0].w[2 * x + 1], qb[0].w[2 * x + 1], kb[0].w[2 * x], kb[0].w[2 * x + 1]);
            mma_bf16_16816(a1, qa[1].w[2 * x], qb[1].w[2 * x], qa[1].w[2 * x + 1], qb[1].w[2 * x + 1], kb[1].w[2 * x], kb[1].w[2 * x + 1]);
        }
        // the one score of this lane: row r8 (positions 0, 1) or r8 + 8 (positions 2, 3), column 2q + (r8>>2)
        const float lo = (r8 >> 2) ? a0[1] + a1[1] : a0[0] + a1[0], hi = (r8 >> 2) ? a0[3] + a1[3] : a0[2] + a1[2];
        return ((q & 1) ? hi : lo) * c.search_scale;
    };
    // four strides (two B tiles): eight 16-byte loads in flight per lane, then two scores per lane
    auto step = [&](int s0, bool check) {
        Words8 ka[2], kb[2];
        fetch(s0, check, ka);
        fetch(s0 + 2, check, kb);
        float xa = score(ka), xb = score(kb);
        if (check) {
            xa = s0 + u_own < n_own ? xa : -CUDART_INF_F;
            xb = s0 + 2 + u_own < n_own ? xb : -CUDART_INF_F;
        }
        if (__any_sync(0xffffffffu, cnt >= CAP - 1)) compact();   // room for both scores
        offer2(s0 + u_own, xa, s0 + 2 + u_own, xb);
    };
    int s0 = s_min;
    for (; s0 + 4 <= n_all; s0 += 4) step(s0, false);
    for (; s0 < n_max; s0 += 4) step(s0, true);

    // ---- the lane's K best with their stride indices, sorted; then the merge with the lane that holds
    // the pair's other strides (q differs in bit 1): the rank of an entry in the union is its rank here
    // plus the number of the partner's entries that come before it
    compact();
    float ex[K];
    int es[K];
#pragma unroll
    for (int j = 0; j < K; ++j) {
        const bool on = j < cnt;
        ex[j] = on ? lx[32 * j] : -CUDART_INF_F;
        es[j] = on ? ls[32 * j] : INT_MAX;
    }
    sort_pairs<K>(ex, es);
    int rank[K];
#pragma unroll
    for (int j = 0; j < K; ++j) rank[j] = j;
#pragma unroll
    for (int e = 0; e < K; ++e) {
        const float pv = __shfl_xor_sync(0xffffffffu, ex[e], 2);
        const int ps = __shfl_xor_sync(0xffffffffu, es[e], 2);
#pragma unroll
        for (int j = 0; j < K; ++j) rank[j] += beats(pv, ps, ex[j], es[j]);
    }
    const int n_pair = cnt + __shfl_xor_sync(0xffffffffu, cnt, 2);
    if (!row_own) return;
    const long long obase = ((((long long)b * c.Hq + g * kG + hh) * c.Lq) + r0 + jq) * c.top_k;
#pragma unroll
    for (int j = 0; j < K; ++j)
        if (j < cnt && rank[j] < c.top_k) {
            out_anchor[obase + rank[j]] = i_own + 1 - stride_offset(c, es[j]);
            out_score[obase + rank[j]] = ex[j];
        }
    if (u_own == 0)   // fewer candidates than slots: pad
        for (int j = n_pair; j < c.top_k; ++j) {
            out_anchor[obase + j] = -1;
            out_score[obase + j] = -CUDART_INF_F;
        }
}

template <int K>
cudaError_t launch_k(const bf16 *q_s, const bf16 *k, const Call &c, int32_t *oa, float *os, cudaStream_t st) {
    constexpr size_t smem = (size_t)kWarps * 2 * ListCap<K>::value * 32 * sizeof(float);
    static bool attr_set[64] = {};
    if (smem > 48 * 1024) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess) return cudaErrorInvalidDevice;
        if (dev < 0 || dev >= 64 || !attr_set[dev]) {
            cudaError_t e = cudaFuncSetAttribute(search_diag<K>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return e;
            if (dev >= 0 && dev < 64) attr_set[dev] = true;
        }
    }
    const dim3 blocks((unsigned)((c.Lq + kWarps * kQW - 1) / (kWarps * kQW)), (unsigned)(c.B * c.Hkv));
    search_diag<K><<<blocks, kWarps * 32, smem, st>>>(q_s, k, c, oa, os);
    return cudaGetLastError();
}

}  // namespace

bool search_diag_supported(const Call &c, int dtype) {
    // (the 32-byte loads want 32-byte aligned rows: strides in multiples of 16 elements)
    return dtype == SLA_BF16 && c.D == 128 && c.G == kG && c.top_k <= 16 && (long long)c.B * c.Hkv <= 65535 &&
           c.kv_st <= INT_MAX && c.q_pos0 + c.Lq <= INT_MAX &&
           (c.q_sb | c.q_sh | c.q_st | c.kv_sb | c.kv_sh | c.kv_st) % 16 == 0;
}

cudaError_t launch_search_diag(const void *q_s, const void *k, const Call &c, int32_t *oa, float *os, cudaStream_t st,
                               long long *launches) {
    const bf16 *qs = (const bf16 *)q_s, *kk = (const bf16 *)k;
    cudaError_t e;
    if (c.top_k <= 2) e = launch_k<2>(qs, kk, c, oa, os, st);
    else if (c.top_k <= 4) e = launch_k<4>(qs, kk, c, oa, os, st);
    else if (c.top_k <= 8) e = launch_k<8>(qs, kk, c, oa, os, st);
    else e = launch_k<16>(qs, kk, c, oa, os, st);
    if (launches) *launches += 1;
    return e;
}

}  // namespace sla
