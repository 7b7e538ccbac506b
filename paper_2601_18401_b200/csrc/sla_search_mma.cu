// Span-search for bf16, head_dim 128 (Section "Span search": s_{i,t} = <Q_s(i), K(t)> over the
// anchors t_s = i + 1 - (s+1)^2, then TopK).
//
// One warp owns one (batch, KV head, query position) and scores the anchors for all G query heads
// of the group at once: 16 anchors x 128 dims of gathered K rows are the A operand of eight
// m16n8k16 tensor-core MMAs, the group's routing queries (up to 8 heads) are the B operand, so every
// K row is fetched once per group.  The work is a skinny gathered product (N = G <= 8) bound by the
// L2 -> SM traffic of the key rows, not a dense contraction, which is why it runs on register-level
// MMAs fed by plain 16-byte loads and not on tcgen05 tiles.  The dims are assigned to the MMA's k
// slots in a permuted order (identical for A and B, which leaves the dot product unchanged) so that
// each lane loads 16 contiguous bytes of a row.
//
// Scores go to shared memory; the k best of each head are then selected with warp votes, the heads
// of the warp side by side (a group of lanes per head): a threshold from the lanes' best scores,
// compaction of the candidates at or above it, and the rank of every candidate among them (largest
// score first, smaller stride index on ties) as its output slot.
#include <limits.h>
#include <math_constants.h>

#include "sla_kernels.h"
#include "sla_topk.cuh"

namespace sla {

namespace {

using bf16 = __nv_bfloat16;
constexpr int kWarps = 8;
using topk::kCap;
using topk::select_topk;
constexpr int kCand = 2 * 4 * topk::kCapG;   // candidate keys and stride indices: 4 heads x kCapG, or 2 x kCap

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__global__ void __launch_bounds__(kWarps * 32)
search_mma(const bf16 *__restrict__ q_s, const bf16 *__restrict__ k, Call c, int32_t *__restrict__ out_anchor,
           float *__restrict__ out_score, int n_max, int head0, int heads) {
    extern __shared__ float smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // grid: x = groups of kWarps query positions, y = batch * Hkv + kv head (no 64-bit divisions here)
    const long long r = (long long)blockIdx.x * kWarps + warp;
    if (r >= c.Lq) return;
    const int bg = blockIdx.y, g = bg % c.Hkv, b = bg / c.Hkv;
    const long long i = c.q_pos0 + r;
    const int n = n_strides(c, i);
    // Algorithm 1: anchors inside the local window are no candidates; t_s lies in W iff (s+1)^2 <= w
    const int s_min = window_strides(c);
    float *sc = smem + (size_t)warp * (heads * n_max + kCand);
    float *cand_v = sc + heads * n_max;
    int *cand_s = reinterpret_cast<int *>(cand_v + kCap);

    const int r8 = lane >> 2, q = lane & 3;
    // B operand: routing queries of heads head0 .. head0+heads-1 of the group (column r8 of the MMA)
    uint32_t bq[4][4];
    {
        const bool hv = r8 < heads;
        const bf16 *qrow = q_s + b * c.q_sb + (long long)(g * c.G + head0 + (hv ? r8 : 0)) * c.q_sh + r * c.q_st;
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) {
            uint4 v = make_uint4(0, 0, 0, 0);
            if (hv) v = __ldg(reinterpret_cast<const uint4 *>(qrow + 32 * ch + 8 * q));
            bq[ch][0] = v.x; bq[ch][1] = v.y; bq[ch][2] = v.z; bq[ch][3] = v.w;
        }
    }
    const bf16 *kbase = k + b * c.kv_sb + g * c.kv_sh + 8 * q;
    const int kv_st = (int)c.kv_st, i32 = (int)i;   // positions and the token stride fit 31 bits: 32x32->64 products
    for (int a0 = s_min; a0 < n; a0 += 16) {
        const int s0 = a0 + r8, s1 = s0 + 8;
        const int t0 = s0 < n ? i32 + 1 - stride_offset(c, s0) : i32;
        const int t1 = s1 < n ? i32 + 1 - stride_offset(c, s1) : i32;
        const bf16 *row0 = kbase + (long long)t0 * kv_st, *row1 = kbase + (long long)t1 * kv_st;
        uint4 ra[4], rb[4];
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) {
            ra[ch] = __ldg(reinterpret_cast<const uint4 *>(row0 + 32 * ch));
            rb[ch] = __ldg(reinterpret_cast<const uint4 *>(row1 + 32 * ch));
        }
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) {
            mma_bf16_16816(acc, ra[ch].x, rb[ch].x, ra[ch].y, rb[ch].y, bq[ch][0], bq[ch][1]);
            mma_bf16_16816(acc, ra[ch].z, rb[ch].z, ra[ch].w, rb[ch].w, bq[ch][2], bq[ch][3]);
        }
        // acc[0],acc[1]: anchor s0, heads 2q, 2q+1;  acc[2],acc[3]: anchor s1
        if (2 * q < heads) {
            if (s0 < n) sc[(2 * q) * n_max + s0 - s_min] = acc[0] * c.search_scale;
            if (s1 < n) sc[(2 * q) * n_max + s1 - s_min] = acc[2] * c.search_scale;
        }
        if (2 * q + 1 < heads) {
            if (s0 < n) sc[(2 * q + 1) * n_max + s0 - s_min] = acc[1] * c.search_scale;
            if (s1 < n) sc[(2 * q + 1) * n_max + s1 - s_min] = acc[3] * c.search_scale;
        }
    }
    __syncwarp();
    const int n_cand = n > s_min ? n - s_min : 0;
    {
        // all heads of the warp at once, a group of lanes per head, when their number and top_k allow it
        const long long obase0 = ((((long long)b * c.Hq + g * c.G + head0) * c.Lq) + r) * c.top_k;
        const long long hstride = c.Lq * c.top_k;
        uint32_t *ck = reinterpret_cast<uint32_t *>(cand_v);
        int *cs = reinterpret_cast<int *>(cand_v) + 4 * topk::kCapG;
        bool done = false;
        if (heads == 4 && c.top_k <= 8)
            done = topk::select_topk_grouped<4, 2>(sc, n_max, n_cand, c.top_k, i, ck, cs, out_anchor + obase0,
                                                   out_score + obase0, hstride, lane, s_min, c.off);
        else if (heads == 4 && c.top_k <= 16)
            done = topk::select_topk_grouped<4, 4>(sc, n_max, n_cand, c.top_k, i, ck, cs, out_anchor + obase0,
                                                   out_score + obase0, hstride, lane, s_min, c.off);
        else if (heads == 2 && c.top_k <= 16)
            done = topk::select_topk_grouped<2, 2>(sc, n_max, n_cand, c.top_k, i, ck, cs, out_anchor + obase0,
                                                   out_score + obase0, hstride, lane, s_min, c.off);
        if (done) return;
    }
    for (int hh = 0; hh < heads; ++hh) {
        const int h = g * c.G + head0 + hh;
        const long long obase = ((((long long)b * c.Hq + h) * c.Lq) + r) * c.top_k;
        select_topk(sc + hh * n_max, n_cand, c.top_k, i, cand_v, cand_s, out_anchor + obase, out_score + obase, lane,
                    s_min, c.off);
    }
}

}  // namespace

bool search_mma_supported(const Call &c, int dtype) {
    if (dtype != SLA_BF16 || c.D != 128 || (long long)c.B * c.Hkv > 65535 || c.kv_st > INT_MAX) return false;
    const int n_max = n_strides(c, c.q_pos0 + c.Lq - 1) + 1;
    const int heads = c.G < 8 ? c.G : 8;
    return (size_t)kWarps * (heads * n_max + kCand) * sizeof(float) <= 200 * 1024;
}

cudaError_t launch_search_mma(const void *q_s, const void *k, const Call &c, int32_t *oa, float *os, cudaStream_t st,
                              long long *launches) {
    const int n_max = n_strides(c, c.q_pos0 + c.Lq - 1) + 1;
    const dim3 blocks((unsigned)((c.Lq + kWarps - 1) / kWarps), (unsigned)(c.B * c.Hkv));
    for (int head0 = 0; head0 < c.G; head0 += 8) {
        const int heads = c.G - head0 < 8 ? c.G - head0 : 8;
        const size_t smem = (size_t)kWarps * (heads * n_max + kCand) * sizeof(float);
        if (smem > 48 * 1024) {
            cudaError_t e = cudaFuncSetAttribute(search_mma, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return e;
        }
        search_mma<<<blocks, kWarps * 32, smem, st>>>((const bf16 *)q_s, (const bf16 *)k, c, oa, os, n_max, head0, heads);
        if (launches) *launches += 1;
    }
    return cudaGetLastError();
}

}  // namespace sla
