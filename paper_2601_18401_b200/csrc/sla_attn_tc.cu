// Tensor-core span-attention for prefill (bf16, head_dim 128): tcgen05 MMA with TMEM accumulators,
// K/V tiles by TMA, one softmax thread per query row.
//
// What it computes is Section "Span attention" (A_{i,t} = Attention(Q(i), K[S_t], V[S_t])) with the
// spans of Algorithm 1.  Union mode: the k spans of a (query, head) row (and its local window) are
// sorted and clipped to disjoint "pieces"; every piece is attended on its own and the per-piece
// results are merged exactly through their log-sum-exp.  Per-span mode (Algorithm 1 literally): the
// pieces are the spans themselves (the part left of the window) plus the window once per row; the
// merge forms every A_t from its span piece and the window piece and applies the gate of Section
// "Combination".
//
// The systems problem (Section "Kernel design"): neighbouring queries pick different spans, so the
// rows of one MMA tile must be made to share a key footprint.  Here pieces are grouped by the
// 64-key block their right end falls in (per batch and KV head) and, inside a group, ordered by how
// many key blocks they cover, with one counting sort (histogram, prefix sum, scatter) -- no
// comparison sort of the queries.  A tile is 128 consecutive pieces of the sorted list (of one group,
// or of neighbouring groups whose end blocks lie next to each other): their Q rows are gathered into
// shared memory and the tile walks the key blocks they cover from left to right.
//
//   tc::prepare          the counting sort and the tile table (sla_attn_prep.cu)
//   tc_attend            persistent CTAs, tile t goes to CTA t mod grid (the table is static once
//                        built); per tile and key block: S = Q K^T (tcgen05, smem x smem -> TMEM), row
//                        softmax in registers, P (bf16) back into TMEM, O += P V (tcgen05, TMEM x smem
//                        -> TMEM); per piece a normalised fp16 block-floating-point partial + lse
//   tc_merge             per row: log-sum-exp merge of its pieces -> out, lse
//   tc_merge_gated       per row: A_t = merge(span piece, window piece), O = sum_t alpha_t A_t
//
// CTA layout of tc_attend (192 threads, two CTAs per SM): warps 0-3 own one tile row each (TMEM lane
// = row): Q gather, softmax, epilogue; one thread of warp 4 issues the MMAs; one thread of warp 5
// issues the TMA loads (K and V as two independent streams).  TMEM: two 64-column S buffers (P aliases
// the S it came from) and 128 columns of O.  Every wait on an mbarrier is bounded; when one runs out
// the CTA raises a status bit, drains and leaves.  The kernel is sensitive to its code size (loops
// over rarely taken paths stay rolled, the spin loops of the waits are not unrolled).
#include <cuda.h>
#include <cudaTypedefs.h>
#include <cuda_fp16.h>
#include <limits.h>
#include <math_constants.h>

#include "sla_attn_tc.cuh"
#include "sla_tc_ptx.cuh"

namespace sla {

namespace {

using bf16 = __nv_bfloat16;

constexpr int kD = 128;
using tc::kBK;    // keys per block
using tc::kRows;  // pieces per tile
constexpr int kThreads = 192;   // 4 row warps, MMA issuer, TMA producer
constexpr int kTmemCols = 256;
constexpr int kMaxWalk = 4096;   // most key blocks a tile walks
constexpr uint32_t kColS = 0;    // S buffers at columns 0 and 64
constexpr uint32_t kColO = 128;
constexpr int kQBytes = kRows * kD * 2;      // 32 KiB, two 64-wide halves of 128 rows x 128 B
constexpr int kKVBytes = kBK * kD * 2;       // 16 KiB, two 64-wide halves of 64 rows x 128 B
constexpr int kKS = 3;           // K stages (a K block is free again as soon as its S = Q K^T is done)
constexpr int kVS = 2;           // V stages (and S/P buffers)
constexpr int kOffQ = 0;
constexpr int kOffK = kQBytes;
constexpr int kOffV = kOffK + kKS * kKVBytes;
constexpr int kOffMeta = kOffV + kVS * kKVBytes;   // 114688
constexpr int kMetaBytes = 1024;
// 113 KiB: two CTAs (plus 1 KiB of system reserve each) fill the 228 KiB of an SM exactly
constexpr int kSmemBytes = kOffMeta + kMetaBytes;
constexpr float kRescaleThreshold = 8.f;     // log2 units: P stays below 2^8

struct Meta {
    unsigned long long q_full, o_full, o_empty;
    unsigned long long k_full[kKS], k_empty[kKS], v_full[kVS], v_empty[kVS], s_full[2], p_ready[2];
    uint32_t tmem_base;
    int abort_flag;
};
static_assert(sizeof(Meta) <= kMetaBytes, "meta block too large");

struct TcParams {
    const bf16 *q;
    long long q_sb, q_sh, q_st;
    int Hq, G, Lc, slots;      // slots: partial results per row (top_k, + 1 with a local window)
    long long r0;              // first query row of the chunk
    float scale2;              // softmax_scale * log2(e)
    int slot_t, slot_h, slot_b;  // positions of (token, head, batch) among tensor-map coordinates 1..3
    const int4 *recs;          // sorted piece records {row, j, lo, hi}
    const int4 *tiles;         // {b*Hkv+g, end block, first record, record count | key blocks to walk << 8}
    const int *n_tiles;
    __half *part_o;            // [rows*slots][128] normalised piece outputs, fp16 with one power-of-two
                               // scale per 32-column chunk (block floating point)
    float2 *part_lse;          // [rows*slots] {log2-domain log-sum-exp of the piece, four chunk exponents}
    int *status;
    int Hkv;
};

// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
// packed fp32x2 arithmetic (two independent fp32 lanes per instruction)
__device__ __forceinline__ unsigned long long pack2(float a, float b) {
    unsigned long long r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
    return r;
}
__device__ __forceinline__ void unpack2(unsigned long long r, float &a, float &b) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(r));
}
__device__ __forceinline__ unsigned long long ffma2(unsigned long long a, unsigned long long b, unsigned long long c) {
    unsigned long long d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ unsigned long long fadd2(unsigned long long a, unsigned long long b) {
    unsigned long long d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
// A shared-memory matrix descriptor moved forward by `bytes` (the start address sits in the low word
// in units of 16 bytes, and the window is far below the field's range, so no carry leaves it).
__device__ __forceinline__ uint64_t desc_advance(uint64_t desc, uint32_t bytes) {
    uint32_t lo, hi;
    asm("mov.b64 {%0, %1}, %2;" : "=r"(lo), "=r"(hi) : "l"(desc));
    lo += bytes >> 4;
    asm("mov.b64 %0, {%1, %2};" : "=l"(desc) : "r"(lo), "r"(hi));
    return desc;
}
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Gathers one Q row (256 B) into the swizzled A-operand layout with 16-byte async copies; a null
// source zero-fills the row.  Kept out of line: it runs once per tile from two places, and the
// kernel's hot loop is faster the less code surrounds it.
__device__ __noinline__ void gather_q_row(const bf16 *src, uint8_t *q_tile, uint32_t q_row, int tid) {
    if (src) {
#pragma unroll
        for (int cidx = 0; cidx < 16; ++cidx) {
            const uint32_t dst = q_row + (cidx >> 3) * (kQBytes / 2) + (((cidx & 7) ^ (tid & 7)) << 4);
            ptx::cp_async16(dst, src + cidx * 8);
        }
    } else {
        uint4 *qdst = reinterpret_cast<uint4 *>(q_tile);
#pragma unroll
        for (int cidx = 0; cidx < 16; ++cidx)
            qdst[(cidx >> 3) * (kQBytes / 32) + tid * 8 + (cidx & 7)] = make_uint4(0, 0, 0, 0);
    }
}

__global__ void __launch_bounds__(kThreads, 2)
tc_attend(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v, TcParams p) {
    extern __shared__ __align__(1024) uint8_t smem[];
    const uint32_t base = ptx::smem_u32(smem);
    Meta *meta = reinterpret_cast<Meta *>(smem + kOffMeta);
    volatile int *abort_flag = &meta->abort_flag;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (base & 1023u) {   // the swizzled tiles need a 1024-byte aligned window: refuse rather than corrupt
        if (tid == 0) atomicOr(p.status, kStatusTimeout);
        return;
    }

    const uint32_t bar_q_full = ptx::smem_u32(&meta->q_full), bar_o_full = ptx::smem_u32(&meta->o_full);
    const uint32_t bar_o_empty = ptx::smem_u32(&meta->o_empty);
    const uint32_t bar_k_full = ptx::smem_u32(&meta->k_full[0]), bar_k_empty = ptx::smem_u32(&meta->k_empty[0]);
    const uint32_t bar_v_full = ptx::smem_u32(&meta->v_full[0]), bar_v_empty = ptx::smem_u32(&meta->v_empty[0]);
    const uint32_t bar_s_full = ptx::smem_u32(&meta->s_full[0]), bar_p_ready = ptx::smem_u32(&meta->p_ready[0]);

    if (tid == 0) {
        ptx::mbar_init(bar_q_full, 4);   // one arrival per row warp
        ptx::mbar_init(bar_o_full, 1);
        ptx::mbar_init(bar_o_empty, 4);
        for (int s = 0; s < kKS; ++s) {
            ptx::mbar_init(bar_k_full + 8 * s, 1);
            ptx::mbar_init(bar_k_empty + 8 * s, 1);
        }
        for (int s = 0; s < 2; ++s) {
            ptx::mbar_init(bar_v_full + 8 * s, 1);
            ptx::mbar_init(bar_v_empty + 8 * s, 1);
            ptx::mbar_init(bar_s_full + 8 * s, 1);
            ptx::mbar_init(bar_p_ready + 8 * s, 4);
        }
        meta->abort_flag = 0;
        ptx::fence_barrier_init();
    }
    if (warp == 5 && lane == 0) {
        ptx::prefetch_tensormap(&tm_k);
        ptx::prefetch_tensormap(&tm_v);
    }
    if (warp == 4) {
        ptx::tmem_alloc(ptx::smem_u32(&meta->tmem_base), kTmemCols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem = meta->tmem_base;

    constexpr uint32_t kIdescS = ptx::idesc_bf16_f32(kRows, kBK, false, false);   // S = Q K^T, both K-major
    constexpr uint32_t kIdescO = ptx::idesc_bf16_f32(kRows, kD, false, true);     // O = P V, V is N-major

    // Tiles are dealt round-robin: CTA c takes tiles c, c + grid, c + 2 grid, ...  Every role reads its
    // tile's table entry {b*Hkv+g, end block, first record, count | blocks << 8} straight from global
    // memory, one tile ahead of where it is working, so nothing but mbarriers couples the roles.
    const int n_tiles = *p.n_tiles;
    const int tile_step = gridDim.x;

    if (warp == 5 && lane == 0) {
        // ---------------- TMA producer, event driven: the K blocks and the V blocks of the CTA's tile
        // sequence are two independent streams, each running as far ahead as its own stages allow (a
        // K stage frees when its S = Q K^T is done, long before the V stage of the same block).
        struct Cursor {
            int tile, j, nblk, sb0, ch, cb;
            uint32_t n;
        };
        auto open_tile = [&](Cursor &cu) {
            if (cu.tile < n_tiles) {
                const int4 ti = p.tiles[cu.tile];
                cu.nblk = ti.w >> 8;
                cu.sb0 = ti.y - cu.nblk + 1;
                cu.ch = ti.x % p.Hkv;
                cu.cb = ti.x / p.Hkv;
                cu.j = 0;
            }
        };
        auto issue = [&](Cursor &cu, const CUtensorMap *tm, uint32_t bar_full, uint32_t dst) {
            int c[4];
            c[1 + p.slot_h] = cu.ch;
            c[1 + p.slot_b] = cu.cb;
            c[1 + p.slot_t] = (cu.sb0 + cu.j) * kBK;
            ptx::mbar_arrive_expect_tx(bar_full, kKVBytes);
            ptx::tma_load_4d(dst, tm, bar_full, 0, c[1], c[2], c[3]);
            ptx::tma_load_4d(dst + kKVBytes / 2, tm, bar_full, 64, c[1], c[2], c[3]);
            ++cu.n;
            if (++cu.j == cu.nblk) {
                cu.tile += tile_step;
                open_tile(cu);
            }
        };
        Cursor ck{(int)blockIdx.x, 0, 0, 0, 0, 0, 0u}, cv{(int)blockIdx.x, 0, 0, 0, 0, 0, 0u};
        open_tile(ck);
        cv = ck;
        uint32_t idle = 0;
        while (cv.tile < n_tiles) {
            bool progressed = false;
            if (ck.tile < n_tiles) {
                const uint32_t st = ck.n % kKS;
                if (ptx::mbar_test_wait(bar_k_empty + 8 * st, ((ck.n / kKS) & 1u) ^ 1u)) {
                    issue(ck, &tm_k, bar_k_full + 8 * st, base + kOffK + st * kKVBytes);
                    progressed = true;
                }
            }
            {
                const uint32_t st = cv.n % kVS;
                if (cv.n < ck.n &&   // K first: V(n) is never requested before K(n)
                    ptx::mbar_test_wait(bar_v_empty + 8 * st, ((cv.n / kVS) & 1u) ^ 1u)) {
                    issue(cv, &tm_v, bar_v_full + 8 * st, base + kOffV + st * kKVBytes);
                    progressed = true;
                }
            }
            if (progressed) {
                idle = 0;
            } else if (__nanosleep(40), ++idle > ptx::kSpinLimit || ((idle & 63u) == 0u && *abort_flag)) {
                *abort_flag = 1;
                break;
            }
        }
    } else if (warp == 4 && lane == 0) {
        // ---------------- MMA issuer, event driven: S(j) as soon as K(j) has landed and an S buffer
        // is free, PV(j) as soon as P(j) and V(j) are there.  S(j+2) reuses the buffer of P(j), so it
        // is only issued after PV(j); the first PV of a tile overwrites O, so it waits until the row
        // threads have read the previous tile's O.
        uint32_t n_kv = 0, T = 0;
        int tile = blockIdx.x;
        int nblk = tile < n_tiles ? (p.tiles[tile].w >> 8) : 0;
        const uint64_t desc_q0 = ptx::smem_desc_sw128(base + kOffQ, 16, 1024);
        const uint64_t desc_k0 = ptx::smem_desc_sw128(base + kOffK, 16, 1024);
        const uint64_t desc_v0 = ptx::smem_desc_sw128(base + kOffV, kKVBytes / 2, 1024);
        for (; tile < n_tiles; tile += tile_step, ++T) {
            const int nblk_next = tile + tile_step < n_tiles ? (p.tiles[tile + tile_step].w >> 8) : 0;
            bool ok = ptx::mbar_wait(bar_q_full, T & 1u, abort_flag);
            ptx::tc_fence_after();
            int is = 0, ipv = 0;
            uint32_t idle = 0;
            while (ok && ipv < nblk) {
                bool progressed = false;
                if (is < nblk && is < ipv + 2) {
                    const uint32_t n = n_kv + is, ks = n % kKS, sbuf = n & 1u;
                    if (ptx::mbar_test_wait(bar_k_full + 8 * ks, (n / kKS) & 1u)) {
                        ptx::tc_fence_after();
                        const uint32_t d_s = tmem + kColS + sbuf * kBK;
                        const uint64_t dk = desc_advance(desc_k0, ks * kKVBytes);
#pragma unroll
                        for (int kk = 0; kk < kD / 16; ++kk) {
                            const uint32_t half = kk >> 2, inner = (kk & 3) * 32;
                            ptx::mma_ss(d_s, desc_advance(desc_q0, half * (kQBytes / 2) + inner),
                                        desc_advance(dk, half * (kKVBytes / 2) + inner), kIdescS, kk > 0);
                        }
                        ptx::mma_commit(bar_s_full + 8 * sbuf);
                        ptx::mma_commit(bar_k_empty + 8 * ks);
                        ++is;
                        progressed = true;
                    }
                }
                if (ipv < is) {
                    const uint32_t n = n_kv + ipv, vs = n & 1u, ph = (n >> 1) & 1u;
                    const bool o_free = ipv > 0 || T == 0 || ptx::mbar_test_wait(bar_o_empty, (T - 1u) & 1u);
                    if (o_free && ptx::mbar_test_wait(bar_p_ready + 8 * vs, ph) && ptx::mbar_test_wait(bar_v_full + 8 * vs, ph)) {
                        ptx::tc_fence_after();
                        const uint32_t a_p = tmem + kColS + vs * kBK;   // P aliases S: 64 bf16 = 32 columns
                        const uint64_t dv = desc_advance(desc_v0, vs * kKVBytes);
#pragma unroll
                        for (int kk = 0; kk < kBK / 16; ++kk)
                            ptx::mma_ts(tmem + kColO, a_p + kk * 8, desc_advance(dv, kk * 2048), kIdescO,
                                        (ipv > 0 || kk > 0) ? 1u : 0u);
                        ptx::mma_commit(bar_v_empty + 8 * vs);
                        if (ipv == nblk - 1) ptx::mma_commit(bar_o_full);
                        ++ipv;
                        progressed = true;
                    }
                }
                if (progressed) {
                    idle = 0;
                } else if (__nanosleep(20), ++idle > ptx::kSpinLimit || ((idle & 63u) == 0u && *abort_flag)) {
                    *abort_flag = 1;
                    ok = false;
                }
            }
            if (!ok) break;
            n_kv += nblk;
            nblk = nblk_next;
        }
    } else if (warp < 4) {
        // ---------------- row threads: Q gather, softmax per key block, epilogue
        const uint32_t lane_addr = tmem + (static_cast<uint32_t>(warp * 32) << 16);
        const uint32_t q_row = base + kOffQ + tid * 128;
        auto gather_q = [&](bool row_valid, int row) {
            const bf16 *src = nullptr;
            if (row_valid) {
                const int rc = row % p.Lc, bh = row / p.Lc;
                const int h = bh % p.Hq, bb = bh / p.Hq;
                src = p.q + bb * p.q_sb + h * p.q_sh + (p.r0 + rc) * p.q_st;
            }
            gather_q_row(src, smem + kOffQ, q_row, tid);
        };
        uint32_t n_kv = 0, T = 0;
        int tile = blockIdx.x;
        int4 ti = tile < n_tiles ? p.tiles[tile] : make_int4(0, 0, 0, 0);
        int4 rec = make_int4(0, 0, INT_MAX, -1);
        if (tile < n_tiles) {
            if (tid < (ti.w & 0xff)) rec = p.recs[ti.z + tid];
            gather_q(tid < (ti.w & 0xff), rec.x);
        }
        // hands the gathered Q tile to the MMA issuer
        auto publish_q = [&]() {
            ptx::cp_async_wait_all();
            ptx::fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(bar_q_full);
        };
        if (tile < n_tiles) publish_q();
        for (; tile < n_tiles; tile += tile_step, ++T) {
            const int nblk = ti.w >> 8, sb0 = ti.y - nblk + 1, cnt = ti.w & 0xff;
            const bool valid = tid < cnt;
            // the next tile: its record is fetched now, its Q row during this tile's last key block
            const bool has_next = tile + tile_step < n_tiles;
            const int4 ti_next = has_next ? p.tiles[tile + tile_step] : make_int4(0, 0, 0, 0);
            const int cnt_next = ti_next.w & 0xff;
            int4 rec_next = make_int4(0, 0, INT_MAX, -1);
            if (has_next && tid < cnt_next) rec_next = p.recs[ti_next.z + tid];

            const int lo = rec.z, hi = rec.w;
            float m_ref = -CUDART_INF_F, l = 0.f;
            bool ok = true;
            for (int j = 0; j < nblk && ok; ++j) {
                const uint32_t n = n_kv + j, st = n & 1u, ph = (n >> 1) & 1u;
                ok = ptx::mbar_wait_warp(bar_s_full + 8 * st, ph, abort_flag);
                if (!ok) break;
                ptx::tc_fence_after();
                // S of the last block is done, so nothing reads this tile's Q any more
                if (j == nblk - 1 && has_next) gather_q(tid < cnt_next, rec_next.x);
                const uint32_t s_addr = lane_addr + kColS + st * kBK;
                uint32_t sr[2][32];
                ptx::tmem_ld32(s_addr, sr[0]);
                ptx::tmem_ld32(s_addr + 32, sr[1]);
                ptx::tmem_wait_ld();
                const int k0 = (sb0 + j) * kBK;
                const bool any = valid && k0 <= hi && k0 + kBK - 1 >= lo;
                if (!(any && k0 >= lo && k0 + kBK - 1 <= hi)) {
                    // bit c of the mask: column c of the block lies inside the piece
                    const int ca = lo > k0 ? lo - k0 : 0, cb = hi - k0 < kBK - 1 ? hi - k0 : kBK - 1;
                    const unsigned long long inside = any ? (~0ull >> (63 - (cb - ca))) << ca : 0ull;
                    const uint32_t in2[2] = {static_cast<uint32_t>(inside), static_cast<uint32_t>(inside >> 32)};
#pragma unroll
                    for (int hlf = 0; hlf < 2; ++hlf)
#pragma unroll
                        for (int cc = 0; cc < 32; ++cc)
                            if (!(in2[hlf] & (1u << cc))) sr[hlf][cc] = 0xff800000u;   // -inf
                }
                // block maximum on the raw logits (softmax_scale > 0 on this path), four independent chains
                float bm;
                {
                    float mx[4] = {-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F};
#pragma unroll
                    for (int hlf = 0; hlf < 2; ++hlf)
#pragma unroll
                        for (int cc = 0; cc < 32; cc += 8)
#pragma unroll
                            for (int u = 0; u < 4; ++u)
                                mx[u] = max3(mx[u], __uint_as_float(sr[hlf][cc + 2 * u]), __uint_as_float(sr[hlf][cc + 2 * u + 1]));
                    bm = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) * p.scale2;
                }
                // running reference maximum; O is rescaled only when it moves by more than the threshold
                const bool first = (l == 0.f);   // no key of this row seen so far
                const bool need = !first && (bm > m_ref + kRescaleThreshold);
                if (__any_sync(0xffffffffu, need)) {
                    // PV of the previous block must have landed before O is touched
                    const uint32_t np = n - 1u;
                    ok = ptx::mbar_wait_warp(bar_v_empty + 8 * (np & 1u), (np >> 1) & 1u, abort_flag);
                    if (!ok) break;
                    ptx::tc_fence_after();
                    const float f = need ? ex2_approx(m_ref - bm) : 1.f;
#pragma unroll 1
                    for (int q4 = 0; q4 < 4; ++q4) {
                        uint32_t o[32];
                        ptx::tmem_ld32(lane_addr + kColO + q4 * 32, o);
                        ptx::tmem_wait_ld();
#pragma unroll
                        for (int cc = 0; cc < 32; ++cc) o[cc] = __float_as_uint(__uint_as_float(o[cc]) * f);
                        ptx::tmem_st32(lane_addr + kColO + q4 * 32, o);
                    }
                    if (need) { l *= f; m_ref = bm; }
                }
                if (first && bm > -CUDART_INF_F) m_ref = bm;   // first keys of this row
                uint32_t pk[32];
                {
                    // p = 2^(s*scale - m_ref), two columns per packed fp32x2 instruction; masked columns
                    // hold -inf and give 0 (a row with no key so far has m_ref = -inf: it subtracts 0)
                    const float neg_m = m_ref > -CUDART_INF_F ? -m_ref : 0.f;
                    const unsigned long long sc2 = pack2(p.scale2, p.scale2), nm2 = pack2(neg_m, neg_m);
                    unsigned long long acc2[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) acc2[u] = pack2(0.f, 0.f);
#pragma unroll
                    for (int cc = 0; cc < 32; ++cc) {
                        const int hlf = cc >> 4, c2 = (cc & 15) * 2;
                        const unsigned long long y = ffma2(
                            pack2(__uint_as_float(sr[hlf][c2]), __uint_as_float(sr[hlf][c2 + 1])), sc2, nm2);
                        float y0, y1;
                        unpack2(y, y0, y1);
                        const float p0 = ex2_approx(y0), p1 = ex2_approx(y1);
                        acc2[cc & 3] = fadd2(acc2[cc & 3], pack2(p0, p1));
                        const __nv_bfloat162 pp = __floats2bfloat162_rn(p0, p1);
                        pk[cc] = *reinterpret_cast<const uint32_t *>(&pp);
                    }
                    float s0, s1, s2, s3;
                    unpack2(fadd2(acc2[0], acc2[1]), s0, s1);
                    unpack2(fadd2(acc2[2], acc2[3]), s2, s3);
                    l += (s0 + s1) + (s2 + s3);
                }
                ptx::tmem_st32(s_addr, pk);
                ptx::tmem_wait_st();
                ptx::tc_fence_before();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(bar_p_ready + 8 * st);
            }
            // the next tile's Q rows were requested a block ago: publish them now, so that its first
            // S = Q K^T runs while this tile drains
            if (ok && has_next) publish_q();
            // epilogue: normalised piece output and its log-sum-exp
            if (ok) ok = ptx::mbar_wait_warp(bar_o_full, T & 1u, abort_flag);
            if (!ok) break;
            ptx::tc_fence_after();
            {
                const float inv = l > 0.f ? 1.f / l : 0.f;
                const long long slot = (long long)rec.x * p.slots + rec.y;
                __half *dst = p.part_o + slot * kD;
                uint32_t exps = 0;   // biased exponent of each 32-column chunk's largest magnitude
                // one 32-column chunk: block exponent, fp16 mantissas, two 32-byte stores
                auto emit = [&](uint32_t (&o)[32], int q4) {
                    if (valid) {
                        float amax = 0.f;
#pragma unroll
                        for (int cc = 0; cc < 32; ++cc) {
                            const float x = __uint_as_float(o[cc]) * inv;
                            o[cc] = __float_as_uint(x);
                            amax = fmaxf(amax, fabsf(x));
                        }
                        uint32_t eb = (__float_as_uint(amax) >> 23) & 0xffu;
                        eb = eb < 1u ? 1u : (eb > 252u ? 252u : eb);
                        exps |= eb << (8 * q4);
                        const float down = __uint_as_float((253u - eb) << 23);   // 2^(126 - eb): chunk into [-1, 1]
#pragma unroll
                        for (int s8 = 0; s8 < 2; ++s8) {
                            uint32_t w[8];
#pragma unroll
                            for (int e = 0; e < 8; ++e) {
                                const __half2 pp = __floats2half2_rn(__uint_as_float(o[s8 * 16 + 2 * e]) * down,
                                                                     __uint_as_float(o[s8 * 16 + 2 * e + 1]) * down);
                                w[e] = *reinterpret_cast<const uint32_t *>(&pp);
                            }
                            ptx::st_global_v8(dst + q4 * 32 + s8 * 16, w);
                        }
                    }
                };
                // the TMEM read of the next chunk is in flight while this one is converted and stored
                uint32_t oa[32], ob[32];
                ptx::tmem_ld32(lane_addr + kColO, oa);
                ptx::tmem_wait_ld();
                ptx::tmem_ld32(lane_addr + kColO + 32, ob);
                emit(oa, 0);
                ptx::tmem_wait_ld();
                ptx::tmem_ld32(lane_addr + kColO + 64, oa);
                emit(ob, 1);
                ptx::tmem_wait_ld();
                ptx::tmem_ld32(lane_addr + kColO + 96, ob);
                emit(oa, 2);
                ptx::tmem_wait_ld();
                // O is in registers: the next tile's first PV may overwrite it
                ptx::tc_fence_before();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(bar_o_empty);
                emit(ob, 3);
                if (valid)
                    p.part_lse[slot] = make_float2(l > 0.f ? m_ref + log2f(l) : -CUDART_INF_F, __uint_as_float(exps));
            }
            n_kv += nblk;
            rec = rec_next;
            ti = ti_next;
        }
        ptx::cp_async_wait_all();
    }

    // ---- teardown
    __syncthreads();
    if (*abort_flag) {
        if (tid == 0) atomicOr(p.status, kStatusTimeout);
        __nanosleep(200000);   // let copies and MMAs that may still be in flight land
        __syncthreads();
    }
    if (warp == 4) {
        __syncwarp();
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem, kTmemCols);
    }
}

// ------------------------------------------------------------------------------------------------
// Per row: merge the normalised piece outputs through their log-sum-exp.  16 threads per row.
__global__ void __launch_bounds__(256)
tc_merge(const __half *__restrict__ part_o, const float2 *__restrict__ part_lse,
         const unsigned char *__restrict__ n_pieces, Call c, int slots, int Lc, long long r0,
         bf16 *__restrict__ out, float *__restrict__ lse) {
    const long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long row = gid >> 4;
    const int sub = (int)(gid & 15);
    const long long rows = (long long)c.B * c.Hq * Lc;
    if (row >= rows) return;
    const int cnt = n_pieces[row];
    const float2 *pl = part_lse + row * slots;
    const __half *po = part_o + row * slots * kD + sub * 8;
    float acc[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[e] = 0.f;
    // running maximum and denominator (log2 domain); the pieces come four at a time so that their
    // loads are in flight together
    float mx = -CUDART_INF_F, den = 0.f;
    for (int j0 = 0; j0 < cnt; j0 += 4) {
        float2 pj[4];
        uint4 raw[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const bool on = j0 + u < cnt;
            pj[u] = on ? __ldg(pl + j0 + u) : make_float2(-CUDART_INF_F, 0.f);
            raw[u] = on ? __ldg(reinterpret_cast<const uint4 *>(po + (long long)(j0 + u) * kD)) : make_uint4(0, 0, 0, 0);
        }
        float bm = fmaxf(fmaxf(pj[0].x, pj[1].x), fmaxf(pj[2].x, pj[3].x));
        if (bm > mx) {
            const float r = mx == -CUDART_INF_F ? 0.f : exp2f(mx - bm);
            den *= r;
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] *= r;
            mx = bm;
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            if (pj[u].x == -CUDART_INF_F) continue;
            const float w = exp2f(pj[u].x - mx);
            den += w;
            const uint32_t eb = (__float_as_uint(pj[u].y) >> (8 * (sub >> 2))) & 0xffu;
            const float ws = w * __uint_as_float((eb + 1u) << 23);   // weight x 2^(eb - 126)
            const uint32_t rw[4] = {raw[u].x, raw[u].y, raw[u].z, raw[u].w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&rw[e]));
                acc[2 * e] = fmaf(ws, f.x, acc[2 * e]);
                acc[2 * e + 1] = fmaf(ws, f.y, acc[2 * e + 1]);
            }
        }
    }
    const float inv = den > 0.f ? 1.f / den : 0.f;
    const int rc = (int)((unsigned)row % (unsigned)Lc);   // rows < 2^31
    const int bh = (int)((unsigned)row / (unsigned)Lc);
    const int h = bh % c.Hq, b = bh / c.Hq;
    const long long r = r0 + rc;
    uint32_t w[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const __nv_bfloat162 pp = __floats2bfloat162_rn(acc[2 * e] * inv, acc[2 * e + 1] * inv);
        w[e] = *reinterpret_cast<const uint32_t *>(&pp);
    }
    *reinterpret_cast<uint4 *>(out + b * c.q_sb + h * c.q_sh + r * c.q_st + sub * 8) = make_uint4(w[0], w[1], w[2], w[3]);
    if (sub == 0)
        lse[((long long)b * c.Hq + h) * c.Lq + r] = den > 0.f ? (mx + log2f(den)) * kLn2 : -CUDART_INF_F;
}

// Per row, per-span mode (Algorithm 1 with the gate of Section "Combination"): slot j holds the
// attention over the part of S_t left of the window, slot top_k the attention over the window; A_t
// merges the two through their log-sum-exp, and O = sum_t alpha_t A_t with alpha = softmax of the
// selected anchors' search scores.  16 threads per row, 8 columns each.
// dst += w x (eight columns of a piece's block-floating-point output; `exps` holds the chunk exponents)
__device__ __forceinline__ void add_piece(const uint4 &raw, float exps, int sub, float w, float (&dst)[8]) {
    const uint32_t eb = (__float_as_uint(exps) >> (8 * (sub >> 2))) & 0xffu;
    const float ws = w * __uint_as_float((eb + 1u) << 23);   // weight x 2^(eb - 126)
    const uint32_t rw[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&rw[e]));
        dst[2 * e] = fmaf(ws, f.x, dst[2 * e]);
        dst[2 * e + 1] = fmaf(ws, f.y, dst[2 * e + 1]);
    }
}

__global__ void __launch_bounds__(256)
tc_merge_gated(const __half *__restrict__ part_o, const float2 *__restrict__ part_lse,
               const int32_t *__restrict__ anchor, const float *__restrict__ score, Call c, int slots, int Lc,
               long long r0, bf16 *__restrict__ out, float *__restrict__ lse, float *__restrict__ lse_span) {
    const long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long row = gid >> 4;
    const int sub = (int)(gid & 15);
    const long long rows = (long long)c.B * c.Hq * Lc;
    if (row >= rows) return;
    const int rc = (int)((unsigned)row % (unsigned)Lc);   // rows < 2^31
    const int bh = (int)((unsigned)row / (unsigned)Lc);
    const int h = bh % c.Hq, b = bh / c.Hq;
    const long long r = r0 + rc, i = c.q_pos0 + r;
    const long long orow = ((long long)b * c.Hq + h) * c.Lq + r;
    const int32_t *an = anchor + orow * c.top_k;
    const float *sc = score + orow * c.top_k;
    const float2 *pl = part_lse + row * slots;
    const long long ell = base_len(c, i);
    const long long w_lo = i - c.window + 1 > 0 ? i - c.window + 1 : 0;
    const bool has_w = c.window > 0;
    // the window piece is needed by nearly every row: request it with the first loads
    const float2 pw = has_w ? __ldg(pl + c.top_k) : make_float2(-CUDART_INF_F, 0.f);
    const uint4 raw_w = has_w ? __ldg(reinterpret_cast<const uint4 *>(part_o + (row * slots + c.top_k) * kD + sub * 8))
                              : make_uint4(0, 0, 0, 0);
    const float lw = pw.x;

    float smax = -CUDART_INF_F;
    int n_sel = 0;
    for (int j = 0; j < c.top_k; ++j)
        if (an[j] >= 0 && an[j] <= i) { smax = fmaxf(smax, sc[j]); ++n_sel; }
    float sden = 0.f;
    for (int j = 0; j < c.top_k; ++j)
        if (an[j] >= 0 && an[j] <= i) sden += expf(sc[j] - smax);
    float acc[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[e] = 0.f;
    // O = sum_t alpha_t (w_t o_t + ww_t o_W) / den_t: the window piece enters once, with the summed
    // coefficient cw; the spans' pieces come four at a time so that their loads are in flight together
    float lse_first = -CUDART_INF_F, cw = 0.f;
    if (n_sel == 0 && has_w) {   // Algorithm 1, empty selection: the window alone
        cw = 1.f;
        lse_first = lw * kLn2;
    }
    bool first = true;
    const __half *po = part_o + row * slots * kD + sub * 8;
    for (int j0 = 0; j0 < c.top_k; j0 += 4) {
        float2 pj[4];
        uint4 raw[4];
        bool sel[4], has_s[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int j = j0 + u;
            const long long t = j < c.top_k ? an[j] : -1;
            sel[u] = t >= 0 && t <= i;
            const long long a = t - (long long)c.back * ell;
            has_s[u] = sel[u] && (!has_w || (a > 0 ? a : 0) < w_lo);   // a part of S_t lies left of the window
            pj[u] = has_s[u] ? __ldg(pl + j) : make_float2(-CUDART_INF_F, 0.f);
            raw[u] = has_s[u] ? __ldg(reinterpret_cast<const uint4 *>(po + (long long)j * kD)) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int j = j0 + u;
            if (j >= c.top_k) break;
            float l_t = -CUDART_INF_F;
            if (sel[u]) {
                const float lj = pj[u].x;
                const float m = fmaxf(lj, lw);
                const float wj = has_s[u] ? exp2f(lj - m) : 0.f, ww = has_w ? exp2f(lw - m) : 0.f;
                const float den = wj + ww;
                const float alpha = expf(sc[j] - smax) / sden;
                cw = fmaf(alpha, ww / den, cw);
                if (has_s[u]) {
                    const uint32_t eb = (__float_as_uint(pj[u].y) >> (8 * (sub >> 2))) & 0xffu;
                    const float ws = alpha * wj / den * __uint_as_float((eb + 1u) << 23);   // weight x 2^(eb - 126)
                    const uint32_t rw[4] = {raw[u].x, raw[u].y, raw[u].z, raw[u].w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&rw[e]));
                        acc[2 * e] = fmaf(ws, f.x, acc[2 * e]);
                        acc[2 * e + 1] = fmaf(ws, f.y, acc[2 * e + 1]);
                    }
                }
                l_t = (m + log2f(den)) * kLn2;
                if (first) { lse_first = l_t; first = false; }
            }
            if (lse_span && sub == 0) lse_span[orow * c.top_k + j] = l_t;
        }
    }
    if (cw != 0.f) add_piece(raw_w, pw.y, sub, cw, acc);
    uint32_t w[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const __nv_bfloat162 pp = __floats2bfloat162_rn(acc[2 * e], acc[2 * e + 1]);
        w[e] = *reinterpret_cast<const uint32_t *>(&pp);
    }
    *reinterpret_cast<uint4 *>(out + b * c.q_sb + h * c.q_sh + r * c.q_st + sub * 8) = make_uint4(w[0], w[1], w[2], w[3]);
    if (sub == 0) lse[orow] = lse_first;
}

// The same for top_k <= 8, arranged so that the per-row arithmetic (gate, log-sum-exp weights, base
// span length) is done once per row: a warp takes 32 consecutive rows; first every lane works out the
// coefficients of its own row (weight of every span piece, summed weight of the window piece, the
// log-sum-exps), then the warp walks its rows two at a time, 16 lanes per row and 8 columns per lane,
// with the coefficients handed over by shuffles.
constexpr int kGateK = 8;
__global__ void __launch_bounds__(256)
tc_merge_gated_rows(const __half *__restrict__ part_o, const float2 *__restrict__ part_lse,
                    const int32_t *__restrict__ anchor, const float *__restrict__ score, Call c, int slots, int Lc,
                    long long r0, bf16 *__restrict__ out, float *__restrict__ lse, float *__restrict__ lse_span) {
    const int lane = threadIdx.x & 31;
    const long long row0 = ((long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5)) * 32;
    const long long rows = (long long)c.B * c.Hq * Lc;
    if (row0 >= rows) return;
    const bool has_w = c.window > 0;
    // ---- phase A: lane = row
    float coef[kGateK], cw = 0.f;       // weights of the span pieces and of the window piece
    uint32_t ex[kGateK], ex_w = 0u;     // their chunk exponents
    long long out_off = 0;
#pragma unroll
    for (int j = 0; j < kGateK; ++j) { coef[j] = 0.f; ex[j] = 0u; }
    {
        const long long row = row0 + lane;
        if (row < rows) {
            const int rc = (int)((unsigned)row % (unsigned)Lc);   // rows < 2^31
            const int bh = (int)((unsigned)row / (unsigned)Lc);
            const int h = bh % c.Hq, b = bh / c.Hq;
            const long long r = r0 + rc, i = c.q_pos0 + r;
            const long long orow = ((long long)b * c.Hq + h) * c.Lq + r;
            out_off = b * c.q_sb + h * c.q_sh + r * c.q_st;
            const int32_t *an = anchor + orow * c.top_k;
            const float *sc = score + orow * c.top_k;
            const float2 *pl = part_lse + row * slots;
            const long long ell = base_len(c, i);
            const long long w_lo = i - c.window + 1 > 0 ? i - c.window + 1 : 0;
            const float2 pw = has_w ? __ldg(pl + c.top_k) : make_float2(-CUDART_INF_F, 0.f);
            const float lw = pw.x;
            ex_w = __float_as_uint(pw.y);
            float scv[kGateK], lj[kGateK];
            bool sel[kGateK], has_s[kGateK];
            float smax = -CUDART_INF_F;
            int n_sel = 0;
#pragma unroll
            for (int j = 0; j < kGateK; ++j) {
                const long long t = j < c.top_k ? an[j] : -1;
                sel[j] = t >= 0 && t <= i;
                scv[j] = sel[j] ? sc[j] : -CUDART_INF_F;
                const long long a = t - (long long)c.back * ell;
                has_s[j] = sel[j] && (!has_w || (a > 0 ? a : 0) < w_lo);   // a part of S_t lies left of the window
                const float2 pj = has_s[j] ? __ldg(pl + j) : make_float2(-CUDART_INF_F, 0.f);
                lj[j] = pj.x;
                ex[j] = __float_as_uint(pj.y);
                if (sel[j]) { smax = fmaxf(smax, scv[j]); ++n_sel; }
            }
            float sden = 0.f;
#pragma unroll
            for (int j = 0; j < kGateK; ++j)
                if (sel[j]) sden += expf(scv[j] - smax);
            float lse_first = -CUDART_INF_F;
            if (n_sel == 0 && has_w) {   // Algorithm 1, empty selection: the window alone
                cw = 1.f;
                lse_first = lw * kLn2;
            }
            bool first = true;
#pragma unroll
            for (int j = 0; j < kGateK; ++j) {
                if (j >= c.top_k) break;
                float l_t = -CUDART_INF_F;
                if (sel[j]) {
                    const float m = fmaxf(lj[j], lw);
                    const float wj = has_s[j] ? exp2f(lj[j] - m) : 0.f, ww = has_w ? exp2f(lw - m) : 0.f;
                    const float den = wj + ww;
                    const float alpha = expf(scv[j] - smax) / sden;
                    cw = fmaf(alpha, ww / den, cw);
                    coef[j] = has_s[j] ? alpha * wj / den : 0.f;
                    l_t = (m + log2f(den)) * kLn2;
                    if (first) { lse_first = l_t; first = false; }
                }
                if (lse_span) lse_span[orow * c.top_k + j] = l_t;
            }
            lse[orow] = lse_first;
        }
    }
    // ---- phase B: two rows per step, 16 lanes per row
    const int sub = lane & 15, hi = lane >> 4;
    const int shift = 8 * (sub >> 2);
#pragma unroll 4
    for (int rr = 0; rr < 16; ++rr) {
        const int src = 2 * rr + hi;
        const long long row = row0 + src;
        const __half *po = part_o + row * slots * kD + sub * 8;
        float acc[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] = 0.f;
        float cf[kGateK + 1];
        uint32_t ee[kGateK + 1];
        uint4 raw[kGateK + 1];
#pragma unroll
        for (int j = 0; j < kGateK; ++j) {
            cf[j] = __shfl_sync(0xffffffffu, coef[j], src);
            ee[j] = __shfl_sync(0xffffffffu, ex[j], src);
        }
        cf[kGateK] = __shfl_sync(0xffffffffu, cw, src);
        ee[kGateK] = __shfl_sync(0xffffffffu, ex_w, src);
        const long long off = __shfl_sync(0xffffffffu, out_off, src);
#pragma unroll
        for (int j = 0; j <= kGateK; ++j) {
            const int slot = j < kGateK ? j : c.top_k;
            raw[j] = cf[j] != 0.f ? __ldg(reinterpret_cast<const uint4 *>(po + (long long)slot * kD)) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int j = 0; j <= kGateK; ++j)
            if (cf[j] != 0.f) {
                const uint32_t eb = (ee[j] >> shift) & 0xffu;
                const float ws = cf[j] * __uint_as_float((eb + 1u) << 23);   // weight x 2^(eb - 126)
                const uint32_t rw[4] = {raw[j].x, raw[j].y, raw[j].z, raw[j].w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&rw[e]));
                    acc[2 * e] = fmaf(ws, f.x, acc[2 * e]);
                    acc[2 * e + 1] = fmaf(ws, f.y, acc[2 * e + 1]);
                }
            }
        if (row < rows) {
            uint32_t w[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const __nv_bfloat162 pp = __floats2bfloat162_rn(acc[2 * e], acc[2 * e + 1]);
                w[e] = *reinterpret_cast<const uint32_t *>(&pp);
            }
            *reinterpret_cast<uint4 *>(out + off + sub * 8) = make_uint4(w[0], w[1], w[2], w[3]);
        }
    }
}

// ------------------------------------------------------------------------------------------------
PFN_cuTensorMapEncodeTiled_v12000 encode_fn() {
    static PFN_cuTensorMapEncodeTiled_v12000 fn = nullptr;
    if (!fn) {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(ptr);
    }
    return fn;
}

// The three outer dimensions of K / V (token, head, batch) ordered by ascending stride, as the tensor
// map wants them.  Dimensions of size 1 go last (their stride is never used and is replaced by one that
// keeps the list ascending).  False when two dimensions of size > 1 overlap in memory (a stride of 0 from
// a broadcast view, or a stride smaller than the extent of the dimensions inside it): such a layout is
// not a tiled tensor, and the caller sends it to the generic kernels, which follow any strides.
struct KvDim { unsigned long long size, stride; int which; };
bool order_kv_dims(const Call &c, KvDim (&d)[3]) {
    d[0] = {(unsigned long long)c.Lkv, (unsigned long long)c.kv_st * 2, 0};
    d[1] = {(unsigned long long)c.Hkv, (unsigned long long)c.kv_sh * 2, 1};
    d[2] = {(unsigned long long)c.B, (unsigned long long)c.kv_sb * 2, 2};
    for (int a = 0; a < 3; ++a)
        for (int bq = a + 1; bq < 3; ++bq) {
            const bool swap = (d[bq].size > 1 && d[a].size == 1) ? true
                              : (d[a].size > 1 && d[bq].size == 1) ? false
                              : d[bq].stride < d[a].stride;
            if (swap) { KvDim t = d[a]; d[a] = d[bq]; d[bq] = t; }
        }
    unsigned long long extent = (unsigned long long)kD * 2;   // bytes the dimensions inside cover
    for (int a = 0; a < 3; ++a) {
        if (d[a].size == 1) d[a].stride = extent;
        else if (d[a].stride < extent) return false;
        if (d[a].stride >= (1ull << 40)) return false;        // the tensor map's stride field
        extent = d[a].stride * d[a].size;
    }
    return true;
}

// Tensor map over K or V [B, Hkv, Lkv, 128] with arbitrary nested (16-byte aligned) strides; slot[] says
// where (token, head, batch) ended up among the outer dimensions.
bool make_kv_map(CUtensorMap *tm, const void *ptr, const Call &c, int slot[3]) {
    auto fn = encode_fn();
    if (!fn) return false;
    KvDim d[3];
    if (!order_kv_dims(c, d)) return false;
    for (int a = 0; a < 3; ++a) slot[d[a].which] = a;
    cuuint64_t gdim[4] = {(cuuint64_t)kD, d[0].size, d[1].size, d[2].size};
    cuuint64_t gstr[3] = {d[0].stride, d[1].stride, d[2].stride};
    cuuint32_t box[4] = {64, 1, 1, 1};
    box[1 + slot[0]] = kBK;
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(ptr), gdim, gstr, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

// out[0] tiles, out[1] pieces, out[2] sum over tiles of (key blocks walked), out[3] sum of pieces x blocks
__global__ void __launch_bounds__(256) tile_stats(const int4 *__restrict__ tiles, const int *__restrict__ n_tiles,
                                                  unsigned long long *out) {
    const int n = *n_tiles;
    unsigned long long a = 0, b = 0, c2 = 0;
    for (int t = blockIdx.x * blockDim.x + threadIdx.x; t < n; t += gridDim.x * blockDim.x) {
        const int w = tiles[t].w, cnt = w & 0xff, nblk = w >> 8;
        a += cnt; b += nblk; c2 += (unsigned long long)cnt * nblk;
    }
    atomicAdd(out + 1, a); atomicAdd(out + 2, b); atomicAdd(out + 3, c2);
    if (blockIdx.x == 0 && threadIdx.x == 0) out[0] = n;
}

}  // namespace

cudaError_t launch_tile_stats(const TcLast &last, long long *out4_device, cudaStream_t st) {
    cudaError_t e = cudaMemsetAsync(out4_device, 0, 4 * sizeof(long long), st);
    if (e != cudaSuccess) return e;
    tile_stats<<<64, 256, 0, st>>>(last.tiles, last.n_tiles, reinterpret_cast<unsigned long long *>(out4_device));
    return cudaGetLastError();
}

bool tc_attention_shape_ok(const Call &c, int dtype) {
    if (dtype != SLA_BF16 || c.D != kD) return false;
    if (c.kv_st < kD || c.top_k > kMaxTopK || !(c.softmax_scale > 0.f)) return false;
    KvDim d[3];
    if (!order_kv_dims(c, d)) return false;   // overlapping K/V dimensions (broadcast views): generic kernels
    const long long ell = base_len(c, c.q_pos0 + c.Lq - 1);
    long long span_tokens = (long long)(c.back + c.fwd) * ell + 1;
    if (c.window > span_tokens) span_tokens = c.window;
    return span_tokens / kBK + 2 <= kMaxWalk;
}

bool tc_attention_supported(const Call &c, int dtype) {
    return tc_attention_shape_ok(c, dtype) && encode_fn() != nullptr;
}

// Scratch layout for a chunk of Lc query positions; returns total bytes.
TcPlan plan_attention_tc(const Call &c, int Lc, size_t gap) {
    TcPlan p;
    p.Lc = Lc;
    p.n_bg = c.B * c.Hkv;
    p.NB = (int)((c.Lkv + kBK - 1) / kBK);
    const long long ell = base_len(c, c.q_pos0 + c.Lq - 1);
    long long span_tokens = (long long)(c.back + c.fwd) * ell + 1;
    if (c.window > span_tokens) span_tokens = c.window;   // the window is a piece too
    if (span_tokens > c.Lkv) span_tokens = c.Lkv;
    p.nb_single = (int)((span_tokens - 1) / kBK + 2);
    // Pieces of a group are ordered by blocks covered, in as many classes as the CTA-local histogram
    // of the counting sort affords (NB * ncls counters in shared memory): up to 8 for the lengths of a
    // single span and, in union mode, up to 32 more for pieces joined from spans that overlap or touch.
    // A tile walks as many key blocks as its longest piece, so a joined piece may only be as long as the
    // classes can still tell apart: when classes of at most kJoinWidth blocks reach up to the longest
    // joined piece there can be (all spans and the window in one), everything that touches is joined;
    // otherwise the classes are shared between single spans and joined pairs, and a piece stops growing
    // at twice a span (measured on the 262144-token configuration: pairs -4 %, triples +1 %).
    const size_t hist_cap = 160 * 1024;
    constexpr int kJoinWidth = 3;
    const int ncls_avail = (int)(hist_cap / ((size_t)p.NB * 4));
    p.ncls1 = p.nb_single < 8 ? p.nb_single : 8;
    while (p.ncls1 > 1 && p.ncls1 > ncls_avail) p.ncls1 /= 2;
    int ncls2 = 0;
    p.nb_max = p.nb_single;
    if (c.mode == SLA_UNION && ncls_avail > p.ncls1) {
        long long joined = (long long)c.top_k * ((long long)(c.back + c.fwd) * ell + 1) + c.window;
        if (joined > c.Lkv) joined = c.Lkv;
        long long nb_full = (joined - 1) / kBK + 2;
        if (nb_full > kMaxWalk) nb_full = kMaxWalk;
        const long long extra = nb_full - p.nb_single;
        const int avail2 = ncls_avail - p.ncls1 < 32 ? ncls_avail - p.ncls1 : 32;
        if (extra > 0 && extra <= (long long)kJoinWidth * avail2) {
            ncls2 = (int)((extra + kJoinWidth - 1) / kJoinWidth);   // fewer classes: fewer global counter updates
            p.nb_max = (int)nb_full;
        } else if (extra > 0 && ncls_avail >= 4) {
            if (p.ncls1 > ncls_avail / 2) p.ncls1 = ncls_avail / 2;
            const int want2 = (p.nb_single + kJoinWidth - 1) / kJoinWidth;
            ncls2 = ncls_avail - p.ncls1 < want2 ? ncls_avail - p.ncls1 : want2;
            if (ncls2 > 32) ncls2 = 32;
            p.nb_max = 2LL * p.nb_single < nb_full ? 2 * p.nb_single : (int)nb_full;
        }
    }
    p.merge_cap = ncls2 > 0 ? (p.nb_max - 2) * kBK : 0;   // a piece of T tokens covers at most (T-1)/64 + 2 blocks
    p.ncls = p.ncls1 + ncls2;
    p.ok = (size_t)p.NB * p.ncls * 4 <= hist_cap;
    // the work-list kernels hold one CTA per SM (their histogram fills the shared memory): no more CTAs
    // than SMs, or the last few would run as a second wave
    p.ctas_per_bg = 148 / p.n_bg > 1 ? 148 / p.n_bg : 1;
    const size_t rows = (size_t)c.B * c.Hq * Lc;
    p.slots = c.top_k + (c.window > 0 ? 1 : 0);
    const size_t slots = rows * p.slots;
    const size_t n_keys = (size_t)p.n_bg * p.NB * p.ncls;
    // every (batch, kv head) list is cut every kRows records (one ragged tile each) and split again at
    // gaps between end blocks (fewer than NB per list)
    p.max_tiles = (long long)(slots / kRows) + (long long)p.n_bg * (p.NB + 1) + 1;
    size_t off = 0;
    // a region of `size` bytes at the next 256-byte boundary, with a canary gap before it when asked for
    auto take = [&](size_t size) {
        if (gap) { p.canaries.add(off); off += gap; }
        const size_t at = off;
        off = align256(off + size);
        return at;
    };
    p.off_counters = take(64 + (size_t)p.n_bg * 8);
    // the two bucket tables are cleared together at the start of every chunk: no gap between them
    p.off_key_count = take(2 * align256(n_keys * 4));
    p.off_key_cursor = p.off_key_count + align256(n_keys * 4);
    p.off_cta_hist = take((size_t)p.ctas_per_bg * n_keys * 4);
    p.off_tiles = take((size_t)p.max_tiles * 16);
    p.off_recs = take(slots * 16);
    p.off_npieces = take(rows);
    p.off_part_lse = take(slots * 8);
    p.off_part_o = take(slots * kD * 2);
    if (gap) { p.canaries.add(off); off += gap; }
    p.bytes = off;
    return p;
}

cudaError_t launch_attn_tc(const void *q, const void *k, const void *v, const Call &c, const int32_t *anchor,
                           const float *score, void *out, float *lse, float *lse_span, void *scratch, size_t scratch_bytes, int sm_count,
                           cudaStream_t st, long long *launches, KernelTimer *timer, bool canaries, TcLast *last) {
    // the largest chunk of query positions whose scratch fits
    const size_t gap = canaries ? Canaries::kBytes : 0;
    long long Lc = c.Lq;
    TcPlan plan = plan_attention_tc(c, (int)Lc, gap);
    while (plan.bytes > scratch_bytes && Lc > 1) {
        Lc = (Lc + 1) / 2;
        plan = plan_attention_tc(c, (int)Lc, gap);
    }
    if (plan.bytes > scratch_bytes || !plan.ok) return cudaErrorMemoryAllocation;
    if (plan.max_tiles > (1ll << 30) || (long long)c.B * c.Hq * Lc * plan.slots > (1ll << 31) - 1) return cudaErrorInvalidValue;

    CUtensorMap tm_k, tm_v;
    int slot[3];
    if (!make_kv_map(&tm_k, k, c, slot) || !make_kv_map(&tm_v, v, c, slot)) return cudaErrorInvalidValue;
    // function attributes belong to a device's context: remember them per device, not per process
    static bool attr_set[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return cudaErrorInvalidDevice;
    if (dev < 0 || dev >= 64 || !attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(tc_attend, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) attr_set[dev] = true;
    }
    char *ws = (char *)scratch;
    int *counters = (int *)(ws + plan.off_counters);
    for (long long r0 = 0; r0 < c.Lq; r0 += Lc) {
        const int lc = (int)((c.Lq - r0 < Lc) ? c.Lq - r0 : Lc);
        const long long rows = (long long)c.B * c.Hq * lc;
        cudaError_t e = cudaMemsetAsync(ws + plan.off_key_count, 0, 2 * (plan.off_key_cursor - plan.off_key_count), st);
        if (e != cudaSuccess) return e;
        if (canaries && (e = launch_canary_fill(ws, plan.canaries, st)) != cudaSuccess) return e;
        tc::PrepArgs pa;
        pa.anchor = anchor; pa.B = c.B; pa.Hq = c.Hq; pa.Hkv = c.Hkv; pa.G = c.G; pa.top_k = c.top_k;
        pa.span_len = c.span_len; pa.back = c.back; pa.fwd = c.fwd; pa.Lq = c.Lq; pa.q_pos0 = c.q_pos0;
        pa.window = c.window; pa.mode = c.mode; pa.len_first = c.len_first; pa.n_len = c.n_len;
        pa.r0 = r0; pa.Lc = lc; pa.NB = plan.NB; pa.nb_max = plan.nb_max; pa.ncls = plan.ncls;
        pa.nb_single = plan.nb_single; pa.ncls1 = plan.ncls1; pa.merge_cap = plan.merge_cap;
        pa.ctas_per_bg = plan.ctas_per_bg;
        pa.key_count = (int *)(ws + plan.off_key_count);
        pa.key_cursor = (int *)(ws + plan.off_key_cursor);
        pa.totals = counters + 16;
        pa.n_tiles = counters;
        pa.tiles = (int4 *)(ws + plan.off_tiles);
        pa.max_tiles = (int)plan.max_tiles;
        pa.recs = (int4 *)(ws + plan.off_recs);
        // the parked pieces borrow the head of the partial-output buffer, which is written only after them
        pa.stage = (int4 *)(ws + plan.off_part_o); pa.slots = plan.slots;
        pa.cta_hist = (int *)(ws + plan.off_cta_hist);
        pa.n_pieces = (unsigned char *)(ws + plan.off_npieces);
        pa.status = c.status;
        e = tc::prepare(pa, st, launches);
        if (e != cudaSuccess) return e;
        TcParams tp;
        tp.q = (const bf16 *)q; tp.q_sb = c.q_sb; tp.q_sh = c.q_sh; tp.q_st = c.q_st;
        tp.Hq = c.Hq; tp.G = c.G; tp.Lc = lc; tp.slots = plan.slots; tp.r0 = r0;
        tp.scale2 = c.softmax_scale * kLog2e;
        tp.slot_t = slot[0]; tp.slot_h = slot[1]; tp.slot_b = slot[2];
        tp.recs = pa.recs; tp.tiles = pa.tiles;
        tp.n_tiles = counters;
        tp.part_o = (__half *)(ws + plan.off_part_o); tp.part_lse = (float2 *)(ws + plan.off_part_lse);
        tp.status = c.status; tp.Hkv = c.Hkv;
        if (last) { last->tiles = pa.tiles; last->n_tiles = counters; }
        if (timer) timer->begin(st);
        tc_attend<<<2 * sm_count, kThreads, kSmemBytes, st>>>(tm_k, tm_v, tp);
        if (timer) timer->end(st);
        const unsigned mblocks = (unsigned)((rows * 16 + 255) / 256);
        if (c.mode == SLA_PER_SPAN && c.top_k <= kGateK)
            tc_merge_gated_rows<<<(unsigned)((rows + 255) / 256), 256, 0, st>>>(tp.part_o, tp.part_lse, anchor, score, c,
                                                                               plan.slots, lc, r0, (bf16 *)out, lse, lse_span);
        else if (c.mode == SLA_PER_SPAN)
            tc_merge_gated<<<mblocks, 256, 0, st>>>(tp.part_o, tp.part_lse, anchor, score, c, plan.slots, lc, r0,
                                                    (bf16 *)out, lse, lse_span);
        else
            tc_merge<<<mblocks, 256, 0, st>>>(tp.part_o, tp.part_lse, pa.n_pieces, c, plan.slots, lc, r0, (bf16 *)out, lse);
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        if (launches) *launches += 2;
        if (canaries && (e = launch_canary_check(ws, plan.canaries, c.status, st)) != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace sla
