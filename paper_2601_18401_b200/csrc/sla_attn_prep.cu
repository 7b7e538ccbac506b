// Work-list construction for the tensor-core span-attention kernel: a counting sort of all pieces
// (clipped spans) of a chunk of query rows by (batch*Hkv + kv head, 64-key block of the piece's
// right end, class of blocks covered), and the table of 128-piece tiles cut from the sorted list.
//
// This is the step Section "Kernel design" describes as grouping (query, span) pairs into buckets by
// key-block footprint without a global sort.  Each CTA owns a slice of the rows of one
// (batch, kv head), counts its pieces in a shared-memory histogram and touches the global counters
// once per non-empty bucket, so that global atomics stay far below one per piece.
//
//   prep_count       the pieces of every row, parked; histogram of bucket sizes; pieces per row
//   prep_scan_local  per (batch, kv head): exclusive offsets of its buckets, record and tile totals
//   prep_scan_global per (batch, kv head): global offsets, tile table entries (a tile = 128 consecutive
//                    records of the sorted list, whatever end blocks they fall in)
//   prep_scatter     the parked pieces to their places in the sorted list
//   prep_tile_bounds per tile: split where neighbouring pieces end far apart; the tile's end block and how
//                    far back its pieces reach (number of key blocks to walk)
#include <limits.h>

#include "sla_attn_tc.cuh"

namespace sla {
namespace tc {

namespace {

constexpr int kPrepThreads = 1024;

// Bucket of a piece: its end block and the class of the number of blocks it covers.  Classes are even
// steps over [0, nb_single) (a single span) and, for joined pieces, over [nb_single, nb_max).
__device__ __forceinline__ int class_of(int len, const PrepArgs &a) {
    int cls;
    if (len < a.nb_single || a.ncls == a.ncls1) {
        cls = (len * a.ncls1) / a.nb_single;
        cls = cls < a.ncls1 ? cls : a.ncls1 - 1;
    } else {
        cls = a.ncls1 + ((len - a.nb_single) * (a.ncls - a.ncls1)) / (a.nb_max - a.nb_single + 1);
        cls = cls < a.ncls ? cls : a.ncls - 1;
    }
    return cls;
}
// Classes run upwards in even end blocks and downwards in odd ones, so that the sorted list changes
// length smoothly from one end block to the next (tiles are cut across those boundaries).
__device__ __forceinline__ int bucket_at(int eb, int cls, const PrepArgs &a) {
    return eb * a.ncls + ((eb & 1) ? a.ncls - 1 - cls : cls);
}
__device__ __forceinline__ int bucket_of(int lo, int hi, const PrepArgs &a) {
    const int eb = hi / kBK, sb = lo / kBK;
    return bucket_at(eb, class_of(eb - sb, a), a);
}

// Union-mode pieces of one row for at most K intervals (anchors + window), streamed: emit(lo, hi, n) is
// called for the n-th piece, left to right.  Same pieces as row_pieces up to the order in which
// intervals with the same left end are clipped (the union, and with it the attention, is the same).
// All spans of a row are equally long before clipping, so ordering them by anchor orders them by
// (lo, hi); the window W = [w_lo, i] takes its place through the anchor that would give lo = w_lo.
// Keys are 2t for a span and 2t_W + 1 for W (after the spans that start at or before w_lo).
template <int K, typename Emit>
__device__ __forceinline__ int union_pieces_stream(const int32_t *__restrict__ an, int top_k, int i, long long ell,
                                                   int back, int fwd, int window, int merge_cap, int *status,
                                                   Emit emit) {
    constexpr unsigned kAbsent = 0xffffffffu;
    const long long bl64 = (long long)back * ell, fl64 = (long long)fwd * ell;
    const int bl = bl64 > INT_MAX ? INT_MAX : (int)bl64, fl = fl64 > INT_MAX ? INT_MAX : (int)fl64;
    const int w_lo = i - window + 1 > 0 ? i - window + 1 : 0;
    unsigned key[K];
#pragma unroll
    for (int j = 0; j < K; ++j) {
        key[j] = kAbsent;
        if (j < top_k) {
            const int t = an[j];
            if (t > i) atomicOr(status, kStatusBadIndex);
            else if (t >= 0) key[j] = 2u * (unsigned)t;
        } else if (j == top_k && window > 0) {
            unsigned tw = (unsigned)w_lo + (unsigned)bl;
            if (tw > (unsigned)i + 1u) tw = (unsigned)i + 1u;
            if (tw > 0x7ffffffeu) tw = 0x7ffffffeu;   // stays below the "absent" key
            key[j] = 2u * tw + 1u;
        }
    }
#pragma unroll
    for (int round = 0; round < K; ++round)
#pragma unroll
        for (int x = round & 1; x + 1 < K; x += 2) {
            const unsigned lo_ = min(key[x], key[x + 1]), hi_ = max(key[x], key[x + 1]);
            key[x] = lo_;
            key[x + 1] = hi_;
        }
    int cnt = 0, cur_lo = 0, cur_hi = -1, next_free = 0;
    bool have = false;
#pragma unroll
    for (int x = 0; x < K; ++x) {
        const unsigned kx = key[x];
        const bool present = kx != kAbsent;
        const int t = (int)(kx >> 1);
        int l0, h0;
        if (kx & 1u) {
            l0 = w_lo;
            h0 = i;
        } else {
            l0 = bl >= t ? 0 : t - bl;
            h0 = fl >= i - t ? i : t + fl;
        }
        const int j0 = l0 > next_free ? l0 : next_free;
        const bool on = present && j0 <= h0;
        // the piece in hand ends at next_free - 1: an interval that continues right there is joined to it
        const bool join = on && have && j0 == next_free && h0 - cur_lo < merge_cap;
        if (on && !join) {
            if (have) emit(cur_lo, cur_hi, cnt++);
            cur_lo = j0;
            have = true;
        }
        if (on) cur_hi = h0;
        if (present && h0 + 1 > next_free) next_free = h0 + 1;
    }
    if (have) emit(cur_lo, cur_hi, cnt++);
    return cnt;
}

// Rows of one (batch, kv head) are shared out evenly among ctas_per_bg CTAs, the same way in both passes.
struct Share {
    int bg, g, b;
    long long q0, q1;
};
__device__ __forceinline__ Share share_of(const PrepArgs &a) {
    Share s;
    s.bg = blockIdx.x / a.ctas_per_bg;
    const int part = blockIdx.x % a.ctas_per_bg;
    s.g = s.bg % a.Hkv;
    s.b = s.bg / a.Hkv;
    const long long rows_bg = (long long)a.G * a.Lc;
    const long long per = (rows_bg + a.ctas_per_bg - 1) / a.ctas_per_bg;
    s.q0 = per * part < rows_bg ? per * part : rows_bg;   // a CTA beyond the last row gets an empty range
    s.q1 = (s.q0 + per < rows_bg) ? s.q0 + per : rows_bg;
    return s;
}
__device__ __forceinline__ int row_of(const PrepArgs &a, const Share &s, long long q, int &h, int &rc) {
    const int hg = (int)((unsigned)q / (unsigned)a.Lc);   // G * Lc < 2^31
    rc = (int)((unsigned)q % (unsigned)a.Lc);
    h = s.g * a.G + hg;
    return (int)(((long long)s.b * a.Hq + h) * a.Lc + rc);
}

// Counting pass.  Every piece of the CTA's rows is built once, counted in the CTA's shared-memory
// histogram (the value the atomic returns is the piece's ordinal within its bucket and CTA) and parked
// in `stage`; the histogram goes to the global bucket counts and, whole, to cta_hist.
// K: compile-time bound on the intervals of a row (anchors + window) for the register-resident piece
// builder, or 0 for the general one.
template <int K>
__global__ void __launch_bounds__(kPrepThreads) prep_count(PrepArgs a) {
    extern __shared__ int hist[];   // [NB * ncls]
    constexpr int KA = K > 0 ? K : kMaxTopK + 1;
    const int nk = a.NB * a.ncls;
    const Share sh = share_of(a);
    // class of every "blocks covered" value, behind the histogram
    unsigned char *cls_tbl = reinterpret_cast<unsigned char *>(hist + nk);
    for (int x = threadIdx.x; x < nk; x += kPrepThreads) hist[x] = 0;
    for (int x = threadIdx.x; x <= a.nb_max; x += kPrepThreads) cls_tbl[x] = (unsigned char)class_of(x, a);
    __syncthreads();
    int lo[KA], hi[KA], slot[KA];
    for (long long q = sh.q0 + threadIdx.x; q < sh.q1; q += kPrepThreads) {
        int h, rc;
        const int row = row_of(a, sh, q, h, rc);
        const long long r = a.r0 + rc, i = a.q_pos0 + r;
        const int32_t *an = a.anchor + (((long long)sh.b * a.Hq + h) * a.Lq + r) * a.top_k;
        const long long ell = base_len(i, a.span_len, a.len_first, a.n_len);
        if constexpr (K > 0) {
            if (a.mode == SLA_UNION) {
                int4 *st = a.stage + (long long)row * a.slots;
                const int n = union_pieces_stream<KA>(an, a.top_k, (int)i, ell, a.back, a.fwd, a.window, a.merge_cap, a.status,
                                                      [&](int l0, int h0, int ordinal) {
                                                          const int eb = h0 / kBK, len = eb - l0 / kBK;
                                                          const int bucket = bucket_at(eb, cls_tbl[len < a.nb_max ? len : a.nb_max], a);
                                                          const int ord = atomicAdd(&hist[bucket], 1);
                                                          st[ordinal] = make_int4(l0, h0, bucket | (ordinal << 24), ord);
                                                      });
                a.n_pieces[row] = (unsigned char)n;
                continue;
            }
        }
        int cnt;
        if constexpr (K > 0)
            cnt = row_pieces_per_span_small<KA>(an, a.top_k, i, ell, a.back, a.fwd, a.window, lo, hi, slot, a.status);
        else
            cnt = row_pieces(an, a.top_k, i, ell, a.back, a.fwd, a.window, a.mode, a.merge_cap, lo, hi, slot, a.status);
        a.n_pieces[row] = (unsigned char)cnt;
        int4 *st = a.stage + (long long)row * a.slots;
        auto park = [&](int j) {
            const int bucket = bucket_of(lo[j], hi[j], a);
            const int ord = atomicAdd(&hist[bucket], 1);
            st[j] = make_int4(lo[j], hi[j], bucket | (slot[j] << 24), ord);
        };
        if constexpr (K > 0) {
#pragma unroll
            for (int j = 0; j < KA; ++j)
                if (j < cnt) park(j);
        } else {
            for (int j = 0; j < cnt; ++j) park(j);
        }
    }
    __syncthreads();
    int *gcount = a.key_count + (long long)sh.bg * nk;
    int *mine = a.cta_hist + (long long)blockIdx.x * nk;
    for (int x = threadIdx.x; x < nk; x += kPrepThreads) {
        const int c = hist[x];
        mine[x] = c;
        if (c) atomicAdd(gcount + x, c);
    }
}

// Scatter pass: the CTA claims a contiguous range of every bucket it has pieces in (its count is in
// cta_hist, the bucket's global offset in key_count by now) and moves its parked pieces to their places.
__global__ void __launch_bounds__(kPrepThreads) prep_scatter(PrepArgs a) {
    extern __shared__ int hist[];   // [NB * ncls]: first record of this CTA in every bucket
    const int nk = a.NB * a.ncls;
    const Share sh = share_of(a);
    const int *gcount = a.key_count + (long long)sh.bg * nk;
    int *gcursor = a.key_cursor + (long long)sh.bg * nk;
    const int *mine = a.cta_hist + (long long)blockIdx.x * nk;
    // four buckets per thread and round, so that the counts, then the claims, are in flight together
    for (int x0 = threadIdx.x; x0 < nk; x0 += 4 * kPrepThreads) {
        int cnt[4], first[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int x = x0 + u * kPrepThreads;
            cnt[u] = x < nk ? mine[x] : 0;
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int x = x0 + u * kPrepThreads;
            first[u] = cnt[u] ? gcount[x] + atomicAdd(gcursor + x, cnt[u]) : 0;
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int x = x0 + u * kPrepThreads;
            if (x < nk) hist[x] = first[u];
        }
    }
    __syncthreads();
    // One thread per parked slot, four slots in flight per thread.  The rows of a (batch, kv head) are
    // consecutive (row = first row + q), so the CTA's slots are one contiguous run of `stage`.
    const unsigned n_el = (unsigned)((sh.q1 - sh.q0) * a.slots);   // rows x slots < 2^31 for the whole chunk
    const long long row_base = ((long long)sh.b * a.Hq + sh.g * a.G) * a.Lc + sh.q0;
    const int4 *st = a.stage + row_base * a.slots;
    constexpr int U = 4;
    for (unsigned e0 = threadIdx.x; e0 < n_el; e0 += U * kPrepThreads) {
        int4 pc[U];
        int row[U], cnt[U], j[U];
        // all loads first (a slot beyond the row's count holds stale bytes that are not looked at)
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const unsigned e = e0 + u * kPrepThreads;
            const unsigned ql = e / (unsigned)a.slots;
            j[u] = (int)(e - ql * (unsigned)a.slots);
            row[u] = (int)(row_base + ql);
            cnt[u] = 0;
            if (e < n_el) {
                cnt[u] = a.n_pieces[row[u]];
                pc[u] = __ldg(st + e);
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (j[u] < cnt[u])
                a.recs[hist[pc[u].z & 0xffffff] + pc[u].w] = make_int4(row[u], pc[u].z >> 24, pc[u].x, pc[u].y);
    }
}

// Exclusive scan over the block: returns this thread's offset, total in `total`.
__device__ inline int block_excl_scan(int v, int &total, int *warp_sum) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int x = v;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int y = __shfl_up_sync(0xffffffffu, x, off);
        if (lane >= off) x += y;
    }
    if (lane == 31) warp_sum[warp] = x;
    __syncthreads();
    if (warp == 0) {
        int w = warp_sum[lane];
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int y = __shfl_up_sync(0xffffffffu, w, off);
            if (lane >= off) w += y;
        }
        warp_sum[lane] = w;
    }
    __syncthreads();
    total = warp_sum[31];
    const int base = warp > 0 ? warp_sum[warp - 1] : 0;
    __syncthreads();
    return base + x - v;
}

// One CTA per (batch, kv head): bucket histogram -> exclusive offsets local to the (batch, kv head),
// plus how many records and tiles it has.
__global__ void __launch_bounds__(kPrepThreads) prep_scan_local(PrepArgs a) {
    __shared__ int warp_sum[32];
    const int nk = a.NB * a.ncls, bg = blockIdx.x, tid = threadIdx.x;
    int *cnt = a.key_count + (long long)bg * nk;
    const int per = (nk + kPrepThreads - 1) / kPrepThreads;
    const int k0 = per * tid, k1 = (k0 + per < nk) ? k0 + per : nk;
    int local = 0;
    for (int k = k0; k < k1; ++k) local += cnt[k];
    int n_recs;
    int run = block_excl_scan(local, n_recs, warp_sum);
    for (int k = k0; k < k1; ++k) {
        const int c = cnt[k];
        cnt[k] = run;
        run += c;
    }
    // tiles: the sorted list of the (batch, kv head) is cut every kRows records, across end blocks
    if (tid == 0) {
        a.totals[2 * bg] = n_recs;
        a.totals[2 * bg + 1] = (n_recs + kRows - 1) / kRows;
    }
}

// One CTA per (batch, kv head): offsets become global, tile table entries are written.
__global__ void __launch_bounds__(kPrepThreads) prep_scan_global(PrepArgs a) {
    __shared__ int s_base[2];
    const int nk = a.NB * a.ncls, bg = blockIdx.x, tid = threadIdx.x, n_bg = a.B * a.Hkv;
    if (tid == 0) {
        int rec_base = 0, tile_base = 0;
        for (int x = 0; x < bg; ++x) { rec_base += a.totals[2 * x]; tile_base += a.totals[2 * x + 1]; }
        s_base[0] = rec_base;
        s_base[1] = tile_base;
        if (bg == n_bg - 1) {
            const int all = tile_base + a.totals[2 * bg + 1];
            a.n_tiles[0] = a.n_tiles[1] = all < a.max_tiles ? all : a.max_tiles;   // [1]: the count as cut here
        }
    }
    __syncthreads();
    const int rec_base = s_base[0], tile_base = s_base[1], n_recs = a.totals[2 * bg];
    int *cnt = a.key_count + (long long)bg * nk;
    // tile entries {batch*Hkv + kv head, (end block: filled in by prep_tile_bounds), first record, records}
    const int nt = (n_recs + kRows - 1) / kRows;
    for (int t = tid; t < nt; t += kPrepThreads) {
        const int left = n_recs - t * kRows;
        if (tile_base + t < a.max_tiles)
            a.tiles[tile_base + t] = make_int4(bg, 0, rec_base + t * kRows, left < kRows ? left : kRows);
    }
    __syncthreads();
    for (int k = tid; k < nk; k += kPrepThreads) cnt[k] += rec_base;
}

// One warp per tile as cut by prep_scan_global (128 consecutive records).  Where two neighbouring
// records of the tile end more than kGap key blocks apart the tile is split there (the pieces left of
// the gap would be walked through it for nothing); the extra tiles are appended to the table.  For
// every tile: the end block of its last piece (second word) and the number of key blocks from the one
// its furthest-reaching piece starts in up to that end block (bits 8.. of the last word).
constexpr int kGap = 2;
__global__ void __launch_bounds__(256) prep_tile_bounds(PrepArgs a) {
    __shared__ int s_eb[8][kRows], s_lo[8][kRows];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int t = blockIdx.x * 8 + warp;
    if (t >= a.n_tiles[1]) return;
    const int4 ti = a.tiles[t];
    const int cnt = ti.w;
    int *eb = s_eb[warp], *lo = s_lo[warp];
    for (int x = lane; x < cnt; x += 32) {
        const int4 rec = a.recs[ti.z + x];
        eb[x] = rec.w / kBK;
        lo[x] = rec.z;
    }
    __syncwarp();
    int seg0 = 0, n_seg = 0;
    while (seg0 < cnt) {
        // first record after seg0 that lies beyond a gap (records are ordered by end block)
        int seg1 = cnt;
        for (int x0 = seg0 + 1; x0 < cnt && seg1 == cnt; x0 += 32) {
            const int x = x0 + lane;
            const bool cut = x < cnt && eb[x] - eb[x - 1] > kGap;
            const unsigned m = __ballot_sync(0xffffffffu, cut);
            if (m) seg1 = x0 + __ffs(m) - 1;
        }
        int lo_min = INT_MAX;
        for (int x = seg0 + lane; x < seg1; x += 32) lo_min = min(lo_min, lo[x]);
        lo_min = __reduce_min_sync(0xffffffffu, lo_min);
        const int eb_last = eb[seg1 - 1];
        int idx = t;
        if (n_seg > 0) {
            if (lane == 0) idx = atomicAdd(a.n_tiles, 1);
            idx = __shfl_sync(0xffffffffu, idx, 0);
        }
        if (lane == 0) {
            if (idx < a.max_tiles)
                a.tiles[idx] = make_int4(ti.x, eb_last, ti.z + seg0, (seg1 - seg0) | ((eb_last - lo_min / kBK + 1) << 8));
            else
                atomicOr(a.status, kStatusBadIndex);   // cannot happen: the table has room for one tile per bucket more
        }
        seg0 = seg1;
        ++n_seg;
    }
}

}  // namespace

cudaError_t prepare(const PrepArgs &a, cudaStream_t st, long long *launches) {
    const int n_bg = a.B * a.Hkv;
    // histogram, and behind it the class table of the counting pass (one byte per length)
    const size_t smem = (size_t)a.NB * a.ncls * sizeof(int) + (((size_t)a.nb_max + 1 + 15) & ~(size_t)15);
    // register-resident piece builder for up to 8 / 16 anchors (+ window), the general one otherwise
    const int n_iv = a.top_k + (a.window > 0 ? 1 : 0);
    const int variant = n_iv <= 9 ? 0 : n_iv <= 17 ? 1 : 2;
    void (*k0)(PrepArgs) = variant == 0 ? prep_count<9> : variant == 1 ? prep_count<17> : prep_count<0>;
    void (*k1)(PrepArgs) = prep_scatter;
    // function attributes belong to a device's context: remember the largest size set per device
    static size_t attr_bytes[64][4] = {};   // the three counting kernels and the scatter kernel
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return cudaErrorInvalidDevice;
    const bool known = dev >= 0 && dev < 64;
    if (smem > 48 * 1024) {
        if (!known || smem > attr_bytes[dev][variant]) {
            cudaError_t e = cudaFuncSetAttribute(k0, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return e;
            if (known) attr_bytes[dev][variant] = smem;
        }
        if (!known || smem > attr_bytes[dev][3]) {
            cudaError_t e = cudaFuncSetAttribute(k1, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return e;
            if (known) attr_bytes[dev][3] = smem;
        }
    }
    const unsigned grid = (unsigned)(n_bg * a.ctas_per_bg);
    k0<<<grid, kPrepThreads, smem, st>>>(a);
    prep_scan_local<<<n_bg, kPrepThreads, 0, st>>>(a);
    prep_scan_global<<<n_bg, kPrepThreads, 0, st>>>(a);
    k1<<<grid, kPrepThreads, smem, st>>>(a);
    prep_tile_bounds<<<(unsigned)((a.max_tiles + 7) / 8), 256, 0, st>>>(a);
    if (launches) *launches += 5;
    return cudaGetLastError();
}

}  // namespace tc
}  // namespace sla
