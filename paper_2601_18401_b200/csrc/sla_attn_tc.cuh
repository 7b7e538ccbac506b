// Definitions shared by the tensor-core span-attention kernel (sla_attn_tc.cu) and the kernels that
// prepare its work list (sla_attn_prep.cu).  Internal to libsla.
#pragma once

#include "sla_kernels.h"

namespace sla {
namespace tc {

constexpr int kBK = 64;     // keys per block
constexpr int kRows = 128;  // pieces per tile

// Work list of one chunk of query positions, as laid out in the scratch memory:
//   recs   int4 {row, slot of the row's partial results, lo, hi}: every piece of every row, ordered by
//          (batch*Hkv + kv head, 64-key block of hi, class of blocks covered)
//   tiles  int4 {batch*Hkv + kv head, end block of the last record, first record, records | key blocks to walk << 8}:
//          128 consecutive records, split where neighbouring records end more than a few key blocks apart
//   n_tiles, n_pieces[row], and the per-piece partial results
struct PrepArgs {
    const int32_t *anchor;   // [B,Hq,Lq,top_k]
    int B, Hq, Hkv, G, top_k, span_len, back, fwd;
    int window, mode;        // local window w (0 = none); sla_mode_t
    const int *len_first;    // steps of l(i) for a span exponent other than 1/2 (device), else NULL
    int n_len;
    long long Lq, q_pos0, r0;
    int Lc;                  // query positions in this chunk
    int NB;                  // 64-key blocks in [0, Lkv)
    int nb_max;              // most blocks a piece can cover
    int nb_single;           // most blocks a single span (or the window) can cover
    int ncls;                // classes of "blocks covered" the pieces are ordered by inside a group:
    int ncls1;               // ncls1 of them divide [0, nb_single), the other ncls - ncls1 divide [nb_single, nb_max)
    int merge_cap;           // union mode: touching pieces are joined while the result stays within this many tokens
    int ctas_per_bg;         // CTAs that share the rows of one (batch, kv head)
    int *key_count;          // [B*Hkv][NB*ncls]: histogram, then exclusive offsets
    int *key_cursor;         // same shape
    int *totals;             // [B*Hkv][2]: records and tiles of each (batch, kv head)
    int *n_tiles;            // total number of tiles
    int4 *tiles;
    int max_tiles;
    int4 *recs;
    int4 *stage;             // [rows][slots] {lo, hi, bucket | slot << 24, ordinal within (CTA, bucket)}: the pieces as
                             // the counting pass found them, so that the scatter pass need not build them again
    int slots;               // partial results (and staged pieces) per row
    int *cta_hist;           // [CTAs][NB*ncls]: every CTA's bucket counts
    unsigned char *n_pieces; // [rows]
    int *status;
};

// Pieces of one row and the slot each one's partial result goes to (slots per row: top_k, plus one
// when there is a local window W = [max(0, i-w+1), i]).
//   union mode     the spans of the selected anchors (Algorithm 1: S_t = [max(0,t-b l), min(i,t+f l)])
//                  and W, sorted by (lo, hi) and clipped so that each key is kept once; a piece that
//                  starts right where the one before it ends is joined to it (while the joined piece
//                  stays within merge_cap tokens): overlapping spans become one longer piece, with one
//                  partial result; slots are the pieces' ordinals left to right;
//   per-span mode  J_t = S_t united with W is attended as two disjoint pieces: the part of S_t left of
//                  W in slot j (the anchor's index in the selection) and W, once per row, in slot top_k.
// Returns the number of pieces; lo[], hi[], slot[] need top_k + 1 entries.
__device__ inline int row_pieces(const int32_t *__restrict__ an, int top_k, long long i, long long ell,
                                 int back, int fwd, int window, int mode, int merge_cap, int *lo, int *hi,
                                 int *slot, int *status) {
    const int w_lo = (int)(i - window + 1 > 0 ? i - window + 1 : 0);
    int n = 0;
    if (mode == SLA_PER_SPAN) {
        for (int j = 0; j < top_k; ++j) {
            const long long t = an[j];
            if (t > i) { atomicOr(status, kStatusBadIndex); continue; }
            if (t < 0) continue;
            const long long a = t - (long long)back * ell, z = t + (long long)fwd * ell;
            const int l0 = (int)(a > 0 ? a : 0);
            int h0 = (int)(z < i ? z : i);
            if (window > 0 && h0 >= w_lo) h0 = w_lo - 1;
            if (l0 > h0) continue;
            lo[n] = l0;
            hi[n] = h0;
            slot[n] = j;
            ++n;
        }
        if (window > 0) {
            lo[n] = w_lo;
            hi[n] = (int)i;
            slot[n] = top_k;
            ++n;
        }
        return n;
    }
    for (int j = 0; j <= top_k; ++j) {
        int l0, h0;
        if (j == top_k) {
            if (window <= 0) break;
            l0 = w_lo;
            h0 = (int)i;
        } else {
            const long long t = an[j];
            if (t > i) { atomicOr(status, kStatusBadIndex); continue; }
            if (t < 0) continue;
            const long long a = t - (long long)back * ell, z = t + (long long)fwd * ell;
            l0 = (int)(a > 0 ? a : 0);
            h0 = (int)(z < i ? z : i);
        }
        int pos = n;   // insertion sort by (lo, hi)
        while (pos > 0 && (lo[pos - 1] > l0 || (lo[pos - 1] == l0 && hi[pos - 1] > h0))) {
            lo[pos] = lo[pos - 1];
            hi[pos] = hi[pos - 1];
            --pos;
        }
        lo[pos] = l0;
        hi[pos] = h0;
        ++n;
    }
    int cnt = 0;
    long long next_free = 0;
    for (int a = 0; a < n; ++a) {
        const int l0 = lo[a], h0 = hi[a];
        const long long j0 = l0 > next_free ? l0 : next_free;
        if (j0 <= h0) {
            // the piece before ends at next_free - 1
            if (cnt > 0 && j0 == next_free && (long long)h0 - lo[cnt - 1] < merge_cap) {
                hi[cnt - 1] = h0;
            } else {
                lo[cnt] = (int)j0;
                hi[cnt] = h0;
                slot[cnt] = cnt;
                ++cnt;
            }
        }
        if ((long long)h0 + 1 > next_free) next_free = (long long)h0 + 1;
    }
    return cnt;
}

// Register-resident form of row_pieces in the per-span mode for at most K - 1 anchors (K intervals with
// the window): every loop is unrolled and nothing is indexed dynamically, so the arrays stay in
// registers.  Same results as row_pieces.  (The union mode has its own streaming builder next to the
// kernel that uses it.)
template <int K>
__device__ __forceinline__ int row_pieces_per_span_small(const int32_t *__restrict__ an, int top_k, long long i,
                                                         long long ell, int back, int fwd, int window, int (&lo)[K],
                                                         int (&hi)[K], int (&slot)[K], int *status) {
    const int w_lo = (int)(i - window + 1 > 0 ? i - window + 1 : 0);
    // intervals in slot order; absent ones are (INT_MAX, -1)
#pragma unroll
    for (int j = 0; j < K; ++j) {
        int l0 = INT_MAX, h0 = -1;
        if (j < top_k) {
            const long long t = an[j];
            if (t > i) {
                atomicOr(status, kStatusBadIndex);
            } else if (t >= 0) {
                const long long a = t - (long long)back * ell, z = t + (long long)fwd * ell;
                l0 = (int)(a > 0 ? a : 0);
                h0 = (int)(z < i ? z : i);
                if (window > 0 && h0 >= w_lo) h0 = w_lo - 1;
                if (l0 > h0) { l0 = INT_MAX; h0 = -1; }
            }
        } else if (j == top_k && window > 0) {
            l0 = w_lo;
            h0 = (int)i;
        }
        lo[j] = l0;
        hi[j] = h0;
        slot[j] = j;
    }
    // pieces keep their slots; compact the present ones to the front, in order
    int cnt = 0;
#pragma unroll
    for (int j = 0; j < K; ++j) {
        const bool on = hi[j] >= 0;
        const int l0 = lo[j], h0 = hi[j];
#pragma unroll
        for (int x = 0; x < K; ++x)
            if (x <= j && on && x == cnt) { lo[x] = l0; hi[x] = h0; slot[x] = j; }
        cnt += on;
    }
    return cnt;
}

// Enqueues the kernels that build the work list of one chunk; adds its launches to *launches.
cudaError_t prepare(const PrepArgs &a, cudaStream_t st, long long *launches);

}  // namespace tc
}  // namespace sla
