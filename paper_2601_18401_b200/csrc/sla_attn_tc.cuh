// Definitions shared by the tensor-core span-attention kernel (sla_attn_tc.cu) and the kernels that
// prepare its work list (sla_attn_prep.cu).  Internal to libsla.
#pragma once

#include "sla_kernels.h"

namespace sla {
namespace tc {

constexpr int kBK = 64;     // keys per block
constexpr int kRows = 128;  // pieces per tile

// Work list of one chunk of query positions, as laid out in the scratch memory:
//   recs   int4 {row, piece index j, lo, hi}: every piece of every row, ordered by
//          (batch*Hkv + kv head, 64-key block of hi, class of blocks covered)
//   tiles  int4 {batch*Hkv + kv head, end block, first record, records | key blocks to walk << 8}
//   n_tiles, n_pieces[row], and the per-piece partial results
struct PrepArgs {
    const int32_t *anchor;   // [B,Hq,Lq,top_k]
    int B, Hq, Hkv, G, top_k, span_len, back, fwd;
    long long Lq, q_pos0, r0;
    int Lc;                  // query positions in this chunk
    int NB;                  // 64-key blocks in [0, Lkv)
    int nb_max;              // most blocks a piece can cover
    int ncls;                // classes of "blocks covered" the pieces are ordered by inside a group
    int ctas_per_bg;         // CTAs that share the rows of one (batch, kv head)
    int *key_count;          // [B*Hkv][NB*ncls]: histogram, then exclusive offsets
    int *key_cursor;         // same shape
    int *totals;             // [B*Hkv][2]: records and tiles of each (batch, kv head)
    int *n_tiles;            // total number of tiles
    int4 *tiles;
    int max_tiles;
    int4 *recs;
    unsigned char *n_pieces; // [rows]
    int *status;
};

// Pieces of one row: spans of the selected anchors (Algorithm 1: S_t = [max(0,t-b l), min(i,t+f l)]),
// sorted by (lo, hi), clipped so that each key is kept once.  Returns the number of pieces;
// lo[]/hi[] hold them left to right.
__device__ inline int row_pieces(const int32_t *__restrict__ an, int top_k, long long i, long long ell,
                                 int back, int fwd, int *lo, int *hi, int *status) {
    int n = 0;
    for (int j = 0; j < top_k; ++j) {
        const long long t = an[j];
        if (t > i) { atomicOr(status, kStatusBadIndex); continue; }
        if (t < 0) continue;
        const long long a = t - (long long)back * ell, z = t + (long long)fwd * ell;
        const int l0 = (int)(a > 0 ? a : 0), h0 = (int)(z < i ? z : i);
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
            lo[cnt] = (int)j0;
            hi[cnt] = h0;
            ++cnt;
        }
        if ((long long)h0 + 1 > next_free) next_free = (long long)h0 + 1;
    }
    return cnt;
}

// Enqueues the kernels that build the work list of one chunk; adds its launches to *launches.
cudaError_t prepare(const PrepArgs &a, cudaStream_t st, long long *launches);

}  // namespace tc
}  // namespace sla
