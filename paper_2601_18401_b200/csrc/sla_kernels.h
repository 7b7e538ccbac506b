// Internal launcher declarations of libsla (the public interface is include/sla.h).
#pragma once

#include "sla_common.cuh"

namespace sla {

// ---- generic SIMT kernels (sla_simt.cu) --------------------------------------------------------
cudaError_t launch_search_simt(const void *q_s, const void *k, const Call &c, int dtype,
                               int32_t *out_anchor, float *out_score, cudaStream_t st);
cudaError_t launch_attn_simt(const void *q, const void *k, const void *v, const Call &c, int dtype,
                             const int32_t *anchor, const float *score, void *out, float *lse, float *lse_span,
                             cudaStream_t st);

// Optional device-side timing of the dominant kernel of a call (CUDA events on the caller's stream).
struct KernelTimer {
    static constexpr int kMaxPairs = 64;
    bool enabled = false;
    int used = 0;                       // event pairs recorded by the last call
    cudaEvent_t ev[2 * kMaxPairs] = {};
    void begin(cudaStream_t st) { if (enabled && used < kMaxPairs) cudaEventRecord(ev[2 * used], st); }
    void end(cudaStream_t st) { if (enabled && used < kMaxPairs) { cudaEventRecord(ev[2 * used + 1], st); ++used; } }
};

// Debug canaries: with a gap of kBytes between the regions of a call's scratch memory (and before the
// first and after the last), filled with a pattern before the kernels run and checked after them, a
// kernel that writes outside its region is reported through the status word instead of going unnoticed.
struct Canaries {
    static constexpr int kMax = 16;
    static constexpr size_t kBytes = 256;
    size_t at[kMax] = {};   // byte offsets of the gaps from the scratch base
    int n = 0;
    void add(size_t off) { if (n < kMax) at[n++] = off; }
};
cudaError_t launch_canary_fill(void *scratch, const Canaries &cn, cudaStream_t st);
cudaError_t launch_canary_check(const void *scratch, const Canaries &cn, int *status, cudaStream_t st);

// ---- tensor-core span-search for bf16 / head_dim 128 (sla_search_mma.cu) -------------------------
bool search_mma_supported(const Call &c, int dtype);
cudaError_t launch_search_mma(const void *q_s, const void *k, const Call &c, int32_t *out_anchor, float *out_score,
                              cudaStream_t st, long long *launches);

// ---- span-search with the selection folded into the scoring loop, bf16 / head_dim 128 / groups of four
// query heads (sla_search_diag.cu)
bool search_diag_supported(const Call &c, int dtype);
cudaError_t launch_search_diag(const void *q_s, const void *k, const Call &c, int32_t *out_anchor, float *out_score,
                               cudaStream_t st, long long *launches);

// ---- tensor-core span-attention for prefill, bf16 / head_dim 128 (sla_attn_tc.cu) ---------------
// Scratch layout for one chunk of Lc query positions (all offsets in bytes).
struct TcPlan {
    int Lc, n_bg, NB, nb_max, nb_single, ncls, ncls1, merge_cap, ctas_per_bg;
    int slots;   // partial results per query row: top_k, plus one for the local window
    bool ok;   // false when the shared-memory histogram of the counting sort cannot hold NB buckets
    long long max_tiles;
    size_t off_counters, off_key_count, off_key_cursor, off_cta_hist, off_tiles, off_recs, off_npieces, off_part_lse,
        off_part_o, bytes;
    Canaries canaries;
};
bool tc_attention_shape_ok(const Call &c, int dtype);  // host-only shape test
bool tc_attention_supported(const Call &c, int dtype); // shape test + driver entry point present
TcPlan plan_attention_tc(const Call &c, int Lc, size_t gap = 0);   // gap: bytes of canary between regions
// Where the tile table of the most recent chunk lives (for sla_attention_tile_stats).
struct TcLast { const int4 *tiles = nullptr; const int *n_tiles = nullptr; };
cudaError_t launch_tile_stats(const TcLast &last, long long *out4_device, cudaStream_t st);
// Splits the query rows into chunks whose scratch fits `scratch_bytes`; adds its kernel launches to
// *launches.  Returns cudaErrorMemoryAllocation when not even one query position fits.
cudaError_t launch_attn_tc(const void *q, const void *k, const void *v, const Call &c, const int32_t *anchor, const float *score,
                           void *out, float *lse, float *lse_span, void *scratch, size_t scratch_bytes, int sm_count,
                           cudaStream_t st, long long *launches, KernelTimer *timer, bool canaries = false,
                           TcLast *last = nullptr);

// ---- decode step (sla_decode.cu) ---------------------------------------------------------------
// Scratch layout of one decode step, all offsets in bytes from the scratch base.
struct DecodePlan {
    int n_anchor;       // anchor candidates of the query position: floor(sqrt(n_ctx)) - floor(sqrt(window))
    int n_splits;       // CTAs that share one attention unit's tokens (unit: a head, or one selected
                        // anchor of a head in the per-span mode)
    size_t off_scores;  // float [B*Hq][n_anchor]
    size_t off_spans;   // int   [units][2*P + 2]: piece starts, cumulative token counts, piece count
                        //       (P = top_k + 1 in the union mode, 2 in the per-span mode)
    size_t off_partial; // float [units][n_splits][D + 2]: running max, denominator, numerator
    size_t off_unit_out; // float [units][D + 2] (per-span mode): log-sum-exp and output of every unit
    size_t bytes;
    Canaries canaries;
};
// cta_slots = SM count x resident decode_attn CTAs per SM (see decode_attn_blocks_per_sm)
DecodePlan plan_decode(const Call &c, long long n_ctx, int cta_slots, size_t gap = 0);
int decode_attn_blocks_per_sm(int dtype, int D);
// counters: B*Hkv + B*Hq*units + B*Hq ints (units = top_k in the per-span mode, else 1), zero on entry
// and zero again on exit (completion counters)
cudaError_t launch_decode(const void *q_s, const void *q, const void *k, const void *v, const Call &c,
                          int dtype, long long n_ctx, const DecodePlan &plan, void *scratch, int *counters,
                          void *out, float *lse, int32_t *out_anchor, float *out_score, cudaStream_t st);

// Sequence-sharded decode step (sla_decode.cu): local candidates of one rank, global selection +
// attention over this rank's part of the spans, merge of the ranks' partial results.
cudaError_t launch_decode_shard_search(const void *q_s, const void *k_local, const Call &c, int dtype,
                                       long long n_ctx, int s_first, int n, void *scratch, int *counters,
                                       int32_t *cand_anchor, float *cand_score, cudaStream_t st);
cudaError_t launch_decode_shard_attend(const void *q, const void *k_local, const void *v_local, const Call &c,
                                       int dtype, long long n_ctx, const DecodePlan &plan, void *scratch,
                                       int *counters, int n_shards, const int32_t *all_anchor,
                                       const float *all_score, int32_t *out_anchor, float *out_score,
                                       float *partial_out, cudaStream_t st);
cudaError_t launch_decode_shard_merge(const float *all_partial, int n_shards, const Call &c, int dtype, void *out,
                                      float *lse, cudaStream_t st);

// ---- diagnostics (sla_diag.cu)
cudaError_t launch_probe_l2_read(const void *buf, size_t bytes, int iters, int n_ctas, unsigned *sink, cudaStream_t st);
cudaError_t launch_selftest_wait_expiry(int max_polls, int *status, int *polls_done, cudaStream_t st);

// argument checks of a decode step without a handle (defined in sla_api.cu)
sla_status_t check_decode_args(const void *q_s, const void *q, const void *k_cache, const void *v_cache,
                               int64_t n_ctx, const sla_layout_t *l, const sla_params_t *p, const void *out,
                               const float *lse, const int32_t *out_anchor, const float *out_score, Call *c_out);

}  // namespace sla
