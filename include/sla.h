/*
 * sla.h -- C interface of libsla: span-search and span-attention of N=2 Superlinear attention
 *          on NVIDIA B200 (sm_100a).
 *
 * The library computes, for every query position i of a causal sequence:
 *
 *   span-search     (paper: Section "Span search", both equations; Algorithm 1, lines
 *                    "T <- Anchors(i) \ W", "s_t <- <Q_s(i), K_a(t)>", "TopK")
 *       anchors  t_s = i + 1 - (s+1)^2,  s = 0 .. n(i)-1,  n(i) = floor(sqrt(i+1))
 *                (Section "Span attention": anchors at i-(s+1)^{1/p}+1 with p = 1/2)
 *       score    s_{i,t} = search_scale * <Q_s[i], K[t]>          (K_a = K)
 *       select   the top_k anchors with the largest score
 *
 *   span-attention  (paper: Section "Span attention", equation for A_{i,t}; Algorithm 1, lines
 *                    "S_t <- [max(0,t-b l(i)), min(i,t+f l(i))]" and "Attention(Q(i),K[J_t],V[J_t])")
 *       span     S_t = [max(0, t - b*l), min(i, t + f*l)]   closed interval of key positions,
 *                l = span_len if span_len > 0, else ceil(sqrt(i))
 *       output   softmax(softmax_scale * <Q[i], K[j]>) . V over j in the union of the selected
 *                spans (each key counted once), plus lse = log sum_j exp(softmax_scale*<Q[i],K[j]>)
 *
 *   decode step     (paper: Section "Kernel design", paragraph "Decoding path")
 *       the two steps above for the single query i = n_ctx - 1 against a KV cache.
 *
 * Conventions fixed by this library where the paper leaves a choice:
 *   - every anchor with t_s >= 0 is a candidate; ties in the selection go to the smaller s;
 *   - selected anchors are reported by descending score; when fewer than top_k candidates
 *     exist the tail is padded with anchor = -1, score = -inf;
 *   - with grouped-query heads each query head routes on its own against the key head of its
 *     group (kv head = q head / (n_q_heads / n_kv_heads));
 *   - no positional encoding and no padding mask are applied.
 *
 * Memory: unless a parameter says "host", every tensor pointer is DEVICE memory owned by the
 * caller, on the device the handle was created for, which must be the CURRENT device of the calling
 * thread (SLA_ERR_INVALID_ARG otherwise).  The innermost (head_dim) axis is contiguous;
 * the other strides are given in ELEMENTS.  Base pointers must be 16-byte aligned and every stride
 * a multiple of 8 elements.  Calls are asynchronous: work is enqueued on the given CUDA stream
 * (a cudaStream_t passed as void*; NULL = the default stream) and outputs are valid once the stream
 * reaches that point.  The library allocates device memory only in sla_create (the workspace);
 * no call allocates per invocation.  One handle must not be used by two streams at the same time
 * (the workspace is shared); calls that follow each other on different streams are fine as far as the
 * library's own tables go (it orders them itself), the caller orders the tensors.
 *
 * Kernels: bf16 tensors with head_dim 128 whose K/V dimensions nest in memory (no broadcast views)
 * run on the tensor-core kernels (span-attention) and the register-MMA kernel (span-search); every
 * other supported layout -- fp32, head_dim 64, a stride-0 K/V dimension, a single call over more than
 * about 2.6 million keys -- runs on generic fp32-accumulating kernels with the same results and far
 * lower throughput.  The choice depends on shapes and strides alone, never on the workspace size: a
 * workspace too small for the chosen kernel is SLA_ERR_WORKSPACE.
 *
 * Errors: every call returns an sla_status_t; 0 is success, negative values are errors.  When
 * argument validation fails nothing is launched.  No exception or abort crosses this interface.
 * Device-side problems (an anchor outside [0, i] handed to sla_span_attention, an internal bounded
 * wait that ran out) never trap: the kernel records a status word, skips the offending work and
 * returns; sla_poll_status reports it.
 */
#ifndef SLA_H_
#define SLA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    SLA_OK = 0,
    SLA_ERR_INVALID_ARG = -1,    /* NULL pointer, bad shape/stride/alignment, out-of-range value   */
    SLA_ERR_UNSUPPORTED = -2,    /* valid request that this build does not implement              */
    SLA_ERR_WORKSPACE = -3,      /* the handle's workspace is too small for this call             */
    SLA_ERR_CUDA = -4,           /* a CUDA runtime call failed (see sla_last_error)               */
    SLA_ERR_DEVICE_TIMEOUT = -5, /* a bounded device-side wait expired                            */
    SLA_ERR_DEVICE_INDEX = -6,   /* a kernel met an anchor outside [0, i] and skipped it          */
    SLA_ERR_DEVICE_OVERRUN = -7  /* debug canaries: a kernel wrote outside its scratch region      */
} sla_status_t;

typedef enum { SLA_F32 = 0, SLA_BF16 = 1 } sla_dtype_t;

/* SLA_UNION: one softmax over the de-duplicated union of the selected spans and the local window
 * (reduces to dense causal attention when the selection covers every key); sla_span_attention and
 * sla_decode_step.  SLA_PER_SPAN: Algorithm 1 literally, one softmax per selected span united with
 * the window, then the softmax gate of Section "Combination"; sla_span_attention_gated. */
typedef enum { SLA_UNION = 0, SLA_PER_SPAN = 1 } sla_mode_t;

typedef struct sla_handle_s *sla_handle_t; /* opaque; owns the device workspace */

/* Shapes and strides shared by the tensors of one call.
 *   q_s, q, out : [batch, n_q_heads, Lq, head_dim]      strides q_stride_{b,h,t}, head_dim contiguous
 *   k, v        : [batch, n_kv_heads, Lkv.., head_dim]  strides kv_stride_{b,h,t}
 * For sla_decode_step the query tensors are [batch, n_q_heads, head_dim] and q_stride_t is ignored. */
typedef struct {
    int32_t batch, n_q_heads, n_kv_heads; /* n_q_heads % n_kv_heads == 0, group size <= 16        */
    int32_t head_dim;                     /* 64 or 128                                             */
    int32_t dtype;                        /* sla_dtype_t of q_s, q, k, v and out                   */
    int32_t reserved;                     /* must be 0                                             */
    int64_t q_stride_b, q_stride_h, q_stride_t;
    int64_t kv_stride_b, kv_stride_h, kv_stride_t;
} sla_layout_t;

typedef struct {
    int32_t top_k;        /* 1 .. 64                                                              */
    int32_t span_len;     /* l > 0: fixed base span length; 0: l(i) = ceil(sqrt(i)) (Algorithm 1)  */
    int32_t back_factor;  /* b >= 0; b >= 2 is needed for full coverage (Section "Span attention") */
    int32_t fwd_factor;   /* f >= 0                                                               */
    int32_t window;       /* local window w of Algorithm 1: W = [max(0,i-w+1), i]; 0 = none;
                             anchors inside W are no candidates                                  */
    int32_t mode;         /* sla_mode_t                                                           */
    float search_scale;   /* multiplies the search score (the paper's equation has none: 1.0f)    */
    float softmax_scale;  /* multiplies the attention logits ("scaled dot-product": 1/sqrt(D))     */
    double search_exponent; /* p of the stride pattern (Section "Span attention", general p): the
                              stride-s anchor of query i is i + 1 - ceil((s+1)^(1/p)); 0 or 0.5: the
                              exact squares (s+1)^2; else 0.2 .. 0.8                             */
    double span_exponent; /* with span_len = 0: l(i) = ceil(i^span_exponent); 0 or 0.5: the exact
                              integer ceil(sqrt(i)); else 0.2 .. 0.8 (Section "Training": e.g. 1/3 for
                              the search and 2/3 for the spans).  The powers are rounded up after
                              taking off one part in 1e12, so that integer powers stay exact     */
} sla_params_t;

/* ---- handle ------------------------------------------------------------------------------- */

/* Creates a handle on CUDA device `device` and allocates `workspace_bytes` of device scratch memory
 * (the only allocation the library ever makes; ask sla_workspace_bytes for the size).  The handle
 * and its workspace are released by sla_destroy.  *handle is set to NULL on failure. */
sla_status_t sla_create(sla_handle_t *handle, int device, size_t workspace_bytes);
sla_status_t sla_destroy(sla_handle_t handle);

/* Scratch bytes that sla_span_search + sla_span_attention with Lq query rows against Lkv keys, and
 * sla_decode_step at n_ctx = Lkv, need for this layout and these parameters.  Returns 0 when the
 * arguments are invalid.  Host-only: touches no device. */
size_t sla_workspace_bytes(const sla_layout_t *layout, const sla_params_t *params, int64_t Lq,
                           int64_t Lkv);

const char *sla_status_string(sla_status_t status); /* static string, never NULL                  */
const char *sla_last_error(sla_handle_t handle);    /* text of the last failure on this handle     */

/* Waits for `stream` and reads the device status word: SLA_OK, SLA_ERR_DEVICE_OVERRUN,
 * SLA_ERR_DEVICE_TIMEOUT or SLA_ERR_DEVICE_INDEX; the word is cleared. */
sla_status_t sla_poll_status(sla_handle_t handle, void *stream);

/* Number of kernels this handle has launched since sla_create (a diagnostic for benchmarks; the
 * paper has no counterpart).  Host-only. */
int64_t sla_kernel_launches(sla_handle_t handle);

/* Device-side timing of the dominant kernel (a diagnostic for benchmarks; the paper has no
 * counterpart).  With timing enabled, sla_span_attention brackets its main attention kernel with
 * CUDA events on the caller's stream (at most 64 launches are kept between two reads);
 * sla_kernel_time_ms waits for them, returns the summed milliseconds of the launches recorded since
 * the previous read and how many they were (n_launches may be NULL), and starts over. */
sla_status_t sla_set_kernel_timing(sla_handle_t handle, int enable);
sla_status_t sla_kernel_time_ms(sla_handle_t handle, float *ms, int32_t *n_launches);

/* Work statistics of the most recent tensor-core span-attention call of this handle (its last chunk of
 * query positions); a diagnostic for benchmarks, the paper has no counterpart.  out4_host (host memory)
 * receives: tiles of up to 128 pieces, pieces, the sum over tiles of 64-key blocks walked, and the sum
 * over pieces of the blocks their tile walked.  128 x 64 x (third value) is the number of (row, key)
 * products the tensor cores executed, against which the attended pairs measure how well the tiles were
 * packed.  Waits for `stream`. */
sla_status_t sla_attention_tile_stats(sla_handle_t handle, int64_t *out4_host, void *stream);

/* Debug canaries (the paper has no counterpart; they stand in for a memory checker).  When enabled,
 * sla_span_attention, sla_span_attention_gated and sla_decode_step separate the regions of their scratch
 * memory by 256-byte gaps, fill the gaps with a pattern before their kernels run and check them
 * afterwards; a damaged gap shows as SLA_ERR_DEVICE_OVERRUN at the next sla_poll_status.  Costs two
 * small launches per call (per chunk of a chunked call); off by default.
 * sla_selftest_canary_trip damages one gap of the most recent sla_decode_step of this handle itself (a
 * 4-byte memset, nothing out of bounds) and runs the check again, to show that the check reports. */
sla_status_t sla_set_debug_canaries(sla_handle_t handle, int enable);
sla_status_t sla_selftest_canary_trip(sla_handle_t handle, void *stream);

/* Read-only L2 bandwidth probe (a diagnostic for benchmarks; the paper has no counterpart): every CTA of
 * a grid of 4 x SM count reads the whole device buffer `buf` (`bytes`: a multiple of 8192, small enough
 * to stay resident in L2) `iters` times with 32-byte loads, the access width of the span-search kernel,
 * whose roofline this bandwidth is (key rows stream out of L2).  Bytes read by one call:
 * 4 * SM count * bytes * iters.  The caller times the call with CUDA events on `stream`.  `sink`: four
 * bytes of device memory or NULL (never written in practice; it keeps the loads alive). */
sla_status_t sla_probe_l2_read(sla_handle_t handle, const void *buf, size_t bytes, int32_t iters, void *sink,
                               void *stream);

/* Self-test of the bounded device-side wait (the paper has no counterpart).  Launches one warp that polls
 * a barrier nothing ever arrives on, at most `max_polls` (1 .. 10000) times -- no copy and no MMA is in
 * flight -- then records the time-out in the status word, exactly as the tensor-core kernels do when
 * one of their waits runs out, and returns by itself.  The next sla_poll_status reports
 * SLA_ERR_DEVICE_TIMEOUT once; the handle stays usable.  polls_done_device: optional device int that
 * receives the number of polls made. */
sla_status_t sla_selftest_wait_expiry(sla_handle_t handle, int32_t max_polls, int32_t *polls_done_device,
                                      void *stream);

/* The two integer tables the library derives from exponents other than 1/2 (host-only diagnostics, so
 * that the rounding rule stated at sla_params_t can be checked without a device; Section "Span
 * attention", anchors at i - (s+1)^(1/p) + 1, and l(i) proportional to i^p):
 *   sla_pattern_offsets    out[s] = ceil((s+1)^(1/search_exponent)) for every stride with out[s] <= reach
 *   sla_pattern_len_steps  out[v-1] = smallest i >= 1 with ceil(i^span_exponent) >= v, for every v
 *                          reached by some i <= reach
 * Both return the number of entries (only the first `cap` are written; out may be NULL when cap = 0),
 * or -1 for an exponent outside [0.2, 0.8] or more than 65536 entries. */
int32_t sla_pattern_offsets(double search_exponent, int64_t reach, int32_t *out, int32_t cap);
int32_t sla_pattern_len_steps(double span_exponent, int64_t reach, int32_t *out, int32_t cap);

/* ---- span-search (Section "Span search"; Algorithm 1 scoring and TopK lines) -------------- */

/* Query row r (0 <= r < Lq) is position i = q_pos0 + r; keys 0 .. Lkv-1 are valid; requires
 * q_pos0 + Lq <= Lkv.  Full prefill: q_pos0 = 0, Lq = Lkv = L.  A chunk of a chunked prefill:
 * q_pos0 = first position of the chunk.
 *   q_s        in   [B, Hq, Lq, D]  device
 *   k          in   [B, Hkv, >=Lkv, D]  device
 *   out_anchor out  [B, Hq, Lq, top_k] int32, contiguous, device: key positions, best first, -1 pad
 *   out_score  out  [B, Hq, Lq, top_k] fp32,  contiguous, device: matching scores, -inf pad        */
sla_status_t sla_span_search(sla_handle_t handle, const void *q_s, const void *k, int64_t Lq,
                             int64_t q_pos0, int64_t Lkv, const sla_layout_t *layout,
                             const sla_params_t *params, int32_t *out_anchor, float *out_score,
                             void *stream);

/* ---- span-attention (Section "Span attention", equation for A_{i,t}; Algorithm 1 span lines) */

/* The anchors may come from any router; entries < 0 are ignored, entries > i are skipped and
 * flagged (SLA_ERR_DEVICE_INDEX on the next sla_poll_status).  Overlapping spans of one row are
 * attended once.
 *   q          in   [B, Hq, Lq, D] device;  k, v in [B, Hkv, >=Lkv, D] device
 *   anchor     in   [B, Hq, Lq, top_k] int32, contiguous, device
 *   out        out  [B, Hq, Lq, D] in the input dtype, strides as q, device
 *   lse        out  [B, Hq, Lq] fp32, contiguous, device; natural log of the softmax denominator;
 *                   -inf (and out = 0) for a row with no valid anchor                              */
sla_status_t sla_span_attention(sla_handle_t handle, const void *q, const void *k, const void *v,
                                int64_t Lq, int64_t q_pos0, int64_t Lkv, const sla_layout_t *layout,
                                const sla_params_t *params, const int32_t *anchor, void *out,
                                float *lse, void *stream);

/* Algorithm 1 literally (params->mode = SLA_PER_SPAN): for every selected anchor t one softmax over
 * J_t = S_t united with the window W (A_t), then O = sum_t alpha_t A_t with alpha = softmax of the
 * search scores of the selected anchors (Section "Combination"); a row without a valid anchor attends
 * to W alone (out = 0, lse = -inf when there is no window either).
 *   score      in   [B, Hq, Lq, top_k] fp32, contiguous, device: the scores sla_span_search returned
 *   lse        out  [B, Hq, Lq] fp32: log-sum-exp of the first (best-scoring) selected span
 *   lse_span   out  [B, Hq, Lq, top_k] fp32 or NULL: log-sum-exp of every J_t, -inf for padding
 * Other arguments, layouts and errors as for sla_span_attention. */
sla_status_t sla_span_attention_gated(sla_handle_t handle, const void *q, const void *k, const void *v,
                                      int64_t Lq, int64_t q_pos0, int64_t Lkv, const sla_layout_t *layout,
                                      const sla_params_t *params, const int32_t *anchor, const float *score,
                                      void *out, float *lse, float *lse_span, void *stream);

/* ---- decode step (Section "Kernel design", "Decoding path") -------------------------------- */

/* One new token per sequence.  The caller has already appended the token's key and value to the
 * cache: positions 0 .. n_ctx-1 are valid and the query position is i = n_ctx - 1.
 *   q_s, q     in   [B, Hq, D] device (strides q_stride_b, q_stride_h)
 *   k_cache, v_cache in [B, Hkv, capacity >= n_ctx, D] device (kv strides)
 *   out        out  [B, Hq, D] input dtype, strides as q;  lse out [B, Hq] fp32 contiguous
 *   out_anchor out  [B, Hq, top_k] int32 contiguous; out_score out [B, Hq, top_k] fp32 contiguous
 * params->window and params->mode act as in the prefill calls: anchors inside the window are no
 * candidates, the window is attended with the spans; in the SLA_PER_SPAN mode `out` is the gated sum
 * of Algorithm 1 and `lse` the log-sum-exp of the first selected span.                             */
sla_status_t sla_decode_step(sla_handle_t handle, const void *q_s, const void *q, const void *k_cache,
                             const void *v_cache, int64_t n_ctx, const sla_layout_t *layout,
                             const sla_params_t *params, void *out, float *lse, int32_t *out_anchor,
                             float *out_score, void *stream);

/* ---- decode step without any allocation ---------------------------------------------------- */

/* (The paper has no counterpart: this entry point exists for the sake of the hosts of this library.)
 *
 * sla_decode_step for callers that may not allocate device memory -- code running under a stream
 * capture or inside a serving loop that forbids cudaMalloc, processes whose device memory has been
 * handed in full to another allocator, plug-ins that are lent a stream and nothing else.  Such
 * callers cannot call sla_create, because the handle's workspace is a cudaMalloc.  This call needs no
 * handle: its scratch (anchor scores, clipped spans, split results, completion counters) is a fixed
 * array of SLA_STATIC_SCRATCH_BYTES inside the library image, which every GPU that loads the library
 * holds until the process exits.  The call allocates nothing and frees nothing, on the host's heap
 * or on the device.
 *
 * Arguments, results and launch behaviour are those of sla_decode_step (same kernels); inputs and
 * outputs are still the caller's device buffers.  Differences:
 *   - only the union mode without a local window and with the exponents of the quadratic pattern
 *     (params->window = 0, params->mode = SLA_UNION, search_exponent and span_exponent 0 or 0.5: other
 *     exponents need tables that live in a handle's workspace); anything else returns
 *     SLA_ERR_UNSUPPORTED;
 *   - a step whose scratch exceeds the fixed array (it grows with batch * heads * sqrt(n_ctx) and
 *     with batch * heads * splits) is rejected with SLA_ERR_WORKSPACE and nothing is launched; the
 *     1M- and 10M-token configurations with 32 query heads need well under 1 MiB;
 *   - set-up happens inside the call, not at load time: the first call on a device resolves the
 *     array's device address (once per device, with that device current); the first call for each
 *     (device, dtype, head_dim) asks the device for its SM count and the kernel's occupancy.  Make one
 *     call per (device, dtype, head_dim) before any stream capture;
 *   - all calls on one device share the array: it keeps the previous call's contents (the part that
 *     must start at zero is cleared on the stream at the start of each call), and two calls that
 *     overlap on the GPU -- different streams, or several threads -- race on it.  Serialise them.
 *   - there is no handle to hold an error text: the status code is all there is
 *     (SLA_ERR_INVALID_ARG, SLA_ERR_UNSUPPORTED, SLA_ERR_WORKSPACE as above, SLA_ERR_CUDA). */
#define SLA_STATIC_SCRATCH_BYTES (2u << 20)
sla_status_t sla_decode_step_static(const void *q_s, const void *q, const void *k_cache, const void *v_cache,
                                    int64_t n_ctx, const sla_layout_t *layout, const sla_params_t *params,
                                    void *out, float *lse, int32_t *out_anchor, float *out_score, void *stream);

/* ---- sequence-sharded decode step --------------------------------------------------------------
 *
 * For a KV cache that is split across devices by position: rank r holds the keys and values of the
 * contiguous positions [shard_lo, shard_lo + shard_len) of every sequence, as tensors
 * [B, Hkv, >= shard_len, D] whose index 0 is position shard_lo (kv strides of the layout).  One decode
 * step is three calls per rank with two small exchanges between them, which the caller carries out
 * (an all-gather each; the Python package does them with torch.distributed):
 *
 *   1. sla_decode_shard_search: scores the anchors of query position n_ctx - 1 that fall into this
 *      rank's range and returns its top_k best (global positions, -1 / -inf padding)       -> gather
 *   2. sla_decode_shard_attend: from the candidates of all ranks [n_shards, B, Hq, top_k] picks the
 *      global top_k (the selection of the unsharded step: larger score first, then the nearer
 *      anchor), builds their spans (Algorithm 1), attends to the part inside this rank's range and
 *      returns out_anchor / out_score (the same on every rank) and `partial`
 *      [B, Hq, D + 2] fp32 = {log-sum-exp, 0, normalised output} of its part                -> gather
 *   3. sla_decode_shard_merge: merges the partial results of all ranks [n_shards, B, Hq, D + 2]
 *      through their log-sum-exp into out [B, Hq, D] (input dtype, q strides) and lse [B, Hq].
 *
 * The result equals sla_decode_step on the whole cache (Section "Kernel design", "Decoding path").
 * Union mode without a local window; q_s, q as for sla_decode_step; positions >= n_ctx of a range are
 * ignored.  All pointers are device memory of this rank. */
sla_status_t sla_decode_shard_search(sla_handle_t handle, const void *q_s, const void *k_local,
                                     int64_t shard_lo, int64_t shard_len, int64_t n_ctx,
                                     const sla_layout_t *layout, const sla_params_t *params,
                                     int32_t *cand_anchor, float *cand_score, void *stream);
sla_status_t sla_decode_shard_attend(sla_handle_t handle, const void *q, const void *k_local,
                                     const void *v_local, int64_t shard_lo, int64_t shard_len, int64_t n_ctx,
                                     const sla_layout_t *layout, const sla_params_t *params, int32_t n_shards,
                                     const int32_t *all_anchor, const float *all_score, int32_t *out_anchor,
                                     float *out_score, float *partial, void *stream);
sla_status_t sla_decode_shard_merge(sla_handle_t handle, int32_t n_shards, const float *all_partial,
                                    const sla_layout_t *layout, void *out, float *lse, void *stream);

/* ---- host-buffer convenience calls ---------------------------------------------------------- */

/* sla_span_search followed by sla_span_attention on HOST buffers (pinned memory gives the best
 * copy rate): copies q_s, q, k, v to the device, runs both steps, copies out, lse, anchors and
 * scores back, and waits for completion.  Sequences of 4096 tokens and more go through in up to
 * thirty-two chunks of query positions (chunked prefill: a chunk needs the keys up to its own end), with
 * the copy-in of the next chunk, the kernels of this one and the copy-out of the previous one
 * overlapping on streams the handle owns; results do not depend on the chunking.  Union mode only.
 * All tensors are dense and contiguous
 * ([B,Hq,L,D] / [B,Hkv,L,D], q_pos0 = 0, Lq = Lkv = L); the layout's strides are ignored.  The
 * device staging buffers come out of the handle's workspace, which therefore has to be
 * sla_workspace_bytes(...) + sla_host_staging_bytes(...) large.  Section references as above. */
size_t sla_host_staging_bytes(const sla_layout_t *layout, const sla_params_t *params, int64_t L);
sla_status_t sla_prefill_host(sla_handle_t handle, const void *q_s_host, const void *q_host,
                              const void *k_host, const void *v_host, int64_t L,
                              const sla_layout_t *layout, const sla_params_t *params, void *out_host,
                              float *lse_host, int32_t *anchor_host, float *score_host, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* SLA_H_ */
