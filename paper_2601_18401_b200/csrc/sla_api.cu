// Host side of libsla: handle, argument validation, workspace carving and kernel dispatch.
// Every exported function is declared and documented in include/sla.h.
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <new>
#include <vector>

#include "sla_kernels.h"

struct sla_handle_s {
    int device = 0;
    int sm_count = 0;
    char *ws = nullptr;       // device workspace; the first kHeaderBytes hold the status word
    size_t ws_bytes = 0;
    long long launches = 0;   // kernels launched through this handle
    size_t scratch_avail = 0; // bytes of workspace after the header that kernels may use as scratch
    sla::KernelTimer timer;   // sla_set_kernel_timing / sla_kernel_time_ms
    sla::TcLast tc_last;      // tile table of the most recent tensor-core attention chunk
    bool canaries = false;    // sla_set_debug_canaries
    sla::Canaries last_canaries;   // of the most recent call that laid any, and where its scratch began
    char *last_canary_base = nullptr;
    // stride-offset and span-length tables for exponents other than 1/2 (host copies; the device
    // copies sit in the workspace header) and what they were built for
    std::vector<int> off_host, len_host;
    double off_p = 0.0, len_p = 0.0;
    long long off_reach = 0, len_reach = 0;
    // the device copies are enqueued on the stream of the call that built them: a later call on another
    // stream waits for this event before its kernels read the tables
    cudaEvent_t tbl_ev = nullptr;
    cudaStream_t tbl_stream = nullptr;
    // sla_prefill_host: copy-in and copy-out streams and per-chunk events, created on first use
    static constexpr int kMaxChunks = 32;
    cudaStream_t s_in = nullptr, s_out = nullptr;
    cudaEvent_t ev_fork = nullptr, ev_join = nullptr, ev_in[kMaxChunks] = {}, ev_done[kMaxChunks] = {};
    char err[256] = {0};
};

namespace {

// header of the workspace: status word at 0, completion counters of the decode step from byte 256,
// then the two pattern tables (stride offsets, span-length steps) of kMaxTable ints each
constexpr size_t kCounterEnd = 64 * 1024;
constexpr int kMaxTable = 65536;
constexpr size_t kOffTableAt = kCounterEnd, kLenTableAt = kCounterEnd + (size_t)kMaxTable * 4;
constexpr size_t kHeaderBytes = kCounterEnd + 2 * (size_t)kMaxTable * 4;
constexpr size_t kCounterOffset = 256;

sla_status_t fail(sla_handle_t h, sla_status_t code, const char *fmt, const char *detail = "") {
    if (h) snprintf(h->err, sizeof h->err, fmt, detail);
    return code;
}

sla_status_t cuda_fail(sla_handle_t h, cudaError_t e, const char *where) {
    if (h) snprintf(h->err, sizeof h->err, "%s: %s", where, cudaGetErrorString(e));
    return SLA_ERR_CUDA;
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Checks that do not depend on the call: layout and parameters.  Returns NULL when fine, else why.
const char *check_layout_params(const sla_layout_t *l, const sla_params_t *p, bool decode) {
    if (!l || !p) return "layout or params is NULL";
    if (l->batch <= 0 || l->n_q_heads <= 0 || l->n_kv_heads <= 0) return "batch and head counts must be positive";
    if (l->n_q_heads % l->n_kv_heads) return "n_q_heads must be a multiple of n_kv_heads";
    if (l->n_q_heads / l->n_kv_heads > sla::kMaxGroup) return "group size above 16";
    if (l->head_dim != 64 && l->head_dim != 128) return "head_dim must be 64 or 128";
    if (l->dtype != SLA_F32 && l->dtype != SLA_BF16) return "dtype must be SLA_F32 or SLA_BF16";
    if (l->reserved != 0) return "reserved must be 0";
    const int64_t strides[6] = {l->q_stride_b, l->q_stride_h, l->q_stride_t,
                                l->kv_stride_b, l->kv_stride_h, l->kv_stride_t};
    for (int j = 0; j < 6; ++j) {
        if (decode && j == 2) continue;
        if (strides[j] < 0 || strides[j] % 8) return "strides must be non-negative multiples of 8 elements";
    }
    if ((!decode && l->q_stride_t < l->head_dim) || l->kv_stride_t < l->head_dim) return "token stride below head_dim";
    if (p->top_k < 1 || p->top_k > sla::kMaxTopK) return "top_k must be in 1..64";
    if (p->span_len < 0 || p->back_factor < 0 || p->fwd_factor < 0) return "span_len and factors must be >= 0";
    if (p->window < 0) return "window must be >= 0";
    if (p->mode != SLA_UNION && p->mode != SLA_PER_SPAN) return "mode must be SLA_UNION or SLA_PER_SPAN";
    if (!(p->softmax_scale == p->softmax_scale) || !(p->search_scale == p->search_scale)) return "scale is NaN";
    for (double e : {p->search_exponent, p->span_exponent})
        if (!(e == 0.0 || (e >= 0.2 && e <= 0.8))) return "exponents must be 0 (= 1/2) or in [0.2, 0.8]";
    return nullptr;
}

// ceil of base^expo, after taking off one part in 1e12: a power that is an integer in exact arithmetic
// (exponent 1/3: cubes) must not be pushed to the next integer by the rounding of 1/p and of pow.
long long ceil_pow(double base, double expo) {
    const double x = pow(base, expo);
    return (long long)ceil(x - 1e-12 * x);
}

bool is_half(double p) { return p == 0.0 || p == 0.5; }

// off[s] = ceil((s+1)^(1/p)) for every stride whose offset is <= reach.  False when there are too many.
bool build_offsets(double p, long long reach, std::vector<int> &off) {
    off.clear();
    for (long long s = 0;; ++s) {
        const long long o = ceil_pow((double)(s + 1), 1.0 / p);
        if (o > reach) break;
        if ((int)off.size() >= kMaxTable) return false;
        off.push_back((int)o);
    }
    return true;
}

// len_first[v-1] = smallest i >= 1 with ceil(i^p) >= v, for every v reached by some i <= reach.
bool build_len_first(double p, long long reach, std::vector<int> &lf) {
    lf.clear();
    long long i = 1;
    for (long long v = 1;; ++v) {
        // l is non-decreasing and grows by at most 1 per position: start near (v-1)^(1/p) and settle
        long long g = (long long)floor(pow((double)(v - 1), 1.0 / p)) - 2;
        if (g > i) i = g;
        while (i <= reach && ceil_pow((double)i, p) < v) ++i;
        if (i > reach) break;
        if ((int)lf.size() >= kMaxTable) return false;
        lf.push_back((int)i);
    }
    return true;
}

// Kernels are launched on the current device: it has to be the one the handle was created on.
const char *check_device(const sla_handle_t h) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev != h->device) return "the handle's device is not the current device";
    return nullptr;
}

sla::Call make_call(const sla_handle_t h, const sla_layout_t *l, const sla_params_t *p, int64_t Lq,
                    int64_t q_pos0, int64_t Lkv) {
    sla::Call c;
    c.B = l->batch; c.Hq = l->n_q_heads; c.Hkv = l->n_kv_heads; c.D = l->head_dim;
    c.G = l->n_q_heads / l->n_kv_heads;
    c.q_sb = l->q_stride_b; c.q_sh = l->q_stride_h; c.q_st = l->q_stride_t;
    c.kv_sb = l->kv_stride_b; c.kv_sh = l->kv_stride_h; c.kv_st = l->kv_stride_t;
    c.Lq = Lq; c.q_pos0 = q_pos0; c.Lkv = Lkv;
    c.top_k = p->top_k; c.span_len = p->span_len; c.back = p->back_factor; c.fwd = p->fwd_factor;
    c.window = p->window; c.mode = p->mode;
    c.search_scale = p->search_scale; c.softmax_scale = p->softmax_scale;
    c.status = h ? reinterpret_cast<int *>(h->ws) : nullptr;
    c.off = c.off_host = c.len_first = c.len_first_host = nullptr;
    c.n_off = c.n_len = 0;
    c.shard_lo = 0;
    c.shard_hi = Lkv;
    if (h && !is_half(p->search_exponent)) {
        c.off = reinterpret_cast<const int *>(h->ws + kOffTableAt);
        c.off_host = h->off_host.data();
        c.n_off = (int)h->off_host.size();
    }
    if (h && !is_half(p->span_exponent) && p->span_len == 0) {
        c.len_first = reinterpret_cast<const int *>(h->ws + kLenTableAt);
        c.len_first_host = h->len_host.data();
        c.n_len = (int)h->len_host.size();
    }
    return c;
}

// Builds (or reuses) the handle's pattern tables for this call's exponents and key range and puts
// the device copies in place on `st`.  Must run before make_call.
sla_status_t prepare_pattern(sla_handle_t h, const sla_params_t *p, int64_t Lkv, cudaStream_t st) {
    const bool need_off = !is_half(p->search_exponent), need_len = !is_half(p->span_exponent) && p->span_len == 0;
    if (!need_off && !need_len) return SLA_OK;
    bool copied = false;
    if (!is_half(p->search_exponent) && (h->off_p != p->search_exponent || h->off_reach < Lkv)) {
        if (!build_offsets(p->search_exponent, Lkv, h->off_host))
            return fail(h, SLA_ERR_UNSUPPORTED, "search_exponent gives more than 65536 strides for this length%s");
        h->off_p = p->search_exponent;
        h->off_reach = Lkv;
        if (!h->off_host.empty() &&
            cudaMemcpyAsync(h->ws + kOffTableAt, h->off_host.data(), h->off_host.size() * 4, cudaMemcpyHostToDevice, st) != cudaSuccess)
            return fail(h, SLA_ERR_CUDA, "copying the stride table failed%s");
        copied = true;
    }
    if (!is_half(p->span_exponent) && p->span_len == 0 && (h->len_p != p->span_exponent || h->len_reach < Lkv)) {
        if (!build_len_first(p->span_exponent, Lkv, h->len_host))
            return fail(h, SLA_ERR_UNSUPPORTED, "span_exponent gives base lengths above 65536 for this length%s");
        h->len_p = p->span_exponent;
        h->len_reach = Lkv;
        if (!h->len_host.empty() &&
            cudaMemcpyAsync(h->ws + kLenTableAt, h->len_host.data(), h->len_host.size() * 4, cudaMemcpyHostToDevice, st) != cudaSuccess)
            return fail(h, SLA_ERR_CUDA, "copying the span-length table failed%s");
        copied = true;
    }
    if (copied) {
        if (!h->tbl_ev && cudaEventCreateWithFlags(&h->tbl_ev, cudaEventDisableTiming) != cudaSuccess)
            return fail(h, SLA_ERR_CUDA, "creating the table event failed%s");
        if (cudaEventRecord(h->tbl_ev, st) != cudaSuccess) return fail(h, SLA_ERR_CUDA, "recording the table event failed%s");
        h->tbl_stream = st;
    } else if (h->tbl_ev && st != h->tbl_stream) {
        if (cudaStreamWaitEvent(st, h->tbl_ev, 0) != cudaSuccess) return fail(h, SLA_ERR_CUDA, "waiting for the tables failed%s");
    }
    return SLA_OK;
}

const char *check_prefill_range(int64_t Lq, int64_t q_pos0, int64_t Lkv) {
    if (Lq <= 0 || q_pos0 < 0 || Lkv <= 0) return "Lq, Lkv must be positive and q_pos0 >= 0";
    if (q_pos0 + Lq > Lkv) return "q_pos0 + Lq exceeds Lkv";
    if (Lkv > 2147483647LL) return "Lkv above 2^31-1";
    return nullptr;
}

size_t elem_size(int dtype) { return dtype == SLA_F32 ? 4 : 2; }

}  // namespace

namespace sla {

// Argument checks of a decode step for callers that have no handle (the no-allocation entry point
// in sla_decode.cu): same rules as sla_decode_step.  Fills *c_out on success.
sla_status_t check_decode_args(const void *q_s, const void *q, const void *k_cache, const void *v_cache,
                               int64_t n_ctx, const sla_layout_t *l, const sla_params_t *p, const void *out,
                               const float *lse, const int32_t *out_anchor, const float *out_score, Call *c_out) {
    if (check_layout_params(l, p, true)) return SLA_ERR_INVALID_ARG;
    if (n_ctx <= 0 || n_ctx > 2147483647LL) return SLA_ERR_INVALID_ARG;
    if (!q_s || !q || !k_cache || !v_cache || !out || !lse || !out_anchor || !out_score) return SLA_ERR_INVALID_ARG;
    if (!aligned16(q_s) || !aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(out))
        return SLA_ERR_INVALID_ARG;
    if (p->window != 0 || p->mode != SLA_UNION || !is_half(p->search_exponent) || !is_half(p->span_exponent))
        return SLA_ERR_UNSUPPORTED;
    *c_out = make_call(nullptr, l, p, 1, n_ctx - 1, n_ctx);
    return SLA_OK;
}

}  // namespace sla

extern "C" {

const char *sla_status_string(sla_status_t s) {
    switch (s) {
        case SLA_OK: return "SLA_OK";
        case SLA_ERR_INVALID_ARG: return "SLA_ERR_INVALID_ARG";
        case SLA_ERR_UNSUPPORTED: return "SLA_ERR_UNSUPPORTED";
        case SLA_ERR_WORKSPACE: return "SLA_ERR_WORKSPACE";
        case SLA_ERR_CUDA: return "SLA_ERR_CUDA";
        case SLA_ERR_DEVICE_TIMEOUT: return "SLA_ERR_DEVICE_TIMEOUT";
        case SLA_ERR_DEVICE_INDEX: return "SLA_ERR_DEVICE_INDEX";
        case SLA_ERR_DEVICE_OVERRUN: return "SLA_ERR_DEVICE_OVERRUN";
    }
    return "SLA_ERR_UNKNOWN";
}

const char *sla_last_error(sla_handle_t h) { return h ? h->err : "NULL handle"; }

int64_t sla_kernel_launches(sla_handle_t h) { return h ? h->launches : 0; }

sla_status_t sla_set_kernel_timing(sla_handle_t h, int enable) {
    if (!h) return SLA_ERR_INVALID_ARG;
    if (enable && !h->timer.ev[0]) {
        for (int j = 0; j < 2 * sla::KernelTimer::kMaxPairs; ++j)
            if (cudaEventCreate(&h->timer.ev[j]) != cudaSuccess) return cuda_fail(h, cudaGetLastError(), "sla_set_kernel_timing");
    }
    h->timer.enabled = enable != 0;
    h->timer.used = 0;
    return SLA_OK;
}

sla_status_t sla_kernel_time_ms(sla_handle_t h, float *ms, int32_t *n_launches) {
    if (!h || !ms) return SLA_ERR_INVALID_ARG;
    *ms = 0.f;
    if (n_launches) *n_launches = h->timer.used;
    for (int j = 0; j < h->timer.used; ++j) {
        float t = 0.f;
        cudaError_t e = cudaEventSynchronize(h->timer.ev[2 * j + 1]);
        if (e == cudaSuccess) e = cudaEventElapsedTime(&t, h->timer.ev[2 * j], h->timer.ev[2 * j + 1]);
        if (e != cudaSuccess) return cuda_fail(h, e, "sla_kernel_time_ms");
        *ms += t;
    }
    h->timer.used = 0;
    return SLA_OK;
}

int32_t sla_pattern_offsets(double p, int64_t reach, int32_t *out, int32_t cap) {
    if (!(p >= 0.2 && p <= 0.8) || reach < 0 || cap < 0 || (cap > 0 && !out)) return -1;
    std::vector<int> t;
    if (!build_offsets(p, reach, t)) return -1;
    for (int j = 0; j < cap && j < (int)t.size(); ++j) out[j] = t[j];
    return (int32_t)t.size();
}

int32_t sla_pattern_len_steps(double p, int64_t reach, int32_t *out, int32_t cap) {
    if (!(p >= 0.2 && p <= 0.8) || reach < 0 || cap < 0 || (cap > 0 && !out)) return -1;
    std::vector<int> t;
    if (!build_len_first(p, reach, t)) return -1;
    for (int j = 0; j < cap && j < (int)t.size(); ++j) out[j] = t[j];
    return (int32_t)t.size();
}

sla_status_t sla_attention_tile_stats(sla_handle_t h, int64_t *out4_host, void *stream) {
    if (!h || !out4_host) return SLA_ERR_INVALID_ARG;
    if (!h->tc_last.tiles) return fail(h, SLA_ERR_INVALID_ARG, "no tensor-core span-attention has run on this handle%s");
    if (const char *why = check_device(h)) return fail(h, SLA_ERR_INVALID_ARG, "%s", why);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // four counters in the status header's spare space (bytes 64..95 of the workspace)
    long long *dev = reinterpret_cast<long long *>(h->ws + 64);
    cudaError_t e = sla::launch_tile_stats(h->tc_last, dev, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(out4_host, dev, 4 * sizeof(long long), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(h, e, "sla_attention_tile_stats");
    return SLA_OK;
}

sla_status_t sla_set_debug_canaries(sla_handle_t h, int enable) {
    if (!h) return SLA_ERR_INVALID_ARG;
    h->canaries = enable != 0;
    h->last_canaries = sla::Canaries();
    h->last_canary_base = nullptr;
    return SLA_OK;
}

sla_status_t sla_selftest_canary_trip(sla_handle_t h, void *stream) {
    if (!h) return SLA_ERR_INVALID_ARG;
    if (!h->last_canary_base || h->last_canaries.n == 0)
        return fail(h, SLA_ERR_INVALID_ARG, "no decode step with canaries has run on this handle%s");
    if (const char *why = check_device(h)) return fail(h, SLA_ERR_INVALID_ARG, "%s", why);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // what an overrun of the first scratch region by one word would leave behind
    cudaError_t e = cudaMemsetAsync(h->last_canary_base + h->last_canaries.at[1], 0, 4, st);
    if (e == cudaSuccess) e = sla::launch_canary_check(h->last_canary_base, h->last_canaries, reinterpret_cast<int *>(h->ws), st);
    if (e != cudaSuccess) return cuda_fail(h, e, "sla_selftest_canary_trip");
    return SLA_OK;
}

sla_status_t sla_probe_l2_read(sla_handle_t h, const void *buf, size_t bytes, int32_t iters, void *sink, void *stream) {
    if (!h) return SLA_ERR_INVALID_ARG;
    if (!buf || !aligned16(buf) || (reinterpret_cast<uintptr_t>(buf) & 31u) || iters < 1 || iters > 4096)
        return fail(h, SLA_ERR_INVALID_ARG, "probe buffer must be 32-byte aligned, iters in 1..4096%s");
    if (bytes < 8192 || bytes % 8192 || bytes > ((size_t)1 << 32))
        return fail(h, SLA_ERR_INVALID_ARG, "probe size must be a multiple of 8192 bytes, at most 4 GiB%s");
    if (const char *why = check_device(h)) return fail(h, SLA_ERR_INVALID_ARG, "%s", why);
    cudaError_t e = sla::launch_probe_l2_read(buf, bytes, iters, 4 * h->sm_count, static_cast<unsigned *>(sink),
                                              static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(h, e, "sla_probe_l2_read");
    h->launches += 1;
    return SLA_OK;
}

sla_status_t sla_selftest_wait_expiry(sla_handle_t h, int32_t max_polls, int32_t *polls_done_device, void *stream) {
    if (!h) return SLA_ERR_INVALID_ARG;
    if (max_polls < 1 || max_polls > 10000) return fail(h, SLA_ERR_INVALID_ARG, "max_polls must be in 1..10000%s");
    if (const char *why = check_device(h)) return fail(h, SLA_ERR_INVALID_ARG, "%s", why);
    cudaError_t e = sla::launch_selftest_wait_expiry(max_polls, reinterpret_cast<int *>(h->ws), polls_done_device,
                                                     static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(h, e, "sla_selftest_wait_expiry");
    h->launches += 1;
    return SLA_OK;
}

sla_status_t sla_create(sla_handle_t *handle, int device, size_t workspace_bytes) {
    if (!handle) return SLA_ERR_INVALID_ARG;
    *handle = nullptr;
    int n_dev = 0;
    cudaError_t e = cudaGetDeviceCount(&n_dev);
    if (e != cudaSuccess) return SLA_ERR_CUDA;
    if (device < 0 || device >= n_dev) return SLA_ERR_INVALID_ARG;
    sla_handle_s *h = new (std::nothrow) sla_handle_s();
    if (!h) return SLA_ERR_CUDA;
    h->device = device;
    int prev = 0;
    cudaGetDevice(&prev);
    e = cudaSetDevice(device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&h->sm_count, cudaDevAttrMultiProcessorCount, device);
    h->ws_bytes = workspace_bytes + kHeaderBytes;
    h->scratch_avail = workspace_bytes;
    if (e == cudaSuccess) e = cudaMalloc(reinterpret_cast<void **>(&h->ws), h->ws_bytes);
    if (e == cudaSuccess) e = cudaMemset(h->ws, 0, kHeaderBytes);
    cudaSetDevice(prev);
    if (e != cudaSuccess) {
        if (h->ws) cudaFree(h->ws);
        delete h;
        return SLA_ERR_CUDA;
    }
    *handle = h;
    return SLA_OK;
}

sla_status_t sla_destroy(sla_handle_t h) {
    if (!h) return SLA_ERR_INVALID_ARG;
    for (int j = 0; j < 2 * sla::KernelTimer::kMaxPairs; ++j)
        if (h->timer.ev[j]) cudaEventDestroy(h->timer.ev[j]);
    for (int j = 0; j < sla_handle_s::kMaxChunks; ++j) {
        if (h->ev_in[j]) cudaEventDestroy(h->ev_in[j]);
        if (h->ev_done[j]) cudaEventDestroy(h->ev_done[j]);
    }
    if (h->tbl_ev) cudaEventDestroy(h->tbl_ev);
    if (h->ev_fork) cudaEventDestroy(h->ev_fork);
    if (h->ev_join) cudaEventDestroy(h->ev_join);
    if (h->s_in) cudaStreamDestroy(h->s_in);
    if (h->s_out) cudaStreamDestroy(h->s_out);
    cudaError_t e = cudaFree(h->ws);
    delete h;
    return e == cudaSuccess ? SLA_OK : SLA_ERR_CUDA;
}

size_t sla_workspace_bytes(const sla_layout_t *l, const sla_params_t *p, int64_t Lq, int64_t Lkv) {
    if (check_layout_params(l, p, true) || Lq <= 0 || Lkv <= 0 || Lq > Lkv) return 0;
    sla::Call c = make_call(nullptr, l, p, Lq, Lkv - Lq, Lkv);
    std::vector<int> off, lf;   // host tables for the plans below, when the exponents are not 1/2
    if (!is_half(p->search_exponent)) {
        if (!build_offsets(p->search_exponent, Lkv, off)) return 0;
        c.off_host = off.data();
        c.n_off = (int)off.size();
    }
    if (!is_half(p->span_exponent) && p->span_len == 0) {
        if (!build_len_first(p->span_exponent, Lkv, lf)) return 0;
        c.len_first_host = lf.data();
        c.n_len = (int)lf.size();
    }
    // the SM count only changes how the decode work is split; size for a generous upper bound
    const sla::DecodePlan dp = sla::plan_decode(c, Lkv, 256 * l->batch * l->n_q_heads);
    size_t need = dp.bytes;
    if (sla::tc_attention_shape_ok(c, l->dtype)) {
        // tensor-core span-attention: scratch for chunks of up to 65536 query positions
        const sla::TcPlan tp = sla::plan_attention_tc(c, (int)(Lq < 65536 ? Lq : 65536));
        if (tp.bytes > need) need = tp.bytes;
    }
    return need + 4096 + (sla::Canaries::kMax + 1) * sla::Canaries::kBytes;   // slack, and room for debug canaries
}

sla_status_t sla_poll_status(sla_handle_t h, void *stream) {
    if (!h) return SLA_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int word = 0;
    cudaError_t e = cudaMemcpyAsync(&word, h->ws, sizeof word, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaMemsetAsync(h->ws, 0, sizeof word, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(h, e, "sla_poll_status");
    if (word & sla::kStatusOverrun) return fail(h, SLA_ERR_DEVICE_OVERRUN, "a kernel wrote outside its scratch region%s");
    if (word & sla::kStatusTimeout) return fail(h, SLA_ERR_DEVICE_TIMEOUT, "a bounded device-side wait expired%s");
    if (word & sla::kStatusBadIndex) return fail(h, SLA_ERR_DEVICE_INDEX, "an anchor outside [0, i] was skipped%s");
    return SLA_OK;
}

sla_status_t sla_span_search(sla_handle_t h, const void *q_s, const void *k, int64_t Lq, int64_t q_pos0,
                             int64_t Lkv, const sla_layout_t *l, const sla_params_t *p,
                             int32_t *out_anchor, float *out_score, void *stream) {
    if (!h) return SLA_ERR_INVALID_ARG;
    if (const char *why = check_layout_params(l, p, false)) return fail(h, SLA_ERR_INVALID_ARG, "%s", why);
    if (const char *why = check_prefill_range(Lq, q_pos0, Lkv)) return fail(h, SLA_ERR_INVALID_ARG, "%s", why);
    if (!q_s || !k || !out_anchor || !out_score) return fail(h, SLA_ERR_INVALID_ARG, "NULL tensor pointer%s");
    if (const char *why = check_device(h)) return fail(h, SLA_ERR_INVALID_ARG, "%s", why);
    if (!aligned16(q_s) || !aligned16(k)) return fail(h, SLA_ERR_INVALID_ARG, "tensor pointers must be 16-byte aligned%s");
    if (sla_status_t ps = prepare_pattern(h, p, Lkv, static_cast<cudaStream_t>(stream))) return ps;
    sla::Call c = make_call(h, l, p, Lq, q_pos0, Lkv);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (sla::search_diag_supported(c, l->dtype) && ((reinterpret_cast<uintptr_t>(q_s) | reinterpret_cast<uintptr_t>(k)) & 31u) == 0) {
        cudaError_t e = sla::launch_search_diag(q_s, k, c, out_anchor, out_score, st, &h->launches);
        if (e != cudaSuccess) return cuda_fail(h, e, "sla_span_search (fused selection)");
        return SLA_OK;
    }
    if (sla::search_mma_supported(c, l->dtype)) {
        cudaError_t e = sla::launch_search_mma(q_s, k, c, out_anchor, out_score, st, &h->launches);
        if (e != cudaSuccess) return cuda_fail(h, e, "sla_span_search (tensor-core path)");
        return SLA_OK;
    }
    cudaError_t e = sla::launch_search_simt(q_s, k, c, l->dtype, out_anchor, out_score, st);
    if (e != cudaSuccess) return cuda_fail(h, e, "sla_span_search");
    h->launches += 1;
    return SLA_OK;
}

namespace {

// Body of the two span-attention entry points (score and lse_span are NULL in the union mode).
sla_status_t span_attention_impl(sla_handle_t h, const void *q, const void *k, const void *v, int64_t Lq,
                                 int64_t q_pos0, int64_t Lkv, const sla_layout_t *l, const sla_params_t *p,
                                 const int32_t *anchor, const float *score, void *out, float *lse,
                                 float *lse_span, void *stream, const char *what) {
    if (const char *why = check_prefill_range(Lq, q_pos0, Lkv)) return fail(h, SLA_ERR_INVALID_ARG, "%s", why);
    if (!q || !k || !v || !anchor || !out || !lse) return fail(h, SLA_ERR_INVALID_ARG, "NULL tensor pointer%s");
    if (const char *why = check_device(h)) return fail(h, SLA_ERR_INVALID_ARG, "%s", why);
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out))
        return fail(h, SLA_ERR_INVALID_ARG, "tensor pointers must be 16-byte aligned%s");
    if (sla_status_t ps = prepare_pattern(h, p, Lkv, static_cast<cudaStream_t>(stream))) return ps;
    sla::Call c = make_call(h, l, p, Lq, q_pos0, Lkv);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (sla::tc_attention_supported(c, l->dtype)) {
        // tensor-core path; needs scratch for at least a modest chunk of query positions.  A workspace
        // that cannot hold it is an error, not a reason to run the (far slower) generic kernel.
        const long long min_chunk = Lq < 1024 ? Lq : 1024;
        const sla::TcPlan probe = sla::plan_attention_tc(c, (int)min_chunk, h->canaries ? sla::Canaries::kBytes : 0);
        if (probe.ok) {
            if (probe.bytes > h->scratch_avail)
                return fail(h, SLA_ERR_WORKSPACE, "workspace too small for span-attention: ask sla_workspace_bytes%s");
            cudaError_t e = sla::launch_attn_tc(q, k, v, c, anchor, score, out, lse, lse_span, h->ws + kHeaderBytes,
                                                h->scratch_avail, h->sm_count, st, &h->launches, &h->timer, h->canaries, &h->tc_last);
            if (e != cudaSuccess) return cuda_fail(h, e, what);
            return SLA_OK;
        }
    }
    cudaError_t e = sla::launch_attn_simt(q, k, v, c, l->dtype, anchor, score, out, lse, lse_span, st);
    if (e != cudaSuccess) return cuda_fail(h, e, what);
    h->launches += 1;
    return SLA_OK;
}

}  // namespace

sla_status_t sla_span_attention(sla_handle_t h, const void *q, const void *k, const void *v, int64_t Lq,
                                int64_t q_pos0, int64_t Lkv, const sla_layout_t *l, const sla_params_t *p,
                                const int32_t *anchor, void *out, float *lse, void *stream) {
    if (!h) return SLA_ERR_INVALID_ARG;
    if (const char *why = check_layout_params(l, p, false)) return fail(h, SLA_ERR_INVALID_ARG, "%s", why);
    if (p->mode != SLA_UNION)
        return fail(h, SLA_ERR_INVALID_ARG, "SLA_PER_SPAN needs the search scores: call sla_span_attention_gated%s");
    return span_attention_impl(h, q, k, v, Lq, q_pos0, Lkv, l, p, anchor, nullptr, out, lse, nullptr, stream,
                               "sla_span_attention");
}

sla_status_t sla_span_attention_gated(sla_handle_t h, const void *q, const void *k, const void *v, int64_t Lq,
                                      int64_t q_pos0, int64_t Lkv, const sla_layout_t *l,
                                      const sla_params_t *p, const int32_t *anchor, const float *score,
                                      void *out, float *lse, float *lse_span, void *stream) {
    if (!h) return SLA_ERR_INVALID_ARG;
    if (const char *why = check_layout_params(l, p, false)) return fail(h, SLA_ERR_INVALID_ARG, "%s", why);
    if (p->mode != SLA_PER_SPAN) return fail(h, SLA_ERR_INVALID_ARG, "sla_span_attention_gated needs mode = SLA_PER_SPAN%s");
    if (!score) return fail(h, SLA_ERR_INVALID_ARG, "NULL tensor pointer%s");
    return span_attention_impl(h, q, k, v, Lq, q_pos0, Lkv, l, p, anchor, score, out, lse, lse_span, stream,
                               "sla_span_attention_gated");
}

sla_status_t sla_decode_step(sla_handle_t h, const void *q_s, const void *q, const void *k_cache,
                             const void *v_cache, int64_t n_ctx, const sla_layout_t *l,
                             const sla_params_t *p, void *out, float *lse, int32_t *out_anchor,
                             float *out_score, void *stream) {
    if (!h) return SLA_ERR_INVALID_ARG;
    if (const char *why = check_layout_params(l, p, true)) return fail(h, SLA_ERR_INVALID_ARG, "%s", why);
    if (n_ctx <= 0 || n_ctx > 2147483647LL) return fail(h, SLA_ERR_INVALID_ARG, "n_ctx must be in 1..2^31-1%s");
    if (const char *why = check_device(h)) return fail(h, SLA_ERR_INVALID_ARG, "%s", why);
    if (!q_s || !q || !k_cache || !v_cache || !out || !lse || !out_anchor || !out_score)
        return fail(h, SLA_ERR_INVALID_ARG, "NULL tensor pointer%s");
    if (!aligned16(q_s) || !aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(out))
        return fail(h, SLA_ERR_INVALID_ARG, "tensor pointers must be 16-byte aligned%s");
    if (sla_status_t ps = prepare_pattern(h, p, n_ctx, static_cast<cudaStream_t>(stream))) return ps;
    sla::Call c = make_call(h, l, p, 1, n_ctx - 1, n_ctx);
    const sla::DecodePlan plan =
        sla::plan_decode(c, n_ctx, h->sm_count * sla::decode_attn_blocks_per_sm(l->dtype, l->head_dim),
                         h->canaries ? sla::Canaries::kBytes : 0);
    if (plan.bytes + kHeaderBytes > h->ws_bytes) return fail(h, SLA_ERR_WORKSPACE, "workspace too small for this decode step%s");
    if ((size_t)plan.n_anchor * sizeof(float) * 8 > 180 * 1024) return fail(h, SLA_ERR_UNSUPPORTED, "context too long for the decode top-k stage%s");
    const size_t units = p->mode == SLA_PER_SPAN ? (size_t)p->top_k : 1;
    if ((size_t)(l->batch) * (l->n_kv_heads + l->n_q_heads * (units + 1)) * sizeof(int) > kCounterEnd - kCounterOffset)
        return fail(h, SLA_ERR_UNSUPPORTED, "too many (batch, head) pairs for the decode step%s");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = sla::launch_canary_fill(h->ws + kHeaderBytes, plan.canaries, st);
    if (e == cudaSuccess)
        e = sla::launch_decode(q_s, q, k_cache, v_cache, c, l->dtype, n_ctx, plan, h->ws + kHeaderBytes,
                               reinterpret_cast<int *>(h->ws + kCounterOffset), out, lse, out_anchor, out_score, st);
    if (e == cudaSuccess) e = sla::launch_canary_check(h->ws + kHeaderBytes, plan.canaries, c.status, st);
    if (e != cudaSuccess) return cuda_fail(h, e, "sla_decode_step");
    h->launches += 2;
    if (plan.canaries.n) { h->last_canaries = plan.canaries; h->last_canary_base = h->ws + kHeaderBytes; }
    return SLA_OK;
}

namespace {

// Common checks of the three sequence-sharded calls; fills the call description of this rank.
sla_status_t shard_call(sla_handle_t h, const sla_layout_t *l, const sla_params_t *p, int64_t n_ctx,
                        int64_t shard_lo, int64_t shard_len, void *stream, sla::Call *c) {
    if (const char *why = check_layout_params(l, p, true)) return fail(h, SLA_ERR_INVALID_ARG, "%s", why);
    if (n_ctx <= 0 || n_ctx > 2147483647LL) return fail(h, SLA_ERR_INVALID_ARG, "n_ctx must be in 1..2^31-1%s");
    if (shard_lo < 0 || shard_len < 0 || shard_lo + shard_len > 2147483647LL)
        return fail(h, SLA_ERR_INVALID_ARG, "shard range out of bounds%s");
    if (const char *why = check_device(h)) return fail(h, SLA_ERR_INVALID_ARG, "%s", why);
    if (p->window != 0 || p->mode != SLA_UNION)
        return fail(h, SLA_ERR_UNSUPPORTED, "the sequence-sharded step implements the union mode without a window%s");
    if (sla_status_t ps = prepare_pattern(h, p, n_ctx, static_cast<cudaStream_t>(stream))) return ps;
    *c = make_call(h, l, p, 1, n_ctx - 1, n_ctx);
    c->shard_lo = shard_lo;
    c->shard_hi = shard_lo + shard_len < n_ctx ? shard_lo + shard_len : n_ctx;   // positions >= n_ctx are not valid yet
    if (c->shard_hi < c->shard_lo) c->shard_hi = c->shard_lo;
    if ((size_t)(l->batch) * (l->n_kv_heads + 2 * l->n_q_heads) * sizeof(int) > kCounterEnd - kCounterOffset)
        return fail(h, SLA_ERR_UNSUPPORTED, "too many (batch, head) pairs for the decode step%s");
    return SLA_OK;
}

}  // namespace

sla_status_t sla_decode_shard_search(sla_handle_t h, const void *q_s, const void *k_local, int64_t shard_lo,
                                     int64_t shard_len, int64_t n_ctx, const sla_layout_t *l,
                                     const sla_params_t *p, int32_t *cand_anchor, float *cand_score, void *stream) {
    if (!h) return SLA_ERR_INVALID_ARG;
    if (!q_s || !k_local || !cand_anchor || !cand_score) return fail(h, SLA_ERR_INVALID_ARG, "NULL tensor pointer%s");
    if (!aligned16(q_s) || !aligned16(k_local)) return fail(h, SLA_ERR_INVALID_ARG, "tensor pointers must be 16-byte aligned%s");
    sla::Call c;
    if (sla_status_t s = shard_call(h, l, p, n_ctx, shard_lo, shard_len, stream, &c)) return s;
    // candidate strides of this rank: anchors t = i + 1 - offset with shard_lo <= t < shard_hi
    const long long i = n_ctx - 1;
    const int s_first = c.shard_hi > i ? 0 : sla::n_strides(c, i - c.shard_hi);      // offsets <= i + 1 - shard_hi lie right of the range
    const int s_end = c.shard_lo > i ? 0 : sla::n_strides(c, i - c.shard_lo);        // offsets <= i + 1 - shard_lo reach into it
    const int n = s_end > s_first ? s_end - s_first : 0;
    const sla::DecodePlan plan =
        sla::plan_decode(c, n_ctx, h->sm_count * sla::decode_attn_blocks_per_sm(l->dtype, l->head_dim));
    if (plan.bytes + kHeaderBytes > h->ws_bytes) return fail(h, SLA_ERR_WORKSPACE, "workspace too small for this decode step%s");
    if ((size_t)n * sizeof(float) * 8 > 180 * 1024) return fail(h, SLA_ERR_UNSUPPORTED, "context too long for the decode top-k stage%s");
    cudaError_t e = sla::launch_decode_shard_search(q_s, k_local, c, l->dtype, n_ctx, s_first, n, h->ws + kHeaderBytes,
                                                    reinterpret_cast<int *>(h->ws + kCounterOffset), cand_anchor,
                                                    cand_score, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(h, e, "sla_decode_shard_search");
    h->launches += 1;
    return SLA_OK;
}

sla_status_t sla_decode_shard_attend(sla_handle_t h, const void *q, const void *k_local, const void *v_local,
                                     int64_t shard_lo, int64_t shard_len, int64_t n_ctx, const sla_layout_t *l,
                                     const sla_params_t *p, int32_t n_shards, const int32_t *all_anchor,
                                     const float *all_score, int32_t *out_anchor, float *out_score, float *partial,
                                     void *stream) {
    if (!h) return SLA_ERR_INVALID_ARG;
    if (!q || !k_local || !v_local || !all_anchor || !all_score || !out_anchor || !out_score || !partial)
        return fail(h, SLA_ERR_INVALID_ARG, "NULL tensor pointer%s");
    if (!aligned16(q) || !aligned16(k_local) || !aligned16(v_local)) return fail(h, SLA_ERR_INVALID_ARG, "tensor pointers must be 16-byte aligned%s");
    if (n_shards < 1 || n_shards > 64) return fail(h, SLA_ERR_INVALID_ARG, "n_shards must be in 1..64%s");
    sla::Call c;
    if (sla_status_t s = shard_call(h, l, p, n_ctx, shard_lo, shard_len, stream, &c)) return s;
    const sla::DecodePlan plan =
        sla::plan_decode(c, n_ctx, h->sm_count * sla::decode_attn_blocks_per_sm(l->dtype, l->head_dim));
    if (plan.bytes + kHeaderBytes > h->ws_bytes) return fail(h, SLA_ERR_WORKSPACE, "workspace too small for this decode step%s");
    cudaError_t e = sla::launch_decode_shard_attend(q, k_local, v_local, c, l->dtype, n_ctx, plan, h->ws + kHeaderBytes,
                                                    reinterpret_cast<int *>(h->ws + kCounterOffset), n_shards,
                                                    all_anchor, all_score, out_anchor, out_score, partial,
                                                    static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(h, e, "sla_decode_shard_attend");
    h->launches += 2;
    return SLA_OK;
}

sla_status_t sla_decode_shard_merge(sla_handle_t h, int32_t n_shards, const float *all_partial,
                                    const sla_layout_t *l, void *out, float *lse, void *stream) {
    if (!h) return SLA_ERR_INVALID_ARG;
    if (!l || !all_partial || !out || !lse) return fail(h, SLA_ERR_INVALID_ARG, "NULL pointer%s");
    if (n_shards < 1 || n_shards > 64) return fail(h, SLA_ERR_INVALID_ARG, "n_shards must be in 1..64%s");
    if (const char *why = check_device(h)) return fail(h, SLA_ERR_INVALID_ARG, "%s", why);
    if (l->batch <= 0 || l->n_q_heads <= 0 || (l->head_dim != 64 && l->head_dim != 128) ||
        (l->dtype != SLA_F32 && l->dtype != SLA_BF16) || l->q_stride_b < 0 || l->q_stride_h < l->head_dim)
        return fail(h, SLA_ERR_INVALID_ARG, "bad layout%s");
    sla::Call c = {};
    c.B = l->batch; c.Hq = l->n_q_heads; c.D = l->head_dim;
    c.q_sb = l->q_stride_b; c.q_sh = l->q_stride_h;
    cudaError_t e = sla::launch_decode_shard_merge(all_partial, n_shards, c, l->dtype, out, lse, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(h, e, "sla_decode_shard_merge");
    h->launches += 1;
    return SLA_OK;
}

size_t sla_host_staging_bytes(const sla_layout_t *l, const sla_params_t *p, int64_t L) {
    if (check_layout_params(l, p, true) || L <= 0) return 0;
    const size_t es = elem_size(l->dtype);
    const size_t qn = (size_t)l->batch * l->n_q_heads * L * l->head_dim;
    const size_t kn = (size_t)l->batch * l->n_kv_heads * L * l->head_dim;
    const size_t rows = (size_t)l->batch * l->n_q_heads * L;
    // q_s, q, out + k, v + lse + anchors + scores, each rounded up to 256 bytes
    return 3 * (qn * es + 256) + 2 * (kn * es + 256) + (rows * 4 + 256) + 2 * (rows * p->top_k * 4 + 256);
}

sla_status_t sla_prefill_host(sla_handle_t h, const void *q_s_host, const void *q_host, const void *k_host,
                              const void *v_host, int64_t L, const sla_layout_t *l, const sla_params_t *p,
                              void *out_host, float *lse_host, int32_t *anchor_host, float *score_host,
                              void *stream) {
    if (!h) return SLA_ERR_INVALID_ARG;
    if (const char *why = check_layout_params(l, p, true)) return fail(h, SLA_ERR_INVALID_ARG, "%s", why);
    if (L <= 0 || L > 2147483647LL) return fail(h, SLA_ERR_INVALID_ARG, "L out of range%s");
    if (!q_s_host || !q_host || !k_host || !v_host || !out_host || !lse_host || !anchor_host || !score_host)
        return fail(h, SLA_ERR_INVALID_ARG, "NULL host pointer%s");
    if (const char *why = check_device(h)) return fail(h, SLA_ERR_INVALID_ARG, "%s", why);
    sla_layout_t dl = *l;
    dl.q_stride_t = dl.kv_stride_t = l->head_dim;
    dl.q_stride_h = dl.kv_stride_h = L * l->head_dim;
    dl.q_stride_b = dl.q_stride_h * l->n_q_heads;
    dl.kv_stride_b = dl.kv_stride_h * l->n_kv_heads;
    const size_t work = sla_workspace_bytes(&dl, p, L, L);
    const size_t stage = sla_host_staging_bytes(&dl, p, L);
    if (kHeaderBytes + work + stage > h->ws_bytes) return fail(h, SLA_ERR_WORKSPACE, "workspace too small for host staging%s");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t es = elem_size(l->dtype);
    const size_t qb = (size_t)l->batch * l->n_q_heads * L * l->head_dim * es;
    const size_t kb = (size_t)l->batch * l->n_kv_heads * L * l->head_dim * es;
    const size_t rows = (size_t)l->batch * l->n_q_heads * L;
    // staging sits at the END of the workspace so that the scratch of the two steps keeps its place
    char *base = h->ws + h->ws_bytes - stage;
    auto take = [&base](size_t n) { char *p0 = base; base += (n + 255) & ~(size_t)255; return p0; };
    char *d_qs = take(qb), *d_q = take(qb), *d_out = take(qb), *d_k = take(kb), *d_v = take(kb);
    float *d_lse = (float *)take(rows * 4);
    int32_t *d_anchor = (int32_t *)take(rows * p->top_k * 4);
    float *d_score = (float *)take(rows * p->top_k * 4);

    // The sequence goes through in chunks of query positions (chunked prefill: chunk c needs the keys
    // up to its own end only), so that the copy-in of chunk c+1, the kernels of chunk c and the
    // copy-out of chunk c-1 overlap on three streams.  The device tensors keep the host layout
    // [B, H, L, D]; a chunk of positions is a 2-D copy (one segment per (batch, head)).  Anchors, scores
    // and lse of a chunk are compact [B, Hq, Lc, ...] blocks, as the search call writes them.
    int n_chunks = (int)(L / 2048);
    if (n_chunks > sla_handle_s::kMaxChunks) n_chunks = sla_handle_s::kMaxChunks;
    if (n_chunks < 1) n_chunks = 1;
    const int64_t Lc = ((L + n_chunks - 1) / n_chunks + 127) / 128 * 128;
    n_chunks = (int)((L + Lc - 1) / Lc);
    cudaError_t e = cudaSuccess;
    if (!h->s_in) {
        e = cudaStreamCreateWithFlags(&h->s_in, cudaStreamNonBlocking);
        if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&h->s_out, cudaStreamNonBlocking);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->ev_fork, cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->ev_join, cudaEventDisableTiming);
        for (int j = 0; j < sla_handle_s::kMaxChunks && e == cudaSuccess; ++j) {
            e = cudaEventCreateWithFlags(&h->ev_in[j], cudaEventDisableTiming);
            if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->ev_done[j], cudaEventDisableTiming);
        }
        if (e != cudaSuccess) return cuda_fail(h, e, "sla_prefill_host (streams)");
    }
    const size_t D = (size_t)l->head_dim;
    const size_t row_q = (size_t)L * D * es;          // pitch of one (batch, head) segment
    const int nq = l->batch * l->n_q_heads, nkv = l->batch * l->n_kv_heads;
    // copy-in stream: ordered after whatever the caller's stream holds so far
    e = cudaEventRecord(h->ev_fork, st);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(h->s_in, h->ev_fork, 0);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(h->s_out, h->ev_fork, 0);
    for (int c = 0; c < n_chunks && e == cudaSuccess; ++c) {
        const int64_t c0 = (int64_t)c * Lc, lc = (L - c0 < Lc) ? L - c0 : Lc;
        const size_t off = (size_t)c0 * D * es, width = (size_t)lc * D * es;
        e = cudaMemcpy2DAsync(d_qs + off, row_q, (const char *)q_s_host + off, row_q, width, nq, cudaMemcpyHostToDevice, h->s_in);
        if (e == cudaSuccess) e = cudaMemcpy2DAsync(d_k + off, row_q, (const char *)k_host + off, row_q, width, nkv, cudaMemcpyHostToDevice, h->s_in);
        if (e == cudaSuccess) e = cudaMemcpy2DAsync(d_q + off, row_q, (const char *)q_host + off, row_q, width, nq, cudaMemcpyHostToDevice, h->s_in);
        if (e == cudaSuccess) e = cudaMemcpy2DAsync(d_v + off, row_q, (const char *)v_host + off, row_q, width, nkv, cudaMemcpyHostToDevice, h->s_in);
        if (e == cudaSuccess) e = cudaEventRecord(h->ev_in[c], h->s_in);
    }
    if (e != cudaSuccess) return cuda_fail(h, e, "sla_prefill_host (copy in)");
    const size_t avail_before = h->scratch_avail;
    h->scratch_avail = h->ws_bytes - kHeaderBytes - stage;   // the staging buffers are not scratch
    sla_status_t s = SLA_OK;
    const size_t k4 = (size_t)p->top_k * 4;
    for (int c = 0; c < n_chunks && s == SLA_OK; ++c) {
        const int64_t c0 = (int64_t)c * Lc, lc = (L - c0 < Lc) ? L - c0 : Lc;
        const size_t off = (size_t)c0 * D * es;
        // compact per-chunk blocks: chunk c starts after the rows of the chunks before it
        const size_t blk = (size_t)nq * c0;
        int32_t *a_c = d_anchor + blk * p->top_k;
        float *s_c = d_score + blk * p->top_k, *l_c = d_lse + blk;
        e = cudaStreamWaitEvent(st, h->ev_in[c], 0);
        if (e != cudaSuccess) { s = cuda_fail(h, e, "sla_prefill_host (wait)"); break; }
        s = sla_span_search(h, d_qs + off, d_k, lc, c0, c0 + lc, &dl, p, a_c, s_c, stream);
        if (s == SLA_OK) s = sla_span_attention(h, d_q + off, d_k, d_v, lc, c0, c0 + lc, &dl, p, a_c, d_out + off, l_c, stream);
        if (s != SLA_OK) break;
        e = cudaEventRecord(h->ev_done[c], st);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(h->s_out, h->ev_done[c], 0);
        const size_t width = (size_t)lc * D * es;
        if (e == cudaSuccess) e = cudaMemcpy2DAsync((char *)out_host + off, row_q, d_out + off, row_q, width, nq, cudaMemcpyDeviceToHost, h->s_out);
        if (e == cudaSuccess) e = cudaMemcpy2DAsync((char *)lse_host + (size_t)c0 * 4, (size_t)L * 4, l_c, (size_t)lc * 4, (size_t)lc * 4, nq, cudaMemcpyDeviceToHost, h->s_out);
        if (e == cudaSuccess) e = cudaMemcpy2DAsync((char *)anchor_host + (size_t)c0 * k4, (size_t)L * k4, a_c, (size_t)lc * k4, (size_t)lc * k4, nq, cudaMemcpyDeviceToHost, h->s_out);
        if (e == cudaSuccess) e = cudaMemcpy2DAsync((char *)score_host + (size_t)c0 * k4, (size_t)L * k4, s_c, (size_t)lc * k4, (size_t)lc * k4, nq, cudaMemcpyDeviceToHost, h->s_out);
        if (e != cudaSuccess) s = cuda_fail(h, e, "sla_prefill_host (copy out)");
    }
    h->scratch_avail = avail_before;
    // join: the caller's stream continues after the last copy-out, and this call returns after it
    e = cudaEventRecord(h->ev_join, h->s_out);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(st, h->ev_join, 0);
    if (e == cudaSuccess) e = cudaStreamSynchronize(h->s_in);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (s != SLA_OK) return s;
    if (e != cudaSuccess) return cuda_fail(h, e, "sla_prefill_host (copy out)");
    return SLA_OK;
}

}  // extern "C"
