// Diagnostics of libsla that are not part of the method: a read-only L2 bandwidth probe (the roofline
// denominator of the span-search kernel, which streams key rows out of L2) and a self-test of the
// bounded device-side wait.  Declared in include/sla.h.
#include "sla_kernels.h"
#include "sla_tc_ptx.cuh"

namespace sla {

namespace {

constexpr int kProbeThreads = 256;

// Every CTA walks the whole buffer `iters` times, a warp reading 1 KiB per step with 32-byte loads
// (the access width of the span-search kernel); CTAs start at different places so that the L2 slices
// are all busy.  The loaded words are folded into a value that is stored only if it takes an
// (impossible) magic value, which keeps the loads alive without a data-dependent store.
__global__ void __launch_bounds__(kProbeThreads) probe_l2_read(const uint4 *__restrict__ buf, size_t n_vec32, int iters,
                                                                unsigned *__restrict__ sink) {
    const size_t per_cta = (size_t)kProbeThreads;              // 32-byte vectors a CTA reads per step
    const size_t steps = n_vec32 / per_cta;
    size_t at = ((size_t)blockIdx.x * 977u) % steps;             // a different starting step per CTA
    unsigned acc = 0;
    const long long total = (long long)steps * iters;
#pragma unroll 4
    for (long long it = 0; it < total; ++it) {
        const uint4 *p = buf + 2 * (at * per_cta + threadIdx.x);
        unsigned w0, w1, w2, w3, w4, w5, w6, w7;
        asm volatile("ld.global.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                     : "=r"(w0), "=r"(w1), "=r"(w2), "=r"(w3), "=r"(w4), "=r"(w5), "=r"(w6), "=r"(w7)
                     : "l"(p));
        acc ^= w0 ^ w1 ^ w2 ^ w3 ^ w4 ^ w5 ^ w6 ^ w7;
        at = at + 1 == steps ? 0 : at + 1;
    }
    if (acc == 0x9e3779b9u && sink) *sink = acc;
}

// One warp: lane 0 waits on an mbarrier that nothing ever arrives on, for at most `max_polls` polls, then
// raises the time-out bit of the status word -- the path every bounded wait of the tensor-core kernels
// takes when it runs out -- and the kernel returns by itself.  No copy or MMA is in flight.
__global__ void __launch_bounds__(32) selftest_wait_expiry(int max_polls, int *status, int *polls_done) {
    __shared__ unsigned long long bar;
    const uint32_t b = ptx::smem_u32(&bar);
    if (threadIdx.x == 0) {
        ptx::mbar_init(b, 1);
        ptx::fence_barrier_init();
        int n = 0;
        bool done = false;
#pragma unroll 1
        for (; n < max_polls && !done; ++n) done = ptx::mbar_test_wait(b, 0);
        if (!done) atomicOr(status, kStatusTimeout);
        if (polls_done) *polls_done = n;
    }
}

constexpr unsigned kCanaryWord = 0xC5A5C5A5u;
// one CTA of 64 threads per gap: a gap is 64 words
__global__ void __launch_bounds__(64) canary_fill(char *scratch, Canaries cn) {
    reinterpret_cast<unsigned *>(scratch + cn.at[blockIdx.x])[threadIdx.x] = kCanaryWord;
}
__global__ void __launch_bounds__(64) canary_check(const char *scratch, Canaries cn, int *status) {
    if (reinterpret_cast<const unsigned *>(scratch + cn.at[blockIdx.x])[threadIdx.x] != kCanaryWord)
        atomicOr(status, kStatusOverrun);
}

}  // namespace

cudaError_t launch_canary_fill(void *scratch, const Canaries &cn, cudaStream_t st) {
    static_assert(Canaries::kBytes == 64 * sizeof(unsigned), "one thread per canary word");
    if (cn.n == 0) return cudaSuccess;
    canary_fill<<<cn.n, 64, 0, st>>>(static_cast<char *>(scratch), cn);
    return cudaGetLastError();
}

cudaError_t launch_canary_check(const void *scratch, const Canaries &cn, int *status, cudaStream_t st) {
    if (cn.n == 0) return cudaSuccess;
    canary_check<<<cn.n, 64, 0, st>>>(static_cast<const char *>(scratch), cn, status);
    return cudaGetLastError();
}

cudaError_t launch_probe_l2_read(const void *buf, size_t bytes, int iters, int n_ctas, unsigned *sink, cudaStream_t st) {
    probe_l2_read<<<n_ctas, kProbeThreads, 0, st>>>((const uint4 *)buf, bytes / 32, iters, sink);
    return cudaGetLastError();
}

cudaError_t launch_selftest_wait_expiry(int max_polls, int *status, int *polls_done, cudaStream_t st) {
    selftest_wait_expiry<<<1, 32, 0, st>>>(max_polls, status, polls_done);
    return cudaGetLastError();
}

}  // namespace sla
