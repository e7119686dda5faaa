// Diagnostic entry point: shows, without hanging or faulting anything, what the library's device
// waits do when the event they wait for never comes. A one-warp kernel waits on an mbarrier that
// nothing arrives on, with the same poll-and-check-the-clock loop the decoder kernel uses for its
// ring and grid barriers but a caller-chosen limit; when the limit passes it ORs FMTP_DEV_TIMEOUT
// into the status word and returns normally, so the context stays usable.
#include "../../include/fastmtp.h"
#include "ptx.cuh"

namespace {

__global__ void wait_probe_kernel(uint32_t *status, unsigned long long limit_ns, unsigned long long *waited_ns) {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        fmtp::mbar_init(&bar, 1);
        fmtp::mbar_fence_init();
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const unsigned long long t0 = fmtp::global_timer_ns();
        bool done = false;
        unsigned long long now = t0;
        for (uint32_t n = 0; !done; ++n) {
            if (fmtp::mbar_try_wait(&bar, 0)) { done = true; break; }     // never: no one arrives
            if ((n & 255u) == 255u) {
                now = fmtp::global_timer_ns();
                if (now - t0 > limit_ns) break;
            }
        }
        if (!done) atomicOr(status, FMTP_DEV_TIMEOUT);
        if (waited_ns) *waited_ns = now - t0;
    }
}

}  // namespace

extern "C" int fmtp_selftest_wait_timeout(uint32_t *dev_status, int limit_ms, unsigned long long *dev_waited_ns, void *stream) {
    if (!dev_status) return FMTP_EINVAL;
    if (limit_ms < 1 || limit_ms > 1000) return FMTP_EINVAL;          // bounded on purpose
    wait_probe_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(dev_status, (unsigned long long)limit_ms * 1000000ull,
                                                                        dev_waited_ns);
    return cudaGetLastError() == cudaSuccess ? FMTP_OK : FMTP_ECUDA;
}
