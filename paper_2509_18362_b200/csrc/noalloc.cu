// fastmtp_verify_accept_static: greedy verification for callers that must not allocate.
//
// Some hosts of this library cannot create device memory at the moment they need a verification:
// a serving process whose allocator has already claimed the whole GPU for its KV-cache pool (a
// cudaMalloc there fails or forces the pool to shrink), code running where an allocation would
// synchronise the device in the middle of a latency-critical decode loop, or a plug-in that is
// only handed raw pointers and has no context or workspace of its own. The regular entry point
// needs a context with a caller-provided workspace for its per-row scratch; this one keeps that
// scratch in a fixed array inside the library image instead, so it needs neither.
#include "../../include/fastmtp.h"
#include "mega.cuh"

#include <mutex>

namespace {

// Scratch of the verification kernel: one 64-bit (value, id) key per logit row, then the arrival
// counter and the internal status word. Every GPU that loads the library holds these 8.3 KB until
// the process exits.
constexpr int kStaticMaxRows = FMTP_STATIC_VERIFY_MAX_ROWS;
static __device__ __align__(256) unsigned long long g_verify_scratch[kStaticMaxRows + 2];

constexpr int kMaxDevices = 64;
std::mutex g_lock;
unsigned long long *g_scratch_ptr[kMaxDevices];   // device address of the array, per device, once resolved

// In host code `g_verify_scratch` is only a handle: the array's device address has to be asked for,
// once per device, with that device current.
int scratch_address(unsigned long long **out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return (int)e;
    if (dev < 0 || dev >= kMaxDevices) return (int)cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> guard(g_lock);
    if (!g_scratch_ptr[dev]) {
        void *p = nullptr;
        e = cudaGetSymbolAddress(&p, g_verify_scratch);
        if (e != cudaSuccess || !p) return e != cudaSuccess ? (int)e : (int)cudaErrorInvalidSymbol;
        g_scratch_ptr[dev] = static_cast<unsigned long long *>(p);
    }
    *out = g_scratch_ptr[dev];
    return 0;
}

}  // namespace

extern "C" int fastmtp_verify_accept_static(const fmtp_bf16 *logits, const int32_t *drafts, int B, int K, int V,
                                            int32_t *out_accept, int32_t *out_bonus, int32_t *out_argmax,
                                            uint32_t *dev_status, void *stream) {
    if (!logits || !out_accept || !out_bonus || (K > 0 && !drafts)) return FMTP_EINVAL;
    if (B <= 0 || K < 0 || V <= 0) return FMTP_EINVAL;
    const long long rows = (long long)B * (K + 1);
    if (rows > kStaticMaxRows) return FMTP_ESHAPE;     // beyond the fixed scratch: use fastmtp_verify_accept
    unsigned long long *scr = nullptr;
    if (scratch_address(&scr) != 0) return FMTP_ECUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // the array keeps whatever the previous call (or an aborted one) left: keys, counter and status of
    // this call start from zero
    if (cudaMemsetAsync(scr, 0, ((size_t)rows + 2) * sizeof(unsigned long long), st) != cudaSuccess) return FMTP_ECUDA;
    uint32_t *counter = reinterpret_cast<uint32_t *>(scr + rows);
    uint32_t *status = reinterpret_cast<uint32_t *>(scr + rows + 1);
    int err = fmtp::verify_launch(logits, drafts, B, K, V, out_accept, out_bonus, out_argmax, scr, counter, status,
                                  dev_status, 0, st);
    return err ? FMTP_ECUDA : FMTP_OK;
}
