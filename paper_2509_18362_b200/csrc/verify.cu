// Greedy verification: full-vocabulary argmax of every target-logit row, then the longest
// accepted draft prefix and the bonus token (Sec. 2.3 "Verification phase" of the paper).
//
// HBM-bound read-once scan. The rows are cut into slices of 16 K elements; a launch has a few CTAs per
// SM and each takes a contiguous range of slices (so most of a CTA's slices belong to one row). A
// thread keeps 8 independent 128-bit streaming loads in flight and requests the next slice's before it
// looks at the current one's; (value, id) pairs are reduced to one 64-bit key -- highest value first,
// then lowest token id, NaN never wins -- and published with atomicMax when the CTA leaves a row (an
// integer maximum: order independent, so the result is reproducible). The CTA that arrives last
// turns the per-row winners into accept_len / bonus and clears the scratch for the next call.
#include "mega.cuh"
#include "ptx.cuh"

namespace fmtp {

namespace {

constexpr int kVThreads = 256;
constexpr int kVecPerThread = 8;                                  // 16-byte loads in flight per thread and slice
constexpr int kSlice = kVThreads * kVecPerThread * 8;             // bf16 elements per slice (16384)
constexpr int kVCtasPerSm = 2;                                 // resident CTAs per SM at this register footprint
constexpr int kNoIdx = 0x7fffffff;

__device__ __forceinline__ void consider(float v, int i, float &best, int &idx) {
    // strict '>' keeps the earliest (lowest) id among equal values; the second clause admits the
    // first non-NaN value even if it is -inf
    if (v > best || (idx == kNoIdx && v == v)) { best = v; idx = i; }
}

struct SliceRef { const bf16_t *src; int lo, hi; bool vec; };

__device__ __forceinline__ SliceRef slice_ref(const bf16_t *logits, int V, int slices_per_row, int item) {
    const int row = item / slices_per_row, slice = item - row * slices_per_row;
    SliceRef r;
    r.src = logits + (size_t)row * V;
    r.lo = slice * kSlice;
    r.hi = min(V, r.lo + kSlice);
    r.vec = (reinterpret_cast<uintptr_t>(r.src) & 15u) == 0;
    return r;
}
__device__ __forceinline__ void slice_load(const SliceRef &r, uint4 (&v)[kVecPerThread]) {
    const int nvec = r.vec ? (r.hi - r.lo) >> 3 : 0;
#pragma unroll
    for (int j = 0; j < kVecPerThread; ++j) {
        const int vi = threadIdx.x + j * kVThreads;
        v[j] = (vi < nvec) ? ldnc128(r.src + r.lo + (size_t)vi * 8) : make_uint4(0, 0, 0, 0);
    }
}

__global__ void __launch_bounds__(kVThreads) verify_kernel(const bf16_t *__restrict__ logits,
                                                            const int32_t *__restrict__ drafts, int B, int K, int V,
                                                            int slices_per_row, int n_items, int32_t *accept_len, int32_t *bonus,
                                                            int32_t *out_argmax, unsigned long long *keys,
                                                            uint32_t *counter, uint32_t *status,
                                                            uint32_t *user_status) {
    __shared__ unsigned long long wkey[kVThreads / 32];
    __shared__ int is_last;
    const int i0 = (int)(((long long)blockIdx.x * n_items) / gridDim.x);
    const int i1 = (int)(((long long)(blockIdx.x + 1) * n_items) / gridDim.x);
    float best = -INFINITY;
    int idx = kNoIdx, cur_row = -1;

    // publishes this CTA's winner of row `row`
    auto flush = [&](int row) {
        unsigned long long key = (idx == kNoIdx) ? 0ull : argmax_key(best, (uint32_t)idx);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            unsigned long long other = __shfl_xor_sync(0xffffffffu, key, o);
            key = other > key ? other : key;
        }
        __syncthreads();                                   // wkey free again
        if ((threadIdx.x & 31) == 0) wkey[threadIdx.x >> 5] = key;
        __syncthreads();
        if (threadIdx.x == 0) {
            unsigned long long m = 0ull;
            for (int w = 0; w < kVThreads / 32; ++w) m = wkey[w] > m ? wkey[w] : m;
            if (m != 0ull) atomicMax(keys + row, m);
        }
    };

    uint4 cur[kVecPerThread], nxt[kVecPerThread];
    SliceRef rc = slice_ref(logits, V, slices_per_row, i0 < i1 ? i0 : 0), rn = rc;
    if (i0 < i1) slice_load(rc, cur);
    for (int item = i0; item < i1; ++item) {
        if (item + 1 < i1) {                               // the next slice's loads go out before this one's values are used
            rn = slice_ref(logits, V, slices_per_row, item + 1);
            slice_load(rn, nxt);
        }
        const int row = item / slices_per_row;
        if (row != cur_row) {
            if (cur_row >= 0) flush(cur_row);
            best = -INFINITY; idx = kNoIdx; cur_row = row;
        }
        if (rc.vec) {
            const int nvec = (rc.hi - rc.lo) >> 3;
#pragma unroll
            for (int j = 0; j < kVecPerThread; ++j) {
                int vi = threadIdx.x + j * kVThreads;
                if (vi < nvec) {
                    int e0 = rc.lo + vi * 8;
                    uint32_t w[4] = {cur[j].x, cur[j].y, cur[j].z, cur[j].w};
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        consider(bf16lo_f32(w[q]), e0 + 2 * q, best, idx);
                        consider(bf16hi_f32(w[q]), e0 + 2 * q + 1, best, idx);
                    }
                }
            }
            for (int i = rc.lo + (nvec << 3) + threadIdx.x; i < rc.hi; i += kVThreads)   // ragged tail
                consider(bf16bits_f32(rc.src[i]), i, best, idx);
        } else {
            for (int i = rc.lo + threadIdx.x; i < rc.hi; i += kVThreads) consider(bf16bits_f32(rc.src[i]), i, best, idx);
        }
        rc = rn;
#pragma unroll
        for (int j = 0; j < kVecPerThread; ++j) cur[j] = nxt[j];
    }
    if (cur_row >= 0) flush(cur_row);
    if (threadIdx.x == 0) {
        __threadfence();
        uint32_t old = atomicAdd(counter, 1u);
        is_last = (old == gridDim.x - 1);
    }
    __syncthreads();
    if (!is_last) return;

    // ---- last CTA: accept lengths
    __threadfence();
    const int M = K + 1;
    for (int b = threadIdx.x; b < B; b += kVThreads) {
        int a = 0;
        bool open = true;
        int bon = 0;
        for (int j = 0; j < M; ++j) {
            unsigned long long k = ldcg_u64(keys + (size_t)b * M + j);
            int g = 0;
            if ((k >> 32) == 0ull) { atomicOr(status, 0x10u); if (user_status) atomicOr(user_status, 0x10u); }
            else g = (int)argmax_key_id(k);
            if (out_argmax) out_argmax[(size_t)b * M + j] = g;
            if (open) {
                bon = g;
                if (j < K && drafts[(size_t)b * K + j] == g) a = j + 1;
                else open = false;
            }
        }
        accept_len[b] = a;
        bonus[b] = bon;
    }
    __syncthreads();
    for (int i = threadIdx.x; i < B * M; i += kVThreads) keys[i] = 0ull;
    if (threadIdx.x == 0) *counter = 0u;
}

// The acceptance rule alone, for callers that already hold the target's greedy token of every row
// (fastmtp_target_step's out_argmax): one thread per sequence walks its K drafts.
__global__ void accept_ids_kernel(const int32_t *__restrict__ target_argmax, const int32_t *__restrict__ drafts, int B, int K,
                                  int32_t *accept_len, int32_t *bonus) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    const int32_t *g = target_argmax + (size_t)b * (K + 1);
    int a = 0;
    while (a < K && drafts[(size_t)b * K + a] == g[a]) ++a;
    accept_len[b] = a;
    bonus[b] = g[a];
}

}  // namespace

int accept_ids_launch(const int32_t *target_argmax, const int32_t *drafts, int B, int K, int32_t *accept_len, int32_t *bonus,
                      cudaStream_t stream) {
    accept_ids_kernel<<<(B + 127) / 128, 128, 0, stream>>>(target_argmax, drafts, B, K, accept_len, bonus);
    return (int)cudaGetLastError();
}

int verify_launch(const bf16_t *logits, const int32_t *drafts, int B, int K, int V, int32_t *accept_len,
                  int32_t *bonus, int32_t *out_argmax, unsigned long long *keys, uint32_t *counter,
                  uint32_t *status, uint32_t *user_status, int n_sm, cudaStream_t stream) {
    if (n_sm <= 0) {                       // a caller without a context: ask the device (no allocation involved)
        int dev = 0;
        cudaError_t e = cudaGetDevice(&dev);
        if (e == cudaSuccess) e = cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return (int)e;
    }
    const int slices = (V + kSlice - 1) / kSlice;
    const long long items = (long long)B * (K + 1) * slices;
    const int grid = (int)(items < (long long)n_sm * kVCtasPerSm ? items : (long long)n_sm * kVCtasPerSm);
    verify_kernel<<<grid, kVThreads, 0, stream>>>(logits, drafts, B, K, V, slices, (int)items, accept_len, bonus, out_argmax,
                                                  keys, counter, status, user_status);
    return (int)cudaGetLastError();
}

}  // namespace fmtp
