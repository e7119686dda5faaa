// Batched draft path (Sec. 2.1 recursion, Sec. 2.2 Eq. 3 compressed head) for groups of up to 64
// sequences: per step, six weight-streaming tcgen05 GEMMs (skinny_gemm.cuh) and the small
// row-wise kernels between them (norms, rotary embedding + cache append, attention, residuals).
// All kernels of a call are enqueued on the caller's stream; none waits on another CTA.
#include "batched.cuh"
#include "skinny_gemm.cuh"

namespace fmtp {

namespace {

constexpr uint32_t kDevBadToken = 0x1u, kDevBadPage = 0x2u, kDevBadPos = 0x4u, kDevAllNan = 0x10u;
constexpr int kRowThreads = 512;

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

__device__ __forceinline__ float block_sum(float v, float *red) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
    __syncthreads();
    if (lane == 0) red[warp] = v;
    __syncthreads();
    float t = 0.f;
    for (int w = 0; w < nw; ++w) t += red[w];     // same order on every thread
    return t;
}

__device__ __forceinline__ void store_hilo(bf16_t *xop, int ld, int r, int j, float v) {
    uint16_t hi, lo;
    split_bf16(v, hi, lo);
    xop[(size_t)(2 * r) * ld + j] = hi;
    xop[(size_t)(2 * r + 1) * ld + j] = lo;
}

// ---- rows of a launch. Row r belongs to sequence r / M. In a target step the M rows of a sequence sit at
// positions L .. L+M-1. In draft step 0 they are the sequence's extend rows (Sec. 2.3 "Drafting phase":
// the pairs of target hidden state and next token committed since the last call), n = n_ext[seq] of them
// at positions L .. L+n-1, the last one being draft step 1; rows beyond n are padding (computed, never
// stored or published). A later draft step has one row per sequence at position L + n - 1 + step.
struct RowGeo {
    int M;                   // rows per sequence in this launch
    int M0;                  // rows per sequence of draft step 0 (the bound of n_ext); target step: M
    int step;                // draft step (0 in a target step)
    const int32_t *n_ext;    // [sequences] or NULL (= M0 for every sequence)
};
__device__ __forceinline__ int geo_next(const RowGeo &g, int seq) { return g.n_ext ? min(max(g.n_ext[seq], 1), g.M0) : g.M0; }
// Position of row r (before clamping to the cache's capacity); *valid = false for a padding row.
__device__ __forceinline__ int geo_pos(const RowGeo &g, const KvPtrs &kv, int r, bool *valid) {
    const int seq = r / g.M, m = r - seq * g.M;
    const int L = max(kv.seq_lens[seq], 0);
    if (g.step > 0) { *valid = true; return L + geo_next(g, seq) - 1 + g.step; }
    const int n = geo_next(g, seq);
    *valid = m < n;
    return L + min(m, n - 1);
}
// Extend step of a draft: only the last extend row of a sequence publishes its result (hidden state, head
// operand), under the sequence's index; -1 for every other row.
__device__ __forceinline__ int geo_out_seq(const RowGeo &g, int r) {
    const int seq = r / g.M, m = r - seq * g.M;
    return m == geo_next(g, seq) - 1 ? seq : -1;
}

// ---- step input: [rms(h; g_h) ; rms(Emb(tok); g_e)] as the projection's operand; also turns the
// previous step's argmax key into its draft token. One block per sequence.
struct PrologueArgs {
    int step, K, d, V, ld, only_tokens;
    RowGeo geo;                  // step 0 of a draft with extend rows: which rows are padding
    float eps;
    const bf16_t *h_last;
    const int32_t *tok_last;
    const float *hout;
    const unsigned long long *keys_prev;
    int32_t *out_drafts;
    const bf16_t *embed, *g_h, *g_e;
    bf16_t *xop;
    uint32_t *status, *user_status;
};

// eight consecutive values -> hi/lo bf16, one 16-byte store each
__device__ __forceinline__ void store_hilo8(bf16_t *xop, int ld, int r, int j, const float (&v)[8]) {
    uint32_t hi[4], lo[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        uint16_t h0, l0, h1, l1;
        split_bf16(v[2 * i], h0, l0);
        split_bf16(v[2 * i + 1], h1, l1);
        hi[i] = (uint32_t)h0 | ((uint32_t)h1 << 16);
        lo[i] = (uint32_t)l0 | ((uint32_t)l1 << 16);
    }
    *reinterpret_cast<uint4 *>(xop + (size_t)(2 * r) * ld + j) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
    *reinterpret_cast<uint4 *>(xop + (size_t)(2 * r + 1) * ld + j) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
}
__device__ __forceinline__ void unpack_bf16x8(const uint4 &u, float (&v)[8]) {
    v[0] = bf16lo_f32(u.x); v[1] = bf16hi_f32(u.x); v[2] = bf16lo_f32(u.y); v[3] = bf16hi_f32(u.y);
    v[4] = bf16lo_f32(u.z); v[5] = bf16hi_f32(u.z); v[6] = bf16lo_f32(u.w); v[7] = bf16hi_f32(u.w);
}
__device__ __forceinline__ void load_f32x8(const float *p, float (&v)[8]) {
    const float4 a = *reinterpret_cast<const float4 *>(p), b = *reinterpret_cast<const float4 *>(p + 4);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}

// Each thread owns eight consecutive columns per pass (d % 64 == 0), so every load and store is 16 bytes.
__global__ void __launch_bounds__(kRowThreads) prologue_kernel(const PrologueArgs a) {
    chain_release();
    chain_wait();
    __shared__ float red[32];
    __shared__ int s_tok;
    const int r = blockIdx.x, tid = threadIdx.x;
    if (tid == 0) {
        int tok;
        if (a.step == 0) {
            const int seq = r / a.geo.M;                   // a padding row's token is never looked at
            tok = (r - seq * a.geo.M < geo_next(a.geo, seq)) ? a.tok_last[r] : 0;
        } else {
            tok = 0;
            if (a.out_drafts) {
                const unsigned long long key = a.keys_prev[r];
                if ((key >> 32) == 0ull) atomicOr(a.status, kDevAllNan);
                tok = (int)argmax_key_id(key);
                a.out_drafts[(size_t)r * a.K + (a.step - 1)] = tok;
            }
        }
        if ((unsigned)tok >= (unsigned)a.V) { atomicOr(a.status, kDevBadToken); tok = 0; }
        s_tok = tok;
    }
    __syncthreads();
    if (a.only_tokens) {
        // last kernel of the call: hand the status word (earlier kernels' flags and this block's) to the caller
        if (tid == 0 && a.user_status) {
            __threadfence();
            const uint32_t st = *reinterpret_cast<volatile uint32_t *>(a.status);
            if (st) atomicOr(a.user_status, st);
        }
        return;
    }
    const bf16_t *erow = a.embed + (size_t)s_tok * a.d;
    float sh = 0.f, se = 0.f;
    for (int j = tid * 8; j < a.d; j += kRowThreads * 8) {
        float h[8], e[8];
        if (a.step == 0) unpack_bf16x8(*reinterpret_cast<const uint4 *>(a.h_last + (size_t)r * a.d + j), h);
        else load_f32x8(a.hout + (size_t)r * a.d + j, h);
        unpack_bf16x8(*reinterpret_cast<const uint4 *>(erow + j), e);
#pragma unroll
        for (int i = 0; i < 8; ++i) { sh += h[i] * h[i]; se += e[i] * e[i]; }
    }
    sh = block_sum(sh, red);
    se = block_sum(se, red);
    const float rh = 1.0f / sqrtf(sh / (float)a.d + a.eps), re = 1.0f / sqrtf(se / (float)a.d + a.eps);
    for (int j = tid * 8; j < a.d; j += kRowThreads * 8) {
        float h[8], e[8], gh[8], ge[8];
        if (a.step == 0) unpack_bf16x8(*reinterpret_cast<const uint4 *>(a.h_last + (size_t)r * a.d + j), h);
        else load_f32x8(a.hout + (size_t)r * a.d + j, h);
        unpack_bf16x8(*reinterpret_cast<const uint4 *>(erow + j), e);
        unpack_bf16x8(*reinterpret_cast<const uint4 *>(a.g_h + j), gh);
        unpack_bf16x8(*reinterpret_cast<const uint4 *>(a.g_e + j), ge);
#pragma unroll
        for (int i = 0; i < 8; ++i) { h[i] = h[i] * rh * gh[i]; e[i] = e[i] * re * ge[i]; }
        store_hilo8(a.xop, a.ld, r, j, h);
        store_hilo8(a.xop, a.ld, r, a.d + j, e);
    }
}

// ---- after a split-K GEMM: x = (residual ? x : 0) + sum of the partials; operand of the next
// GEMM = rms(x; gain) as hi/lo. With `final`: the normed vector is the step's output hidden state.
struct PostArgs {
    int d, splits, rows, ldp, ld, residual, final, K, step;
    int map_out, seq0;           // final norm of a draft's extend step: row r publishes as sequence seq0 + geo_out_seq(r)
    RowGeo geo;
    float eps;
    const float *partial;
    float *x, *hout;
    bf16_t *out_h;
    const bf16_t *gain;
    bf16_t *xop;
};

__global__ void __launch_bounds__(kRowThreads) post_kernel(const PostArgs a) {
    chain_release();
    chain_wait();
    __shared__ float red[32];
    const int r = blockIdx.x, tid = threadIdx.x;
    float ss = 0.f;
    for (int j = tid * 8; j < a.d; j += kRowThreads * 8) {
        float v[8], part[kBatchMaxSplits][8];
        // every load of this pass is issued before the first use
#pragma unroll
        for (int s = 0; s < kBatchMaxSplits; ++s)
            if (s < a.splits) load_f32x8(a.partial + ((size_t)s * a.rows + r) * a.ldp + j, part[s]);
        if (a.residual) load_f32x8(a.x + (size_t)r * a.d + j, v);
        else {
#pragma unroll
            for (int i = 0; i < 8; ++i) v[i] = 0.f;
        }
#pragma unroll
        for (int s = 0; s < kBatchMaxSplits; ++s)
            if (s < a.splits) {
#pragma unroll
                for (int i = 0; i < 8; ++i) v[i] += part[s][i];
            }
        *reinterpret_cast<float4 *>(a.x + (size_t)r * a.d + j) = make_float4(v[0], v[1], v[2], v[3]);
        *reinterpret_cast<float4 *>(a.x + (size_t)r * a.d + j + 4) = make_float4(v[4], v[5], v[6], v[7]);
#pragma unroll
        for (int i = 0; i < 8; ++i) ss += v[i] * v[i];
    }
    ss = block_sum(ss, red);
    const float rs = 1.0f / sqrtf(ss / (float)a.d + a.eps);
    int dst = r;
    if (a.map_out) {
        const int o = geo_out_seq(a.geo, r);
        if (o < 0) return;                       // an extend row that is not its sequence's last: nothing to publish
        dst = a.seq0 + o;
    }
    for (int j = tid * 8; j < a.d; j += kRowThreads * 8) {
        float v[8], gn[8];
        load_f32x8(a.x + (size_t)r * a.d + j, v);
        unpack_bf16x8(*reinterpret_cast<const uint4 *>(a.gain + j), gn);
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = v[i] * rs * gn[i];
        store_hilo8(a.xop, a.ld, dst, j, v);
        if (a.final) {
            *reinterpret_cast<float4 *>(a.hout + (size_t)dst * a.d + j) = make_float4(v[0], v[1], v[2], v[3]);
            *reinterpret_cast<float4 *>(a.hout + (size_t)dst * a.d + j + 4) = make_float4(v[4], v[5], v[6], v[7]);
            if (a.out_h) {
                uint32_t o[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) o[i] = (uint32_t)f32_bf16bits(v[2 * i]) | ((uint32_t)f32_bf16bits(v[2 * i + 1]) << 16);
                *reinterpret_cast<uint4 *>(a.out_h + ((size_t)dst * a.K + a.step) * a.d + j) = make_uint4(o[0], o[1], o[2], o[3]);
            }
        }
    }
}

// ---- after the QKV GEMM: sum the partials, rotate q and k at the row's position, keep q in fp32,
// append k and v (rounded to bf16) to the paged cache. Block = (head, sequence), dh/2 threads.
struct QkvArgs {
    int qdim, kvdim, dh, Hq, Hkv, splits, rows, ldp, page, max_ctx;
    RowGeo geo;                  // which sequence and position a row has
    const float *partial;
    float *q;
    KvPtrs kv;
    const float *rope_cos, *rope_sin;
    uint32_t *status;
};

__global__ void qkv_finish_kernel(const QkvArgs a) {
    chain_release();
    chain_wait();
    const int head = blockIdx.x, r = blockIdx.y, e = threadIdx.x, half = a.dh >> 1;
    const int max_tokens = min(a.kv.max_pages * a.page, a.max_ctx);
    const int seq = r / a.geo.M;
    bool valid;
    const int pos_true = geo_pos(a.geo, a.kv, r, &valid);
    const int pos = min(pos_true, max_tokens - 1);
    const int col = head * a.dh;              // q heads, then k heads, then v heads: the GEMM's row order
    float lo = 0.f, hi = 0.f;
    for (int s = 0; s < a.splits; ++s) {
        const float *pp = a.partial + ((size_t)s * a.rows + r) * a.ldp + col;
        lo += pp[e];
        hi += pp[e + half];
    }
    if (head < a.Hq + a.Hkv) {
        const float cs = a.rope_cos[(size_t)pos * half + e], sn = a.rope_sin[(size_t)pos * half + e];
        const float x = lo, y = hi;
        lo = x * cs - y * sn;
        hi = y * cs + x * sn;
    }
    if (head < a.Hq) {
        // stored ready for the attention MMA: scaled by log2(e) / sqrt(dh), each value as its two bf16 parts
        // (hi in the low half-word, lo in the high one)
        const float sc = (1.0f / sqrtf((float)a.dh)) * 1.4426950408889634f;
        uint32_t *qq = reinterpret_cast<uint32_t *>(a.q);
        uint16_t h0, l0, h1, l1;
        split_bf16(lo * sc, h0, l0);
        split_bf16(hi * sc, h1, l1);
        qq[(size_t)r * a.qdim + col + e] = (uint32_t)h0 | ((uint32_t)l0 << 16);
        qq[(size_t)r * a.qdim + col + e + half] = (uint32_t)h1 | ((uint32_t)l1 << 16);
        return;
    }
    if (!valid) return;                       // padding row: nothing to store
    if (pos_true >= max_tokens) {             // no slot for this position: flagged, nothing written
        if (head == a.Hq && e == 0) atomicOr(a.status, kDevBadPos);
        return;
    }
    const bool is_k = head < a.Hq + a.Hkv;
    const int kvh = is_k ? head - a.Hq : head - a.Hq - a.Hkv;
    int page = a.kv.block_table[(size_t)seq * a.kv.max_pages + pos / a.page];
    if ((unsigned)page >= (unsigned)a.kv.num_pages) { atomicOr(a.status, kDevBadPage); page = 0; }
    bf16_t *dst = (is_k ? a.kv.k_pages : a.kv.v_pages) + (((size_t)page * a.Hkv + kvh) * a.page + (pos % a.page)) * a.dh;
    dst[e] = f32_bf16bits(lo);
    dst[e + half] = f32_bf16bits(hi);
}

// ---- attention. A work item is one 256-token chunk of one (sequence, KV head); the Hq/Hkv query
// heads of the group share the K/V stream. One persistent CTA per SM walks its items (item index =
// CTA, CTA + grid, ...) as one continuous stream of 64-token blocks through a shared-memory ring,
// so the copies of the next items are in flight while the current one is computed. Scores and the
// weighted sum run on mma.sync.m16n8k16 with the query (and the probabilities) as the A operand,
// rows 0-7 the high bf16 parts of the heads and rows 8-15 the low parts, so both products carry
// fp32-accurate inputs. Each warp owns 16 tokens of every block and keeps its own running
// (max, sum, output); the four warps merge in fixed order at the end of the item.
// Output per item: unnormalised o, running max m and sum l per head.
struct AttnArgs {
    int Hq, Hkv, dh, page, page_shift, max_ctx, max_chunks, B;    // B: rows
    RowGeo geo;                  // which sequence and position a row has
    unsigned long long wait_limit_ns;   // a ring wait gives up after this long
    const float *q;              // [rows][Hq*dh] words: the scaled query values as {hi, lo} bf16 pairs
    KvPtrs kv;
    float *att_part;             // [rows][Hq][max_chunks][dh+2]
    uint32_t *status;
};

constexpr int kAttnBlk = 64;                 // tokens per ring stage
constexpr int kAttnStages = 5;
constexpr int kAttnThreads = 128;            // compute threads (warps 0-3); warps 4-7 only issue the copies

struct AttnItem {                            // one (sequence, KV head, chunk), CTA-uniform
    int r, kvh, chunk, t0, n_ctx, n_blk;
    const int32_t *bt;
};

template <int DH>
struct AttnSmem {
    static constexpr int ROWB = DH * 2 + 16;                     // padded row: conflict-free fragment loads
    static constexpr int QB = 8 * DH * 4;                        // the group's query vectors (fp32)
    static constexpr int STAGE = 2 * kAttnBlk * ROWB + QB;       // K block, V block, queries (first block of an item)
    static constexpr int MERGE = 4 * 8 * (DH + 2) * 4 + 64 * 4;  // per-warp (o, m, l) of 8 heads, then 4 x 8 weights, 8 maxima, 8 sums
    static constexpr int TOTAL = kAttnStages * STAGE + MERGE + (kBatchRows + 1) * 4 + kBatchRows * 4 + (2 * kAttnStages + 1) * 8;
};

template <int DH>
__global__ void __launch_bounds__(2 * kAttnThreads, 1) attn_kernel(const AttnArgs a) {
    chain_release();
    chain_wait();
    using L = AttnSmem<DH>;
    constexpr int ROWB = L::ROWB, STAGE = L::STAGE;
    extern __shared__ __align__(16) unsigned char smem[];
    float *mo = reinterpret_cast<float *>(smem + kAttnStages * STAGE);                    // [4][8][DH + 2]
    // 8-byte barriers first (STAGE and MERGE are multiples of 16), then the 4-byte tables
    uint64_t *full = reinterpret_cast<uint64_t *>(smem + kAttnStages * STAGE + L::MERGE);  // [stages] copies landed
    uint64_t *empty = full + kAttnStages;                                                  // [stages] stage consumed
    volatile uint32_t *abort_flag = reinterpret_cast<volatile uint32_t *>(empty + kAttnStages);
    int *prefix = reinterpret_cast<int *>(empty + kAttnStages + 1);                        // [B + 1] chunks before sequence r
    int *nctx = prefix + kBatchRows + 1;
    const bool producer = threadIdx.x >= kAttnThreads;
    const int tid = threadIdx.x & (kAttnThreads - 1), warp = tid >> 5, lane = tid & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < kAttnStages; ++s) { mbar_init(&full[s], kAttnThreads); mbar_init(&empty[s], kAttnThreads); }
        *abort_flag = 0;
        mbar_fence_init();
    }
    // a wait that gives up after two seconds (or when another thread has), so a logic error cannot hang the device
    auto wait = [&](uint64_t *bar, uint32_t parity) -> bool {
        if (mbar_try_wait(bar, parity)) return true;
        const unsigned long long t_begin = global_timer_ns();
        uint32_t polls = 0;
        while (!mbar_try_wait(bar, parity)) {
            if ((++polls & 63u) == 0) {
                if (*abort_flag) return false;
                if (global_timer_ns() - t_begin > a.wait_limit_ns) { *abort_flag = 1u; return false; }
            }
        }
        return true;
    };
    const int gq = a.Hq / a.Hkv;
    const int max_tokens = min(a.kv.max_pages * a.page, a.max_ctx);
    if (threadIdx.x < a.B) {     // visible positions 0 .. n-1 of every row
        bool valid;
        nctx[threadIdx.x] = min(geo_pos(a.geo, a.kv, threadIdx.x, &valid), max_tokens - 1) + 1;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int acc = 0;
        for (int r = 0; r < a.B; ++r) { prefix[r] = acc; const int ct = attn_chunk_tokens(nctx[r]); acc += (nctx[r] + ct - 1) / ct; }
        prefix[a.B] = acc;
    }
    __syncthreads();
    const int n_items = prefix[a.B] * a.Hkv;

    auto load_item = [&](AttnItem &it, int item) {
        const int cidx = item / a.Hkv;
        it.kvh = item - cidx * a.Hkv;
        int r = it.r;                        // a CTA's items come in ascending order: search on from the last one
        while (prefix[r + 1] <= cidx) ++r;
        it.r = r;
        it.chunk = cidx - prefix[r];
        it.n_ctx = nctx[r];
        const int ct = attn_chunk_tokens(it.n_ctx);
        it.t0 = it.chunk * ct;
        it.n_blk = (min(ct, it.n_ctx - it.t0) + kAttnBlk - 1) / kAttnBlk;
        it.bt = a.kv.block_table + (size_t)(r / a.geo.M) * a.kv.max_pages;
    };

    if (producer) {
    // ---- copy warps: block fb of item fc goes into stage fi % kAttnStages once its previous reader is done.
    // The block-table entries of a block are loaded one block ahead, so their latency is off the issue path.
    constexpr int PIECES = DH / 8;                      // 16-byte pieces per row
    constexpr int NIT = kAttnBlk * PIECES / kAttnThreads;
    constexpr int TSTEP = kAttnThreads / PIECES;        // tokens between a thread's consecutive pieces
    const int pc = tid % PIECES, tl = tid / PIECES;
    const uint64_t kv_policy = l2_evict_first();
    auto load_pages = [&](const AttnItem &it_, int blk, int (&pg)[NIT]) {
#pragma unroll
        for (int it = 0; it < NIT; ++it) {
            int pos = it_.t0 + blk * kAttnBlk + tl + it * TSTEP;
            if (pos >= it_.n_ctx) pos = it_.n_ctx - 1;
            pg[it] = it_.bt[a.page_shift >= 0 ? pos >> a.page_shift : pos / a.page];
        }
    };
    AttnItem fc, fn;
    fc.r = 0;
    int f_item = blockIdx.x, fb = 0, fi = 0;
    int pg_cur[NIT], pg_next[NIT];
    if (f_item < n_items) { load_item(fc, f_item); load_pages(fc, 0, pg_cur); }
    while (f_item < n_items) {
        // where the next block is, and its block-table entries
        int n_item = f_item, nb = fb + 1;
        fn = fc;
        if (nb == fc.n_blk) {
            nb = 0;
            n_item += gridDim.x;
            if (n_item < n_items) load_item(fn, n_item);
        }
        if (n_item < n_items) load_pages(fn, nb, pg_next);
        const int stage = fi % kAttnStages;
        if (!wait(&empty[stage], ((fi / kAttnStages) & 1) ^ 1)) break;
        unsigned char *st = smem + (size_t)stage * STAGE;
        size_t off[NIT];
        uint32_t ok[NIT];
#pragma unroll
        for (int it = 0; it < NIT; ++it) {
            int pos = fc.t0 + fb * kAttnBlk + tl + it * TSTEP;
            ok[it] = pos < fc.n_ctx ? 16u : 0u;
            if (pos >= fc.n_ctx) pos = fc.n_ctx - 1;
            const int pgi = a.page_shift >= 0 ? pos >> a.page_shift : pos / a.page;
            const int in_page = pos - pgi * a.page;
            int page = pg_cur[it];
            if ((unsigned)page >= (unsigned)a.kv.num_pages) { atomicOr(a.status, kDevBadPage); page = 0; }
            off[it] = (((size_t)page * a.Hkv + fc.kvh) * a.page + in_page) * DH + pc * 8;
        }
        const uint32_t d0 = smem_u32(st + tl * ROWB + pc * 16);
#pragma unroll
        for (int it = 0; it < NIT; ++it) {
            cp_async16_off_hint<0>(d0 + it * TSTEP * ROWB, a.kv.k_pages + off[it], ok[it], kv_policy);
            cp_async16_off_hint<0>(d0 + kAttnBlk * ROWB + it * TSTEP * ROWB, a.kv.v_pages + off[it], ok[it], kv_policy);
        }
        if (fb == 0) {     // the item's query vectors ride with its first block
            const float *qsrc = a.q + ((size_t)fc.r * a.Hq + (size_t)fc.kvh * gq) * DH;    // packed {hi, lo} words
            for (int i = tid; i < gq * DH / 4; i += kAttnThreads)
                cp_async16_off<0>(smem_u32(st + 2 * kAttnBlk * ROWB + i * 16), qsrc + i * 4, 16u);
        }
        cp_async_arrive(&full[stage]);      // this thread's arrival fires when its copies above have landed
        ++fi;
        fc = fn; f_item = n_item; fb = nb;
#pragma unroll
        for (int it = 0; it < NIT; ++it) pg_cur[it] = pg_next[it];
    }
    cp_async_wait_all();
    } else {

    // ---- compute side
    const int hrow = lane >> 2, kq = (lane & 3) * 2;
    AttnItem cc;
    cc.r = 0;
    int c_item = blockIdx.x, cb = 0, ci = 0;
    if (c_item < n_items) load_item(cc, c_item);
    uint32_t qa[DH / 16][4];
    float m_run = -INFINITY, l_run = 0.f;       // of head hrow, this warp's tokens (replicated on the 4 lanes of a row)
    float o[DH / 8][4];                          // MMA accumulators: [0],[1] the hi-part products, [2],[3] the lo-part ones
    while (c_item < n_items) {
        const int stage = ci % kAttnStages;
        // the 128 compute threads agree on the outcome of the wait before any of them moves on
        if (epi_any(!wait(&full[stage], (ci / kAttnStages) & 1))) break;
        const unsigned char *sk = smem + (size_t)stage * STAGE;
        const unsigned char *sv = sk + kAttnBlk * ROWB;
        if (cb == 0) {
            // query fragments: A rows 0-7 = hi parts of heads 0..gq-1, rows 8-15 = lo parts
            // (the rotary kernel stored every query value as {hi, lo} bf16 halves of one word, already scaled)
            const uint32_t *qh = reinterpret_cast<const uint32_t *>(sv + kAttnBlk * ROWB) + hrow * DH;
#pragma unroll
            for (int ks = 0; ks < DH / 16; ++ks) {
                uint2 w0 = make_uint2(0u, 0u), w1 = make_uint2(0u, 0u);
                if (hrow < gq) {
                    w0 = *reinterpret_cast<const uint2 *>(qh + ks * 16 + kq);
                    w1 = *reinterpret_cast<const uint2 *>(qh + ks * 16 + kq + 8);
                }
                qa[ks][0] = __byte_perm(w0.x, w0.y, 0x5410);      // row hrow (hi parts), k = kq, kq+1
                qa[ks][1] = __byte_perm(w0.x, w0.y, 0x7632);      // row hrow + 8 (lo parts)
                qa[ks][2] = __byte_perm(w1.x, w1.y, 0x5410);      // row hrow,     k = kq+8, kq+9
                qa[ks][3] = __byte_perm(w1.x, w1.y, 0x7632);
            }
            m_run = -INFINITY; l_run = 0.f;
#pragma unroll
            for (int nt = 0; nt < DH / 8; ++nt) o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f;
        }
        const int tw = warp * 16;                              // this warp's tokens inside the block
        const int tbase = cc.t0 + cb * kAttnBlk + tw;
        if (tbase < cc.n_ctx) {
            // scores: two n-tiles of 8 tokens; one ldmatrix.x4 brings both tiles' K fragments of a 16-wide slice
            float s[2][4];
            s[0][0] = s[0][1] = s[0][2] = s[0][3] = 0.f;
            s[1][0] = s[1][1] = s[1][2] = s[1][3] = 0.f;
            const uint32_t kaddr = smem_u32(sk) + (uint32_t)((tw + (lane & 7) + ((lane >> 4) << 3)) * ROWB + ((lane >> 3) & 1) * 16);
#pragma unroll
            for (int ks = 0; ks < DH / 16; ++ks) {
                uint32_t b00, b01, b10, b11;
                asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                             : "=r"(b00), "=r"(b01), "=r"(b10), "=r"(b11) : "r"(kaddr + ks * 32));
                mma_bf16(s[0], qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3], b00, b01);
                mma_bf16(s[1], qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3], b10, b11);
            }
            // thread holds, for head hrow: tokens tw + nt*8 + kq + {0,1}: hi part in [0],[1], lo part in [2],[3]
            float sc[4];
            float mx = -INFINITY;
#pragma unroll
            for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                    float v = s[nt][j] + s[nt][j + 2];
                    if (tbase + nt * 8 + kq + j >= cc.n_ctx) v = -INFINITY;
                    sc[nt * 2 + j] = v;
                    mx = fmaxf(mx, v);
                }
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
            const float m_new = fmaxf(m_run, mx);                 // finite: the warp's first token is visible
            const float corr = exp2f(m_run - m_new);              // 0 on the item's first block (m_run = -inf)
            float psum = 0.f;
            uint32_t pa[4];
            {
                float pr[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) { pr[i] = exp2f(sc[i] - m_new); psum += pr[i]; }
                uint16_t h0, l0, h1, l1, h2, l2, h3, l3;
                split_bf16(pr[0], h0, l0); split_bf16(pr[1], h1, l1); split_bf16(pr[2], h2, l2); split_bf16(pr[3], h3, l3);
                pa[0] = (uint32_t)h0 | ((uint32_t)h1 << 16);      // row hrow,   tokens kq, kq+1
                pa[1] = (uint32_t)l0 | ((uint32_t)l1 << 16);      // row hrow+8
                pa[2] = (uint32_t)h2 | ((uint32_t)h3 << 16);      // row hrow,   tokens 8+kq, 8+kq+1
                pa[3] = (uint32_t)l2 | ((uint32_t)l3 << 16);
            }
            psum += __shfl_xor_sync(0xffffffffu, psum, 1);
            psum += __shfl_xor_sync(0xffffffffu, psum, 2);
            l_run = l_run * corr + psum;
            m_run = m_new;
            // weighted sum, accumulated in the MMA: rescale the running output only when some row's maximum moved
            if (__any_sync(0xffffffffu, corr != 1.0f)) {
#pragma unroll
                for (int nt = 0; nt < DH / 8; ++nt) { o[nt][0] *= corr; o[nt][1] *= corr; o[nt][2] *= corr; o[nt][3] *= corr; }
            }
            // B[k = token][n = dim] read with a transposing ldmatrix from V[token][dim], two n-tiles per load
            const uint32_t vaddr = smem_u32(sv) + (uint32_t)((tw + (lane & 7) + ((lane >> 3) & 1) * 8) * ROWB + (lane >> 4) * 16);
#pragma unroll
            for (int nt = 0; nt < DH / 8; nt += 2) {
                uint32_t b00, b01, b10, b11;
                asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                             : "=r"(b00), "=r"(b01), "=r"(b10), "=r"(b11) : "r"(vaddr + nt * 16));
                mma_bf16(o[nt], pa[0], pa[1], pa[2], pa[3], b00, b01);
                mma_bf16(o[nt + 1], pa[0], pa[1], pa[2], pa[3], b10, b11);
            }
        }
        mbar_arrive(&empty[stage]);        // this thread has read all it needs from the stage
        ++ci;
        if (++cb == cc.n_blk) {
            // ---- end of the item: merge the four warps (fixed order) and write the chunk's partial
            float *dst = mo + ((size_t)warp * 8 + hrow) * (DH + 2);
#pragma unroll
            for (int nt = 0; nt < DH / 8; ++nt) { dst[nt * 8 + kq] = o[nt][0] + o[nt][2]; dst[nt * 8 + kq + 1] = o[nt][1] + o[nt][3]; }
            if ((lane & 3) == 0) { dst[DH] = m_run; dst[DH + 1] = l_run; }
            bar_sync(1, kAttnThreads);
            float *wgt = mo + 4 * 8 * (DH + 2);          // [4][8] weights, [8] maxima, [8] sums
            if (tid < 32) {                               // thread = (head tid >> 2, warp tid & 3)
                const int h = tid >> 2, w = tid & 3;
                float m = -INFINITY;
                for (int u = 0; u < 4; ++u) m = fmaxf(m, mo[((size_t)u * 8 + h) * (DH + 2) + DH]);
                const float mw = mo[((size_t)w * 8 + h) * (DH + 2) + DH];
                wgt[w * 8 + h] = mw == -INFINITY ? 0.f : exp2f(mw - m);
                if (w == 0) {
                    float l = 0.f;
                    for (int u = 0; u < 4; ++u) {         // ascending warp order
                        const float mu = mo[((size_t)u * 8 + h) * (DH + 2) + DH];
                        l += mo[((size_t)u * 8 + h) * (DH + 2) + DH + 1] * (mu == -INFINITY ? 0.f : exp2f(mu - m));
                    }
                    wgt[32 + h] = m;
                    wgt[40 + h] = l;
                }
            }
            bar_sync(1, kAttnThreads);
            for (int i = tid; i < gq * DH; i += kAttnThreads) {
                const int h = i / DH, j = i - h * DH;
                float acc = 0.f;
#pragma unroll
                for (int w = 0; w < 4; ++w) acc += mo[((size_t)w * 8 + h) * (DH + 2) + j] * wgt[w * 8 + h];
                float *out = a.att_part + (((size_t)cc.r * a.Hq + (size_t)cc.kvh * gq + h) * a.max_chunks + cc.chunk) * (DH + 2);
                out[j] = acc;
                if (j == 0) { out[DH] = wgt[32 + h] * 0.6931471805599453f; out[DH + 1] = wgt[40 + h]; }     // the chunk maximum in natural-log units
            }
            bar_sync(1, kAttnThreads);     // merge buffer free for the next item
            cb = 0;
            c_item += gridDim.x;
            if (c_item < n_items) load_item(cc, c_item);
        }
    }
    }
    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag) atomicOr(a.status, 0x8u);
}

// ---- combine a head's chunk partials in ascending order; write the O-projection's operand.
struct MergeArgs {
    int Hq, dh, page, max_ctx, max_chunks, ld;
    RowGeo geo;
    KvPtrs kv;
    const float *att_part;
    bf16_t *xop;
};

__global__ void attn_merge_kernel(const MergeArgs a) {
    chain_release();
    chain_wait();
    __shared__ float red[8];
    const int head = blockIdx.x, r = blockIdx.y, j = threadIdx.x;
    const int max_tokens = min(a.kv.max_pages * a.page, a.max_ctx);
    bool valid;
    const int n_ctx = min(geo_pos(a.geo, a.kv, r, &valid), max_tokens - 1) + 1;
    const int n_chunks = (n_ctx + attn_chunk_tokens(n_ctx) - 1) / attn_chunk_tokens(n_ctx);
    const int stride = a.dh + 2;
    const float *base = a.att_part + ((size_t)r * a.Hq + head) * a.max_chunks * stride;
    // the chunks' maxima: each thread reads some, then a block-wide maximum (exact, order-free)
    float m = -INFINITY;
    for (int c = j; c < n_chunks; c += blockDim.x) m = fmaxf(m, base[(size_t)c * stride + a.dh]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if ((j & 31) == 0) red[j >> 5] = m;
    __syncthreads();
    m = red[0];
    for (int w = 1; w < (int)(blockDim.x >> 5); ++w) m = fmaxf(m, red[w]);
    // weighted sums in ascending chunk order
    float acc = 0.f, l = 0.f;
    int c = 0;
    for (; c + 8 <= n_chunks; c += 8) {          // eight chunks' loads in flight, added in ascending order
        float mv[8], lv[8], ov[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const float *src = base + (size_t)(c + u) * stride;
            mv[u] = src[a.dh]; lv[u] = src[a.dh + 1]; ov[u] = src[j];
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const float f = expf(mv[u] - m);
            acc += ov[u] * f;
            l += lv[u] * f;
        }
    }
    for (; c + 2 <= n_chunks; c += 2) {
        float mv[2], lv[2], ov[2];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const float *src = base + (size_t)(c + u) * stride;
            mv[u] = src[a.dh]; lv[u] = src[a.dh + 1]; ov[u] = src[j];
        }
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const float f = expf(mv[u] - m);
            acc += ov[u] * f;
            l += lv[u] * f;
        }
    }
    for (; c < n_chunks; ++c) {
        const float *src = base + (size_t)c * stride;
        const float f = expf(src[a.dh] - m);
        acc += src[j] * f;
        l += src[a.dh + 1] * f;
    }
    store_hilo(a.xop, a.ld, r, head * a.dh + j, acc / l);
}

// ---- target step input: x = Emb(token) per row (fp32 residual stream). One block per row.
__global__ void __launch_bounds__(kRowThreads) embed_kernel(const int32_t *tokens, const bf16_t *embed, int d, int V, float *x,
                                                            uint32_t *status) {
    chain_release();
    chain_wait();
    const int r = blockIdx.x;
    int tok = tokens[r];
    if ((unsigned)tok >= (unsigned)V) { if (threadIdx.x == 0) atomicOr(status, kDevBadToken); tok = 0; }
    const bf16_t *erow = embed + (size_t)tok * d;
    for (int j = threadIdx.x * 8; j < d; j += kRowThreads * 8) {
        float e[8];
        unpack_bf16x8(*reinterpret_cast<const uint4 *>(erow + j), e);
        *reinterpret_cast<float4 *>(x + (size_t)r * d + j) = make_float4(e[0], e[1], e[2], e[3]);
        *reinterpret_cast<float4 *>(x + (size_t)r * d + j + 4) = make_float4(e[4], e[5], e[6], e[7]);
    }
}

// ---- the subset in ascending id order. The argmax over the subset does not depend on the order of
// its rows, and gathering head rows in address order keeps the 128 rows of a GEMM tile within a few
// memory pages (an unsorted subset spreads them over the whole matrix and the address translation
// misses cost ~25 % of the head's stream rate). Membership bitmap, then a one-block compaction.
// (The two kernels run under the first kernels of step 0; the head GEMM, the only reader of the sorted ids, waits
// for the whole chain before it looks at them.)
__global__ void ids_mark_kernel(const int32_t *ids, int N, int V, uint32_t *bitmap, uint32_t *status) {
    chain_release();
    chain_wait();
    for (int j = blockIdx.x * blockDim.x + threadIdx.x; j < N; j += gridDim.x * blockDim.x) {
        int id = ids[j];
        if ((unsigned)id >= (unsigned)V) { atomicOr(status, kDevBadToken); id = 0; }
        atomicOr(&bitmap[id >> 5], 1u << (id & 31));
    }
}

// Compaction of the membership bitmap into ascending ids. Block b owns a contiguous range of bitmap words; the
// number of ids before its range is the population count of all earlier words, which every block sums for itself
// (the whole bitmap is 19 KB at V = 152064), so no block waits for another. Duplicates in the caller's array leave
// fewer distinct ids than N: the tail repeats `fill` (a member of the subset; a repeated row cannot change an argmax).
constexpr int kCompactThreads = 256;
__global__ void __launch_bounds__(kCompactThreads) ids_compact_kernel(const uint32_t *bitmap, int n_words, int32_t *sorted, int N,
                                                                      const int32_t *ids, int V) {
    chain_release();
    chain_wait();
    __shared__ int wsum[kCompactThreads / 32];
    __shared__ int s_base, s_total;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int w0 = (int)(((long long)blockIdx.x * n_words) / gridDim.x), w1 = (int)(((long long)(blockIdx.x + 1) * n_words) / gridDim.x);
    // ids before this block's words, and in the whole bitmap
    int before = 0, all = 0;
    for (int w = tid; w < n_words; w += kCompactThreads) {
        const int c = __popc(bitmap[w]);
        all += c;
        if (w < w0) before += c;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) { before += __shfl_xor_sync(0xffffffffu, before, o); all += __shfl_xor_sync(0xffffffffu, all, o); }
    if (lane == 0) wsum[warp] = before;
    __syncthreads();
    if (tid == 0) { int t = 0; for (int w = 0; w < kCompactThreads / 32; ++w) t += wsum[w]; s_base = t; }
    __syncthreads();
    if (lane == 0) wsum[warp] = all;
    __syncthreads();
    if (tid == 0) { int t = 0; for (int w = 0; w < kCompactThreads / 32; ++w) t += wsum[w]; s_total = t; }
    __syncthreads();
    // this block's words: one word per thread and round, exclusive scan of the counts within the block
    int run = s_base;
    for (int r0 = w0; r0 < w1; r0 += kCompactThreads) {
        const int w = r0 + tid;
        uint32_t bits = w < w1 ? bitmap[w] : 0u;
        const int cnt = __popc(bits);
        int incl = cnt;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += t;
        }
        __syncthreads();
        if (lane == 31) wsum[warp] = incl;
        __syncthreads();
        int base = run;
        for (int q = 0; q < warp; ++q) base += wsum[q];
        int pos = base + incl - cnt;
        while (bits) {
            const int b = __ffs(bits) - 1;
            bits &= bits - 1;
            if (pos < N) sorted[pos] = w * 32 + b;
            ++pos;
        }
        for (int q = 0; q < kCompactThreads / 32; ++q) run += wsum[q];
    }
    if (blockIdx.x == 0) {
        int fill = ids[0];
        if ((unsigned)fill >= (unsigned)V) fill = 0;
        for (int j = min(s_total, N) + tid; j < N; j += kCompactThreads) sorted[j] = fill;
    }
}

int pick_splits(int n_tiles, int n_kb, int n_sm) {
    int best = 1;
    double best_eff = 0.0;
    for (int s = 1; s <= kBatchMaxSplits; ++s) {
        if (s > 1 && n_kb / s < 8) break;
        const int items = n_tiles * s;
        const int waves = (items + n_sm - 1) / n_sm;
        const double eff = (double)items / ((double)waves * n_sm);
        if (eff > best_eff + 0.02) { best_eff = eff; best = s; }
    }
    return best;
}

}  // namespace

size_t batched_layout(BatchedWs &ws, unsigned char *base, const BatchedShape &sh) {
    const int rows = sh.max_rows < kBatchRows ? sh.max_rows : kBatchRows;
    const int qdim = sh.Hq * sh.dh, kvdim = sh.Hkv * sh.dh;
    const int widest_in = 2 * sh.d > qdim ? 2 * sh.d : qdim;
    const int widest_out = sh.d > qdim + 2 * kvdim ? sh.d : qdim + 2 * kvdim;
    ws.rows = rows;
    ws.ld0 = (int)align_up((size_t)widest_in, 64);
    ws.ldF = (int)align_up((size_t)sh.F, 64);
    ws.ldp = (int)align_up((size_t)widest_out, 128);
    ws.max_chunks = (sh.max_ctx + kBatchAttnChunk - 1) / kBatchAttnChunk;
    size_t off = 0;
    auto take = [&](size_t bytes) {
        off = align_up(off, 256);
        unsigned char *p = base ? base + off : nullptr;
        off += bytes;
        return p;
    };
    ws.xop0 = reinterpret_cast<bf16_t *>(take((size_t)128 * ws.ld0 * 2));
    ws.xopF = reinterpret_cast<bf16_t *>(take((size_t)128 * ws.ldF * 2));
    ws.xopH = reinterpret_cast<bf16_t *>(take((size_t)128 * ws.ld0 * 2));
    ws.partial = reinterpret_cast<float *>(take((size_t)kBatchMaxSplits * rows * ws.ldp * 4));
    ws.x = reinterpret_cast<float *>(take((size_t)rows * sh.d * 4));
    ws.hout = reinterpret_cast<float *>(take((size_t)rows * sh.d * 4));
    ws.q = reinterpret_cast<float *>(take((size_t)rows * qdim * 4));
    ws.att_part = reinterpret_cast<float *>(take((size_t)rows * sh.Hq * ws.max_chunks * (sh.dh + 2) * 4));
    ws.keys_bytes = (size_t)(sh.max_K > 1 ? sh.max_K : 1) * kBatchRows * 8 + 256;
    ws.keys = reinterpret_cast<unsigned long long *>(take(ws.keys_bytes));
    ws.id_bitmap = reinterpret_cast<uint32_t *>(take((size_t)((sh.V + 31) / 32) * 4));
    ws.sorted_ids = reinterpret_cast<int32_t *>(take((size_t)sh.V * 4));
    ws.status = reinterpret_cast<uint32_t *>(reinterpret_cast<unsigned char *>(ws.keys) + ws.keys_bytes - 256);
    if (!base) ws.status = nullptr;
    return align_up(off, 256);
}

int batched_draft(const BatchedCall &c, cudaStream_t st, long long *launches) {
    const BatchedShape &sh = c.sh;
    const BatchedWs &ws = c.ws;
    const int B = c.B, K = c.K, d = sh.d;
    const int M0 = c.M0 > 1 ? c.M0 : 1;
    const bool ext = M0 > 1;                       // step 0 carries up to M0 extend rows per sequence
    int inject_left = c.inject_gemm_timeout ? 1 : 0;
    const int qdim = sh.Hq * sh.dh, kvdim = sh.Hkv * sh.dh;
    cudaError_t e = cudaMemsetAsync(ws.keys, 0, ws.keys_bytes, st);     // argmax keys and the status word
    if (e != cudaSuccess) return (int)e;

    // head rows in ascending id order (the debug logits keep the caller's order, so they skip this)
    const int32_t *head_ids = c.ids;
    if (c.ids && !c.out_logits) {
        const int n_words = (sh.V + 31) / 32;
        e = cudaMemsetAsync(ws.id_bitmap, 0, (size_t)n_words * 4, st);
        if (e != cudaSuccess) return (int)e;
        e = launch_chained(ids_mark_kernel, dim3((c.N + 255) / 256 < 1024 ? (c.N + 255) / 256 : 1024), dim3(256), 0, st, c.ids, c.N, sh.V,
                           ws.id_bitmap, ws.status);
        if (e == cudaSuccess) e = launch_chained(ids_compact_kernel, dim3(32), dim3(kCompactThreads), 0, st, ws.id_bitmap, n_words, ws.sorted_ids, c.N, c.ids, sh.V);
        *launches += 2;
        if (e != cudaSuccess) return (int)e;
        head_ids = ws.sorted_ids;
    }

    auto gemm = [&](GemmArgs &g, int rows, int n_rows, int Kdim, int lda, const bf16_t *x, int ldx) -> int {
        g.n_rows = n_rows; g.K = Kdim; g.lda = lda; g.x = x; g.ldx = ldx; g.NB = (2 * rows + 15) / 16 * 16; g.R = rows;
        g.status = ws.status;
        g.wait_limit_ns = c.wait_limit_ns;
        g.extra_arrivals = inject_left > 0 ? 1 : 0;      // self-test: the call's first GEMM waits for a copy that never comes
        if (inject_left > 0) --inject_left;
        const int n_tiles = (n_rows + kGemmTileM - 1) / kGemmTileM, n_kb = (Kdim + kGemmBK - 1) / kGemmBK;
        g.splits = g.epi == EPI_PARTIAL ? pick_splits(n_tiles, n_kb, c.n_sm) : 1;
        g.kb_per_split = (n_kb + g.splits - 1) / g.splits;
        g.splits = (n_kb + g.kb_per_split - 1) / g.kb_per_split;      // no empty range
        g.partial = ws.partial; g.ldp = ws.ldp;
        ++*launches;
        return skinny_gemm_launch(g, c.n_sm, c.smem_optin, st, c.cache);
    };
    int rc = 0;
    const size_t attn_smem = sh.dh == 128 ? AttnSmem<128>::TOTAL : AttnSmem<64>::TOTAL;
    if (c.cache->attn_smem < (int)attn_smem) {
        if (sh.dh == 128) e = cudaFuncSetAttribute(attn_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)attn_smem);
        else e = cudaFuncSetAttribute(attn_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)attn_smem);
        if (e != cudaSuccess) return (int)e;
        c.cache->attn_smem = (int)attn_smem;
    }
    int page_shift = -1;
    for (int b = 0; b < 31; ++b) if ((1 << b) == sh.page) page_shift = b;

    // One pass of the MTP module (projection, decoder layer, final norm) over `rows` activation rows of the sequences
    // seq0 .. seq0 + rows / geo.M - 1 of the group. The final norm publishes into `xop_head` (the output head's operand),
    // hout and out_h, under the row's own index or, in an extend pass, under its sequence's.
    auto mtp_pass = [&](int step, int rows, int seq0, const RowGeo &geo, bf16_t *xop_head, int map_out) -> int {
        KvPtrs kv = c.kv;
        kv.block_table += (size_t)seq0 * kv.max_pages;
        kv.seq_lens += seq0;
        auto post = [&](int splits, int residual, int final, const bf16_t *gain) -> int {
            PostArgs a{};
            a.d = d; a.splits = splits; a.rows = rows; a.ldp = ws.ldp; a.ld = ws.ld0; a.residual = residual; a.final = final;
            a.K = K; a.step = step; a.eps = sh.eps; a.partial = ws.partial; a.x = ws.x; a.hout = ws.hout;
            a.out_h = c.out_h; a.gain = gain; a.xop = final ? xop_head : ws.xop0;
            a.map_out = final ? map_out : 0; a.seq0 = seq0; a.geo = geo;
            ++*launches;
            return (int)launch_chained(post_kernel, dim3(rows), dim3(kRowThreads), 0, st, a);
        };
        PrologueArgs pa{};
        pa.step = step; pa.K = K; pa.d = d; pa.V = sh.V; pa.ld = ws.ld0; pa.only_tokens = 0; pa.geo = geo;
        pa.eps = sh.eps; pa.h_last = c.h_last + (size_t)seq0 * M0 * d; pa.tok_last = c.tok_last + (size_t)seq0 * M0; pa.hout = ws.hout;
        pa.keys_prev = step > 0 ? ws.keys + (size_t)(step - 1) * kBatchRows : nullptr;
        pa.out_drafts = c.out_drafts; pa.embed = c.embed; pa.g_h = c.g_hnorm; pa.g_e = c.g_enorm;
        pa.xop = ws.xop0; pa.status = ws.status; pa.user_status = c.user_status;
        ++*launches;
        int rc = 0;
        if ((rc = (int)launch_chained(prologue_kernel, dim3(rows), dim3(kRowThreads), 0, st, pa))) return rc;
        GemmArgs g{};
        // x = W_p [rms(h); rms(e)]
        g.a[0] = c.w_proj; g.a_rows[0] = d; g.n_seg = 1; g.epi = EPI_PARTIAL;
        if ((rc = gemm(g, rows, d, 2 * d, 2 * d, ws.xop0, ws.ld0))) return rc;
        if ((rc = post(g.splits, 0, 0, c.layer.g_in))) return rc;
        // q, k, v
        g = GemmArgs{};
        g.a[0] = c.layer.wq; g.a[1] = c.layer.wk; g.a[2] = c.layer.wv;
        g.a_rows[0] = qdim; g.a_rows[1] = kvdim; g.a_rows[2] = kvdim; g.n_seg = 3; g.epi = EPI_PARTIAL;
        if ((rc = gemm(g, rows, qdim + 2 * kvdim, d, d, ws.xop0, ws.ld0))) return rc;
        {
            QkvArgs a{};
            a.qdim = qdim; a.kvdim = kvdim; a.dh = sh.dh; a.Hq = sh.Hq; a.Hkv = sh.Hkv; a.splits = g.splits; a.rows = rows;
            a.ldp = ws.ldp; a.page = sh.page; a.max_ctx = sh.max_ctx; a.geo = geo; a.partial = ws.partial; a.q = ws.q;
            a.kv = kv; a.rope_cos = c.rope_cos; a.rope_sin = c.rope_sin; a.status = ws.status;
            ++*launches;
            if ((rc = (int)launch_chained(qkv_finish_kernel, dim3(sh.Hq + 2 * sh.Hkv, rows), dim3(sh.dh / 2), 0, st, a))) return rc;
        }
        {
            AttnArgs a{};
            a.Hq = sh.Hq; a.Hkv = sh.Hkv; a.dh = sh.dh; a.page = sh.page; a.max_ctx = sh.max_ctx; a.geo = geo;
            a.max_chunks = ws.max_chunks; a.q = ws.q; a.kv = kv; a.att_part = ws.att_part; a.status = ws.status;
            a.page_shift = page_shift; a.B = rows; a.wait_limit_ns = c.wait_limit_ns;
            ++*launches;
            if (sh.dh == 128) rc = (int)launch_chained(attn_kernel<128>, dim3(c.n_sm), dim3(2 * kAttnThreads), attn_smem, st, a);
            else rc = (int)launch_chained(attn_kernel<64>, dim3(c.n_sm), dim3(2 * kAttnThreads), attn_smem, st, a);
            if (rc) return rc;
            MergeArgs m{};
            m.Hq = sh.Hq; m.dh = sh.dh; m.page = sh.page; m.max_ctx = sh.max_ctx; m.geo = geo; m.max_chunks = ws.max_chunks;
            m.ld = ws.ld0; m.kv = kv; m.att_part = ws.att_part; m.xop = ws.xop0;
            ++*launches;
            if ((rc = (int)launch_chained(attn_merge_kernel, dim3(sh.Hq, rows), dim3(sh.dh), 0, st, m))) return rc;
        }
        // x += W_o o
        g = GemmArgs{};
        g.a[0] = c.layer.wo; g.a_rows[0] = d; g.n_seg = 1; g.epi = EPI_PARTIAL;
        if ((rc = gemm(g, rows, d, qdim, qdim, ws.xop0, ws.ld0))) return rc;
        if ((rc = post(g.splits, 1, 0, c.layer.g_post))) return rc;
        // act = silu(W_gate n) * (W_up n), written as the down projection's operand
        g = GemmArgs{};
        g.a[0] = c.layer.w_gate; g.a_up = c.layer.w_up; g.a_rows[0] = sh.F; g.n_seg = 1; g.epi = EPI_SWIGLU;
        g.xop_out = ws.xopF; g.ld_out = ws.ldF;
        if ((rc = gemm(g, rows, sh.F, d, d, ws.xop0, ws.ld0))) return rc;
        // x += W_down act; h_out = rms(x; g_final)
        g = GemmArgs{};
        g.a[0] = c.layer.w_down; g.a_rows[0] = d; g.n_seg = 1; g.epi = EPI_PARTIAL;
        if ((rc = gemm(g, rows, d, sh.F, sh.F, ws.xopF, ws.ldF))) return rc;
        return post(g.splits, 1, 1, c.g_final);
    };

    for (int step = 0; step < K; ++step) {
        const bf16_t *xop_head = ws.xop0;
        if (step == 0 && ext) {
            // extend rows: whole sequences in passes of up to 64 rows; each pass streams the module's weights once and
            // publishes its sequences' last rows into the head's operand, so the output head runs once for the group
            const int Gs = kBatchRows / M0;
            for (int s0 = 0; s0 < B; s0 += Gs) {
                const int Bs = B - s0 < Gs ? B - s0 : Gs;
                const RowGeo geo{M0, M0, 0, c.n_ext ? c.n_ext + s0 : nullptr};
                if ((rc = mtp_pass(0, Bs * M0, s0, geo, ws.xopH, 1))) return rc;
            }
            xop_head = ws.xopH;
        } else {
            const RowGeo geo{1, M0, step, c.n_ext};
            if ((rc = mtp_pass(step, B, 0, geo, ws.xop0, 0))) return rc;
        }
        // compressed head + argmax (Eq. 3)
        GemmArgs g{};
        g.a[0] = c.lm_head; g.a_rows[0] = c.N; g.n_seg = 1; g.epi = EPI_ARGMAX;
        g.row_ids = head_ids; g.V = sh.V;
        g.keys = ws.keys + (size_t)step * kBatchRows;
        g.logits = c.out_logits ? c.out_logits + (size_t)step * c.N : nullptr;
        g.logits_stride = (long long)K * c.N;
        if ((rc = gemm(g, B, c.N, d, d, xop_head, ws.ld0))) return rc;
    }
    // the last step's argmax keys -> draft tokens; status word -> caller
    PrologueArgs pa{};
    pa.step = K; pa.K = K; pa.d = d; pa.V = sh.V; pa.ld = ws.ld0; pa.only_tokens = 1; pa.geo = RowGeo{1, M0, K, c.n_ext};
    pa.eps = sh.eps; pa.keys_prev = ws.keys + (size_t)(K - 1) * kBatchRows;
    pa.out_drafts = c.out_drafts; pa.status = ws.status; pa.user_status = c.user_status;
    ++*launches;
    return (int)launch_chained(prologue_kernel, dim3(B), dim3(kRowThreads), 0, st, pa);
}

int batched_target(const BatchedTargetCall &c, cudaStream_t st, long long *launches) {
    const BatchedShape &sh = c.sh;
    const BatchedWs &ws = c.ws;
    const int R = c.B * c.M, d = sh.d;
    const int qdim = sh.Hq * sh.dh, kvdim = sh.Hkv * sh.dh;
    const int NB = (2 * R + 15) / 16 * 16;
    const RowGeo geo{c.M, c.M, 0, nullptr};       // M rows per sequence at positions L .. L+M-1, all of them real
    cudaError_t e = cudaMemsetAsync(ws.keys, 0, ws.keys_bytes, st);     // argmax keys and the status word
    if (e != cudaSuccess) return (int)e;
    auto gemm = [&](GemmArgs &g, int n_rows, int Kdim, int lda, const bf16_t *x, int ldx) -> int {
        g.n_rows = n_rows; g.K = Kdim; g.lda = lda; g.x = x; g.ldx = ldx; g.NB = NB; g.R = R;
        g.status = ws.status;
        g.wait_limit_ns = c.wait_limit_ns;
        const int n_tiles = (n_rows + kGemmTileM - 1) / kGemmTileM, n_kb = (Kdim + kGemmBK - 1) / kGemmBK;
        g.splits = g.epi == EPI_PARTIAL ? pick_splits(n_tiles, n_kb, c.n_sm) : 1;
        g.kb_per_split = (n_kb + g.splits - 1) / g.splits;
        g.splits = (n_kb + g.kb_per_split - 1) / g.kb_per_split;
        g.partial = ws.partial; g.ldp = ws.ldp;
        ++*launches;
        return skinny_gemm_launch(g, c.n_sm, c.smem_optin, st, c.cache);
    };
    auto post = [&](int splits, int final, const bf16_t *gain) -> int {
        PostArgs a{};
        a.d = d; a.splits = splits; a.rows = R; a.ldp = ws.ldp; a.ld = ws.ld0; a.residual = 1; a.final = final;
        a.K = 1; a.step = 0; a.eps = sh.eps; a.partial = ws.partial; a.x = ws.x; a.hout = ws.hout;
        a.out_h = c.out_h; a.gain = gain; a.xop = ws.xop0;
        ++*launches;
        return (int)launch_chained(post_kernel, dim3(R), dim3(kRowThreads), 0, st, a);
    };
    int rc = 0;
    const size_t attn_smem = sh.dh == 128 ? AttnSmem<128>::TOTAL : AttnSmem<64>::TOTAL;
    if (c.cache->attn_smem < (int)attn_smem) {
        if (sh.dh == 128) e = cudaFuncSetAttribute(attn_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)attn_smem);
        else e = cudaFuncSetAttribute(attn_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)attn_smem);
        if (e != cudaSuccess) return (int)e;
        c.cache->attn_smem = (int)attn_smem;
    }
    int page_shift = -1;
    for (int b = 0; b < 31; ++b) if ((1 << b) == sh.page) page_shift = b;

    // x = Emb(tokens); operand of the first layer = rms(x; g_in)
    ++*launches;
    if ((rc = (int)launch_chained(embed_kernel, dim3(R), dim3(kRowThreads), 0, st, c.tokens, c.embed, d, sh.V, ws.x, ws.status))) return rc;
    if ((rc = post(0, 0, c.layers[0].g_in))) return rc;
    for (int l = 0; l < c.n_layers; ++l) {
        const LayerPtrs &L = c.layers[l];
        const KvPtrs &kv = c.kvs[l];
        GemmArgs g{};
        g.a[0] = L.wq; g.a[1] = L.wk; g.a[2] = L.wv;
        g.a_rows[0] = qdim; g.a_rows[1] = kvdim; g.a_rows[2] = kvdim; g.n_seg = 3; g.epi = EPI_PARTIAL;
        if ((rc = gemm(g, qdim + 2 * kvdim, d, d, ws.xop0, ws.ld0))) return rc;
        {
            QkvArgs a{};
            a.qdim = qdim; a.kvdim = kvdim; a.dh = sh.dh; a.Hq = sh.Hq; a.Hkv = sh.Hkv; a.splits = g.splits; a.rows = R;
            a.ldp = ws.ldp; a.page = sh.page; a.max_ctx = sh.max_ctx; a.geo = geo; a.partial = ws.partial; a.q = ws.q;
            a.kv = kv; a.rope_cos = c.rope_cos; a.rope_sin = c.rope_sin; a.status = ws.status;
            ++*launches;
            if ((rc = (int)launch_chained(qkv_finish_kernel, dim3(sh.Hq + 2 * sh.Hkv, R), dim3(sh.dh / 2), 0, st, a))) return rc;
        }
        {
            AttnArgs a{};
            a.Hq = sh.Hq; a.Hkv = sh.Hkv; a.dh = sh.dh; a.page = sh.page; a.max_ctx = sh.max_ctx; a.geo = geo;
            a.max_chunks = ws.max_chunks; a.q = ws.q; a.kv = kv; a.att_part = ws.att_part; a.status = ws.status;
            a.page_shift = page_shift; a.B = R; a.wait_limit_ns = c.wait_limit_ns;
            ++*launches;
            if (sh.dh == 128) rc = (int)launch_chained(attn_kernel<128>, dim3(c.n_sm), dim3(2 * kAttnThreads), attn_smem, st, a);
            else rc = (int)launch_chained(attn_kernel<64>, dim3(c.n_sm), dim3(2 * kAttnThreads), attn_smem, st, a);
            if (rc) return rc;
            MergeArgs m{};
            m.Hq = sh.Hq; m.dh = sh.dh; m.page = sh.page; m.max_ctx = sh.max_ctx; m.geo = geo; m.max_chunks = ws.max_chunks;
            m.ld = ws.ld0; m.kv = kv; m.att_part = ws.att_part; m.xop = ws.xop0;
            ++*launches;
            if ((rc = (int)launch_chained(attn_merge_kernel, dim3(sh.Hq, R), dim3(sh.dh), 0, st, m))) return rc;
        }
        g = GemmArgs{};
        g.a[0] = L.wo; g.a_rows[0] = d; g.n_seg = 1; g.epi = EPI_PARTIAL;
        if ((rc = gemm(g, d, qdim, qdim, ws.xop0, ws.ld0))) return rc;
        if ((rc = post(g.splits, 0, L.g_post))) return rc;
        g = GemmArgs{};
        g.a[0] = L.w_gate; g.a_up = L.w_up; g.a_rows[0] = sh.F; g.n_seg = 1; g.epi = EPI_SWIGLU;
        g.xop_out = ws.xopF; g.ld_out = ws.ldF;
        if ((rc = gemm(g, sh.F, d, d, ws.xop0, ws.ld0))) return rc;
        g = GemmArgs{};
        g.a[0] = L.w_down; g.a_rows[0] = d; g.n_seg = 1; g.epi = EPI_PARTIAL;
        if ((rc = gemm(g, d, sh.F, sh.F, ws.xopF, ws.ldF))) return rc;
        const bool last = l + 1 == c.n_layers;
        if ((rc = post(g.splits, last ? 1 : 0, last ? c.g_final : c.layers[l + 1].g_in))) return rc;
    }
    if (c.out_logits || c.out_argmax) {
        // full output head; the greedy choice is made on the bf16-rounded logits a caller would see
        GemmArgs g{};
        g.a[0] = c.lm_head; g.a_rows[0] = sh.V; g.n_seg = 1; g.epi = EPI_ARGMAX; g.V = sh.V;
        g.keys = c.out_argmax ? ws.keys : nullptr;
        g.round_bf16 = 1; g.logits_bf16 = c.out_logits; g.logits_stride = sh.V;
        if ((rc = gemm(g, sh.V, d, d, ws.xop0, ws.ld0))) return rc;
    }
    // argmax keys -> token ids (if asked for), status word -> caller
    PrologueArgs pa{};
    pa.step = 1; pa.K = 1; pa.d = d; pa.V = sh.V; pa.ld = ws.ld0; pa.only_tokens = 1; pa.eps = sh.eps;
    pa.geo = geo;
    pa.keys_prev = ws.keys; pa.out_drafts = c.out_argmax; pa.status = ws.status; pa.user_status = c.user_status;
    ++*launches;
    return (int)launch_chained(prologue_kernel, dim3(R), dim3(kRowThreads), 0, st, pa);
}

}  // namespace fmtp
