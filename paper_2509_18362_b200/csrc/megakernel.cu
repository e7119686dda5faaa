// Persistent decoder kernel: one cooperative launch runs every phase of K recursive MTP draft
// steps (or of one target-decoder step) with grid barriers in between, so a draft call never
// returns to the host between steps.
//
// Structure of a CTA (one per SM): 8 consumer warps + 1 producer warp.
//   * The producer streams bf16 weight rows from HBM into a ring of shared-memory stages with
//     1-D bulk async copies (TMA engine) that complete on mbarriers. Weight addresses do not
//     depend on activations, so the producer runs ahead of the grid barriers: while the
//     consumers wait for the previous phase's vector, HBM keeps streaming the next phase's rows.
//   * A matrix-vector phase gives every CTA a contiguous range of output rows. A stage holds up
//     to 32 rows x KC columns; the 8 consumer warps each take a fixed k-slice of the stage and
//     multiply with mma.sync m16n8k16 (weights = A operand, activation rows = B operand columns),
//     then reduce across warps in a fixed order. The activation vector is fp32 carried as two
//     bf16 numbers (hi + lo), so products are exact and the sum is fp32-accurate; each of the up
//     to 8 activation rows occupies its own MMA column, so a row's result does not depend on how
//     many other rows the call carries.
//   * RMSNorm is folded: the producing phase stores x*g (split hi/lo) plus per-CTA partial sums of
//     x^2; the consuming phase multiplies its accumulators by rsqrt(mean(x^2)+eps).
//   * Attention splits the context into fixed 128-token chunks (work items over sequence x KV head
//     x chunk), fp32 online softmax, and the CTA that finishes a (sequence, KV head) group last
//     merges its chunks in a fixed order -- no float atomics anywhere, results are reproducible.
//   * The output head gathers rows W[ids[j]] (Eq. 3 of the paper), keeps a running (value, id)
//     maximum per activation row and publishes it with one 64-bit atomicMax per CTA; logits are
//     never written unless a debug buffer is passed.
#include "mega.cuh"
#include "ptx.cuh"

#include <cooperative_groups.h>

namespace fmtp {

namespace {

constexpr uint32_t kDevBadToken = 0x1u, kDevBadPage = 0x2u, kDevBadPos = 0x4u, kDevTimeout = 0x8u,
                   kDevAllNan = 0x10u;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // a wait gives up after 2 s

enum Kind { PROJ = 0, QKV = 1, OPROJ = 2, GATEUP = 3, DOWN = 4, HEAD = 5 };

struct Misc {   // small shared-memory block
    uint64_t full[kMaxStages];
    uint64_t empty[kMaxStages];
    float scale0[kMaxRows];
    float scale1[kMaxRows];
    float ssred[kConsumerWarps][kMaxRows][2];
    float colred[kTileRows][kMaxRows];
    unsigned long long keyred[kConsumerWarps][kMaxRows];
    int tok[kMaxRows];
    int flag;
    uint32_t aborted;
};

struct Cta {
    const MegaParams *p;
    Misc *misc;
    float *red;            // [2][8 warps][32 rows][R]
    unsigned char *scr;    // per-phase scratch (activation staging / attention)
    unsigned char *ring;
    int cta, grid, tid, warp, lane;
    uint32_t stage;        // running stage counter (same sequence in producer and consumers)
    uint32_t bar_target;   // grid barrier generation
    int redbuf;
};

__device__ __forceinline__ void raise(const Cta &c, uint32_t bits) { atomicOr(c.p->s.status, bits); }

__device__ __forceinline__ bool aborted(const Cta &c) { return *((volatile uint32_t *)&c.misc->aborted) != 0; }

__device__ void do_abort(const Cta &c) {
    c.misc->aborted = 1;
    atomicOr(c.p->s.status, kDevTimeout);
    atomicExch(c.p->s.abort_flag, 1u);
}

// Bounded wait on an mbarrier phase. Returns false (and raises the abort flag) on timeout.
__device__ bool wait_bar(const Cta &c, uint64_t *bar, uint32_t parity) {
    if (aborted(c)) return false;
    unsigned long long t0 = 0;
    for (uint32_t n = 0;; ++n) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((n & 255u) == 255u) {
            if (ldcg_u32(c.p->s.abort_flag) != 0) {
                c.misc->aborted = 1;
                return false;
            }
            unsigned long long now = global_timer_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > kWaitLimitNs) break;
        }
    }
    do_abort(c);
    return false;
}

// Grid-wide barrier among the consumer threads of all CTAs (the producer warp never joins).
__device__ void grid_barrier(Cta &c) {
    bar_sync(1, kConsumerThreads);
    c.bar_target += (uint32_t)c.grid;
    if (c.tid == 0) {
        __threadfence();
        atomicAdd(c.p->s.barrier, 1u);
        if (!aborted(c)) {
            uint32_t n = 0;
            unsigned long long t0 = 0;
            while ((int32_t)(ld_acquire_u32(c.p->s.barrier) - c.bar_target) < 0) {
                if ((++n & 255u) == 255u) {
                    if (ldcg_u32(c.p->s.abort_flag) != 0) { c.misc->aborted = 1; break; }
                    unsigned long long now = global_timer_ns();
                    if (t0 == 0) t0 = now;
                    else if (now - t0 > kWaitLimitNs) { do_abort(c); break; }
                }
                __nanosleep(32);
            }
        }
        __threadfence();
    }
    bar_sync(1, kConsumerThreads);
}

// ---- phase geometry ----------------------------------------------------------------------
struct Geom { int rows, K, cap, nks, v0, v1; };

__device__ __forceinline__ Geom geom(const Cta &c, int kind) {
    const MegaParams &p = *c.p;
    Geom g;
    switch (kind) {
        case PROJ:   g.rows = p.d;                    g.K = 2 * p.d; break;
        case QKV:    g.rows = p.qdim + 2 * p.kvdim;   g.K = p.d;     break;
        case OPROJ:  g.rows = p.d;                    g.K = p.qdim;  break;
        case GATEUP: g.rows = p.F;                    g.K = p.d;     break;
        case DOWN:   g.rows = p.d;                    g.K = p.F;     break;
        default:     g.rows = p.N;                    g.K = p.d;     break;
    }
    g.cap = (kind == GATEUP) ? kTileRows / 2 : kTileRows;
    g.nks = (g.K + p.KC - 1) / p.KC;
    g.v0 = (int)(((long long)c.cta * g.rows) / c.grid);
    g.v1 = (int)(((long long)(c.cta + 1) * g.rows) / c.grid);
    return g;
}

// Address of weight row `j` (0..31) of the tile whose first virtual row is vr0; nullptr if the
// tile row is unused.
__device__ __forceinline__ const bf16_t *tile_row_ptr(const Cta &c, int kind, const LayerPtrs &L, int vr0, int nv,
                                                      int j) {
    const MegaParams &p = *c.p;
    if (kind == GATEUP) {
        int jj = j & 15;
        if (jj >= nv) return nullptr;
        const bf16_t *base = (j < 16) ? L.w_gate : L.w_up;
        return base + (size_t)(vr0 + jj) * p.d;
    }
    if (j >= nv) return nullptr;
    int r = vr0 + j;
    switch (kind) {
        case PROJ: return p.w_proj + (size_t)r * (2 * p.d);
        case QKV:
            if (r < p.qdim) return L.wq + (size_t)r * p.d;
            if (r < p.qdim + p.kvdim) return L.wk + (size_t)(r - p.qdim) * p.d;
            return L.wv + (size_t)(r - p.qdim - p.kvdim) * p.d;
        case OPROJ: return L.wo + (size_t)r * p.qdim;
        case DOWN: return L.w_down + (size_t)r * p.F;
        default: {
            int id = p.ids ? p.ids[r] : r;
            if ((unsigned)id >= (unsigned)p.V) { raise(c, kDevBadToken); id = 0; }
            return p.lm_head + (size_t)id * p.d;
        }
    }
}

// ---- producer ------------------------------------------------------------------------------
__device__ void produce_phase(Cta &c, int kind, const LayerPtrs &L) {
    const MegaParams &p = *c.p;
    Geom g = geom(c, kind);
    for (int vr0 = g.v0; vr0 < g.v1; vr0 += g.cap) {
        int nv = min(g.cap, g.v1 - vr0);
        const bf16_t *src = tile_row_ptr(c, kind, L, vr0, nv, c.lane);
        int nrows = (kind == GATEUP) ? 2 * nv : nv;
        for (int ks = 0; ks < g.nks; ++ks) {
            int slot = c.stage % p.n_stages;
            uint32_t parity = (c.stage / p.n_stages) & 1u;
            bool ok = true;
            if (c.lane == 0) ok = wait_bar(c, &c.misc->empty[slot], parity ^ 1u);
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) return;   // abort: stop issuing copies
            int klen = min(p.KC, g.K - ks * p.KC);
            uint32_t bytes = (uint32_t)klen * 2u;
            if (c.lane == 0) mbar_arrive_expect_tx(&c.misc->full[slot], bytes * (uint32_t)nrows);
            __syncwarp();
            if (src)
                bulk_g2s(c.ring + (size_t)slot * p.stage_bytes + (size_t)c.lane * p.row_stride,
                         src + (size_t)ks * p.KC, bytes, &c.misc->full[slot]);
            c.stage++;
        }
    }
}

// ---- consumer: matrix-vector core --------------------------------------------------------------
struct ActSrc {          // where the B operand (activations) is read from
    const bf16_t *hi, *lo;   // shared-memory staging area, or global scratch written by other CTAs
    int stride;              // elements per activation row
    bool in_smem;
};

template <int KIND>
struct Epi;   // epilogue functors, specialised below

// Runs all tiles of one phase for this CTA. `epi(vrow, col, v0, v1)` is called once per valid
// (virtual row, activation row) by exactly one thread; v1 is the paired "up" value for GATEUP.
template <int KIND, typename EpiF>
__device__ void consume_phase(Cta &c, const ActSrc &act, int seg_stage, EpiF &&epi) {
    const MegaParams &p = *c.p;
    Geom geo = geom(c, KIND);
    const int R = p.R;
    const int g = c.lane >> 2, t = c.lane & 3;
    const int nchunk_full = p.KC / 32;
    for (int vr0 = geo.v0; vr0 < geo.v1; vr0 += geo.cap) {
        int nv = min(geo.cap, geo.v1 - vr0);
        float acc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
        float acc0[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
        for (int ks = 0; ks < geo.nks; ++ks) {
            int slot = c.stage % p.n_stages;
            uint32_t parity = (c.stage / p.n_stages) & 1u;
            wait_bar(c, &c.misc->full[slot], parity);
            int klen = min(p.KC, geo.K - ks * p.KC);
            int nchunk = (klen == p.KC) ? nchunk_full : (klen + 31) / 32;
            const unsigned char *st = c.ring + (size_t)slot * p.stage_bytes;
            for (int ch = c.warp; ch < nchunk; ch += kConsumerWarps) {
                const unsigned char *a = st + ch * 64 + t * 16;
                uint4 u0 = lds128(a + (size_t)g * p.row_stride);
                uint4 v0 = lds128(a + (size_t)(g + 8) * p.row_stride);
                uint4 u1 = lds128(a + (size_t)(g + 16) * p.row_stride);
                uint4 v1 = lds128(a + (size_t)(g + 24) * p.row_stride);
                uint4 bh = make_uint4(0, 0, 0, 0), bl = make_uint4(0, 0, 0, 0);
                if (g < R) {
                    size_t off = (size_t)g * act.stride + (size_t)ks * p.KC + ch * 32 + t * 8;
                    if (act.in_smem) {
                        bh = lds128(act.hi + off);
                        bl = lds128(act.lo + off);
                    } else {   // produced by other CTAs in the previous phase: read through L2
                        bh = ldcg128(act.hi + off);
                        bl = ldcg128(act.lo + off);
                    }
                }
                mma_bf16(acc[0], u0.x, v0.x, u0.y, v0.y, bh.x, bh.y);
                mma_bf16(acc[1], u1.x, v1.x, u1.y, v1.y, bh.x, bh.y);
                mma_bf16(acc[0], u0.z, v0.z, u0.w, v0.w, bh.z, bh.w);
                mma_bf16(acc[1], u1.z, v1.z, u1.w, v1.w, bh.z, bh.w);
                mma_bf16(acc[0], u0.x, v0.x, u0.y, v0.y, bl.x, bl.y);
                mma_bf16(acc[1], u1.x, v1.x, u1.y, v1.y, bl.x, bl.y);
                mma_bf16(acc[0], u0.z, v0.z, u0.w, v0.w, bl.z, bl.w);
                mma_bf16(acc[1], u1.z, v1.z, u1.w, v1.w, bl.z, bl.w);
            }
            __syncwarp();
            if (c.lane == 0) mbar_arrive(&c.misc->empty[slot]);
            c.stage++;
            if (KIND == PROJ && ks + 1 == seg_stage) {
#pragma unroll
                for (int i = 0; i < 2; ++i)
#pragma unroll
                    for (int j = 0; j < 4; ++j) { acc0[i][j] = acc[i][j]; acc[i][j] = 0.f; }
            }
        }
        // cross-warp reduction in a fixed order
        float *red = c.red + (size_t)c.redbuf * kConsumerWarps * kTileRows * R + (size_t)c.warp * kTileRows * R;
#pragma unroll
        for (int i = 0; i < 2; ++i) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                int row = i * 16 + g + ((j >> 1) << 3);
                int col = 2 * t + (j & 1);
                if (col < R) {
                    float v = acc[i][j];
                    if (KIND == PROJ) v = acc0[i][j] * c.misc->scale0[col] + v * c.misc->scale1[col];
                    red[row * R + col] = v;
                }
            }
        }
        bar_sync(1, kConsumerThreads);
        {
            const float *rb = c.red + (size_t)c.redbuf * kConsumerWarps * kTileRows * R;
            int row = c.tid >> 3, col = c.tid & 7;
            if (KIND == GATEUP) {
                if (row < 16 && row < nv && col < R) {
                    float a = 0.f, b = 0.f;
#pragma unroll
                    for (int w = 0; w < kConsumerWarps; ++w) {
                        a += rb[(size_t)w * kTileRows * R + row * R + col];
                        b += rb[(size_t)w * kTileRows * R + (row + 16) * R + col];
                    }
                    epi(vr0 + row, col, a, b);
                }
            } else if (row < nv && col < R) {
                float a = 0.f;
#pragma unroll
                for (int w = 0; w < kConsumerWarps; ++w) a += rb[(size_t)w * kTileRows * R + row * R + col];
                epi(vr0 + row, col, a, 0.f);
            }
        }
        c.redbuf ^= 1;
    }
}

// Sum over CTAs of a per-CTA partial-sums-of-squares table [grid][8], for activation row `col`.
// Called by one full warp; fixed reduction tree => reproducible.
__device__ float sum_partials(const Cta &c, const float *tbl, int col) {
    float s = 0.f;
    for (int i = c.lane; i < c.grid; i += 32) s += ldcg_f32(tbl + (size_t)i * kMaxRows + col);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    return s;
}

// Copies R rows of a hi/lo activation pair from global scratch into the shared staging area.
// `len` elements per row (multiple of 8), rows `stride_s` apart in shared memory, starting at
// element offset `dst_off`.
__device__ void stage_hilo(const Cta &c, const bf16_t *ghi, const bf16_t *glo, int gstride, int len, bf16_t *shi,
                           bf16_t *slo, int sstride, int dst_off) {
    int per_row = len / 8;
    int total = c.p->R * per_row;
    for (int i = c.tid; i < total; i += kConsumerThreads) {
        int r = i / per_row, k = (i - r * per_row) * 8;
        uint4 a = ldcg128(ghi + (size_t)r * gstride + k);
        uint4 b = ldcg128(glo + (size_t)r * gstride + k);
        *reinterpret_cast<uint4 *>(shi + (size_t)r * sstride + dst_off + k) = a;
        *reinterpret_cast<uint4 *>(slo + (size_t)r * sstride + dst_off + k) = b;
    }
}

// Block-wide sum of up to 2 values per activation row, all consumer threads participate.
// Result for (col, which) is left in misc->ssred[0][col][which].
__device__ void block_sum2(const Cta &c, float (&v)[kMaxRows][2], int R) {
    for (int r = 0; r < R; ++r)
#pragma unroll
        for (int w = 0; w < 2; ++w) {
            float s = v[r][w];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
            if (c.lane == 0) c.misc->ssred[c.warp][r][w] = s;
        }
    bar_sync(1, kConsumerThreads);
    if (c.tid < R * 2) {
        int r = c.tid >> 1, w = c.tid & 1;
        float s = 0.f;
        for (int i = 0; i < kConsumerWarps; ++i) s += c.misc->ssred[i][r][w];
        c.misc->ssred[0][r][w] = s;
    }
    bar_sync(1, kConsumerThreads);
}

// Per-thread accumulation of v^2 per activation row across the tiles of a phase, reduced over
// the CTA's rows at phase end and written to this CTA's line of a partial table.
struct SqAcc {
    float a, b;
    __device__ SqAcc() : a(0.f), b(0.f) {}
};
__device__ void flush_sq(const Cta &c, const SqAcc &q, float *tblA, float *tblB) {
    // thread (row = tid>>3, col = tid&7)
    int row = c.tid >> 3, col = c.tid & 7;
    for (int which = 0; which < 2; ++which) {
        float *tbl = which ? tblB : tblA;
        if (!tbl) continue;
        bar_sync(1, kConsumerThreads);
        c.misc->colred[row][col] = which ? q.b : q.a;
        bar_sync(1, kConsumerThreads);
        if (c.tid < kMaxRows) {
            float s = 0.f;
            for (int i = 0; i < kTileRows; ++i) s += c.misc->colred[i][c.tid];
            tbl[(size_t)c.cta * kMaxRows + c.tid] = s;
        }
    }
}

__device__ __forceinline__ void store_split(bf16_t *hi, bf16_t *lo, size_t idx, float v) {
    uint16_t h, l;
    split_bf16(v, h, l);
    hi[idx] = h;
    lo[idx] = l;
}

// ---- attention phase -------------------------------------------------------------------------
// Rows r = b*M + m sit at position seq_lens[b] + posoff + m. Scratch layout (floats):
//   qs[M*Gq][dh]  rotated, pre-scaled queries of one KV head
//   kn[M][dh], vn[M][dh]  this call's new keys / values (after bf16 rounding)
//   wp[8 warps][Gq][dh + 2] per-warp partial (o, m, l) for the row being processed
__device__ void attention_phase(Cta &c, const KvPtrs &kv, int posoff) {
    const MegaParams &p = *c.p;
    const int dh = p.dh, half = dh >> 1, Gq = p.Hq / p.Hkv, M = p.M;
    const int epl = dh >> 5;   // elements per lane (2 or 4)
    float *qs = reinterpret_cast<float *>(c.scr);
    float *kn = qs + (size_t)M * Gq * dh;
    float *vn = kn + (size_t)M * dh;
    float *wp = vn + (size_t)M * dh;
    const int wstride = dh + 2;
    const float qscale = rsqrtf((float)dh);
    const int max_tokens = min(kv.max_pages * p.page, p.max_ctx);   // positions beyond are flagged, not touched

    // work list: per sequence Hkv * nch items
    int total = 0;
    for (int b = 0; b < p.B; ++b) {
        int last = kv.seq_lens[b] + posoff + M - 1;
        total += p.Hkv * (last / kAttnChunk + 1);
    }
    for (int item = c.cta; item < total; item += c.grid) {
        int b = 0, rem = item, Lb = 0, nch = 1;
        for (; b < p.B; ++b) {
            Lb = kv.seq_lens[b];
            nch = (Lb + posoff + M - 1) / kAttnChunk + 1;
            if (rem < p.Hkv * nch) break;
            rem -= p.Hkv * nch;
        }
        const int kvh = rem / nch, chunk = rem - kvh * nch;
        const int base = Lb + posoff;              // position of row m = 0
        const int32_t *bt = kv.block_table + (size_t)b * kv.max_pages;

        // -- stage rotated queries and the new K/V of this KV head
        for (int i = c.tid; i < M * Gq * half; i += kConsumerThreads) {
            int qi = i / half, e = i - qi * half;
            int m = qi / Gq, hq = kvh * Gq + (qi - m * Gq);
            int r = b * M + m, pos = base + m;
            if (pos >= max_tokens) pos = max_tokens - 1;
            const float *q = p.s.qkv + (size_t)r * (p.qdim + 2 * p.kvdim) + hq * dh;
            float x = ldcg_f32(q + e), y = ldcg_f32(q + e + half);
            float cs = p.s.rope_cos[(size_t)pos * half + e], sn = p.s.rope_sin[(size_t)pos * half + e];
            qs[qi * dh + e] = (x * cs - y * sn) * qscale;
            qs[qi * dh + e + half] = (y * cs + x * sn) * qscale;
        }
        for (int i = c.tid; i < M * half; i += kConsumerThreads) {
            int m = i / half, e = i - m * half;
            int r = b * M + m, pos = base + m;
            bool pos_ok = pos < max_tokens;
            if (!pos_ok) { raise(c, kDevBadPos); pos = max_tokens - 1; }
            const float *kk = p.s.qkv + (size_t)r * (p.qdim + 2 * p.kvdim) + p.qdim + kvh * dh;
            const float *vv = kk + p.kvdim;
            float x = ldcg_f32(kk + e), y = ldcg_f32(kk + e + half);
            float cs = p.s.rope_cos[(size_t)pos * half + e], sn = p.s.rope_sin[(size_t)pos * half + e];
            uint16_t k0 = f32_bf16bits(x * cs - y * sn), k1 = f32_bf16bits(y * cs + x * sn);
            uint16_t v0 = f32_bf16bits(ldcg_f32(vv + e)), v1 = f32_bf16bits(ldcg_f32(vv + e + half));
            kn[m * dh + e] = bf16bits_f32(k0);
            kn[m * dh + e + half] = bf16bits_f32(k1);
            vn[m * dh + e] = bf16bits_f32(v0);
            vn[m * dh + e + half] = bf16bits_f32(v1);
            if (pos_ok && pos / kAttnChunk == chunk) {   // the item that owns this position appends it
                int page = bt[pos / p.page];
                if ((unsigned)page >= (unsigned)kv.num_pages) { raise(c, kDevBadPage); page = 0; }
                size_t o = (((size_t)page * p.Hkv + kvh) * p.page + (pos % p.page)) * dh;
                kv.k_pages[o + e] = k0;
                kv.k_pages[o + e + half] = k1;
                kv.v_pages[o + e] = v0;
                kv.v_pages[o + e + half] = v1;
            }
        }
        bar_sync(1, kConsumerThreads);

        const int j0 = chunk * kAttnChunk + c.warp * 16;     // this warp's 16 tokens
        const int e0 = c.lane * epl;
        for (int m = 0; m < M; ++m) {
            const int npos = min(base + m, max_tokens - 1);  // last visible position of this row
            float q[8][4];
#pragma unroll
            for (int h = 0; h < 8; ++h)
#pragma unroll
                for (int e = 0; e < 4; ++e) q[h][e] = (h < Gq && e < epl) ? qs[(m * Gq + h) * dh + e0 + e] : 0.f;
            float sc[8];
#pragma unroll
            for (int h = 0; h < 8; ++h) sc[h] = -INFINITY;
            // pass 1: scores; lane `tk` keeps the score of token j0 + tk
            for (int tk = 0; tk < 16; ++tk) {
                int j = j0 + tk;
                if (j > npos) break;
                float kf[4] = {0.f, 0.f, 0.f, 0.f};
                if (j >= base) {
#pragma unroll
                    for (int e = 0; e < 4; ++e) if (e < epl) kf[e] = kn[(j - base) * dh + e0 + e];
                } else {
                    int page = bt[j / p.page];
                    if ((unsigned)page >= (unsigned)kv.num_pages) { raise(c, kDevBadPage); page = 0; }
                    const bf16_t *kr = kv.k_pages + (((size_t)page * p.Hkv + kvh) * p.page + (j % p.page)) * dh + e0;
                    if (epl == 4) {
                        uint2 w = ldcg64(kr);
                        kf[0] = bf16lo_f32(w.x); kf[1] = bf16hi_f32(w.x); kf[2] = bf16lo_f32(w.y); kf[3] = bf16hi_f32(w.y);
                    } else {
                        uint32_t w = ldcg_u32(kr);
                        kf[0] = bf16lo_f32(w); kf[1] = bf16hi_f32(w);
                    }
                }
#pragma unroll
                for (int h = 0; h < 8; ++h) {
                    if (h < Gq) {
                        float s = q[h][0] * kf[0] + q[h][1] * kf[1];
                        s += q[h][2] * kf[2] + q[h][3] * kf[3];
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
                        if (c.lane == tk) sc[h] = s;
                    }
                }
            }
            // softmax statistics over the warp's tokens
            float mw[8], lw[8], pj[8];
#pragma unroll
            for (int h = 0; h < 8; ++h) {
                float mx = sc[h];
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
                mw[h] = mx;
                pj[h] = (sc[h] == -INFINITY) ? 0.f : expf(sc[h] - mx);
                float sm = pj[h];
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) sm += __shfl_xor_sync(0xffffffffu, sm, o);
                lw[h] = sm;
            }
            // pass 2: o[h][e] = sum_j p_j V[j][e]
            float o[8][4];
#pragma unroll
            for (int h = 0; h < 8; ++h)
#pragma unroll
                for (int e = 0; e < 4; ++e) o[h][e] = 0.f;
            for (int tk = 0; tk < 16; ++tk) {
                int j = j0 + tk;
                if (j > npos) break;
                float vf[4] = {0.f, 0.f, 0.f, 0.f};
                if (j >= base) {
#pragma unroll
                    for (int e = 0; e < 4; ++e) if (e < epl) vf[e] = vn[(j - base) * dh + e0 + e];
                } else {
                    int page = bt[j / p.page];
                    if ((unsigned)page >= (unsigned)kv.num_pages) page = 0;
                    const bf16_t *vr = kv.v_pages + (((size_t)page * p.Hkv + kvh) * p.page + (j % p.page)) * dh + e0;
                    if (epl == 4) {
                        uint2 w = ldcg64(vr);
                        vf[0] = bf16lo_f32(w.x); vf[1] = bf16hi_f32(w.x); vf[2] = bf16lo_f32(w.y); vf[3] = bf16hi_f32(w.y);
                    } else {
                        uint32_t w = ldcg_u32(vr);
                        vf[0] = bf16lo_f32(w); vf[1] = bf16hi_f32(w);
                    }
                }
#pragma unroll
                for (int h = 0; h < 8; ++h) {
                    if (h < Gq) {
                        float pr = __shfl_sync(0xffffffffu, pj[h], tk);
#pragma unroll
                        for (int e = 0; e < 4; ++e) o[h][e] += pr * vf[e];
                    }
                }
            }
            // per-warp partial -> shared
#pragma unroll
            for (int h = 0; h < 8; ++h) {
                if (h < Gq) {
                    float *w = wp + ((size_t)c.warp * Gq + h) * wstride;
#pragma unroll
                    for (int e = 0; e < 4; ++e) if (e < epl) w[e0 + e] = o[h][e];
                    if (c.lane == 0) { w[dh] = mw[h]; w[dh + 1] = lw[h]; }
                }
            }
            bar_sync(1, kConsumerThreads);
            // merge the 8 warps (fixed order) -> chunk partial in global memory
            for (int i = c.tid; i < Gq * dh; i += kConsumerThreads) {
                int h = i / dh, e = i - h * dh;
                float mx = -INFINITY;
                for (int w = 0; w < kConsumerWarps; ++w) mx = fmaxf(mx, wp[((size_t)w * Gq + h) * wstride + dh]);
                float ov = 0.f, l = 0.f;
                for (int w = 0; w < kConsumerWarps; ++w) {
                    const float *pw = wp + ((size_t)w * Gq + h) * wstride;
                    float f = (pw[dh] == -INFINITY) ? 0.f : expf(pw[dh] - mx);
                    ov += f * pw[e];
                    l += f * pw[dh + 1];
                }
                int r = b * M + m, hq = kvh * Gq + h;
                float *dst = p.s.att_part + (((size_t)r * p.Hq + hq) * p.max_chunks + chunk) * wstride;
                dst[e] = ov;
                if (e == 0) { dst[dh] = mx; dst[dh + 1] = l; }
            }
            bar_sync(1, kConsumerThreads);
        }
        // -- last CTA of this (sequence, KV head) merges the chunks
        __threadfence();
        bar_sync(1, kConsumerThreads);
        if (c.tid == 0) {
            uint32_t old = atomicAdd(p.s.att_cnt + b * p.Hkv + kvh, 1u);
            c.misc->flag = (old == (uint32_t)(nch - 1));
        }
        bar_sync(1, kConsumerThreads);
        if (c.misc->flag) {
            __threadfence();
            for (int i = c.tid; i < M * Gq * dh; i += kConsumerThreads) {
                int mh = i / dh, e = i - mh * dh;
                int m = mh / Gq, h = mh - m * Gq;
                int r = b * M + m, hq = kvh * Gq + h;
                const float *src = p.s.att_part + ((size_t)r * p.Hq + hq) * p.max_chunks * wstride;
                int ncm = min(base + m, max_tokens - 1) / kAttnChunk + 1;   // chunks visible to this row
                float mx = -INFINITY;
                for (int ch = 0; ch < ncm; ++ch) mx = fmaxf(mx, ldcg_f32(src + (size_t)ch * wstride + dh));
                float ov = 0.f, l = 0.f;
                for (int ch = 0; ch < ncm; ++ch) {
                    float mc = ldcg_f32(src + (size_t)ch * wstride + dh);
                    float f = (mc == -INFINITY) ? 0.f : expf(mc - mx);
                    ov += f * ldcg_f32(src + (size_t)ch * wstride + e);
                    l += f * ldcg_f32(src + (size_t)ch * wstride + dh + 1);
                }
                store_split(p.s.actO_hi, p.s.actO_lo, (size_t)r * p.qp + hq * dh + e, ov / l);
            }
            if (c.tid == 0) p.s.att_cnt[b * p.Hkv + kvh] = 0;
        }
        bar_sync(1, kConsumerThreads);
    }
}

// ---- the kernel --------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads, 1) mega_kernel(const __grid_constant__ MegaParams p) {
    extern __shared__ __align__(128) unsigned char smem[];
    Cta c;
    c.p = &p;
    c.misc = reinterpret_cast<Misc *>(smem);
    size_t off = (sizeof(Misc) + 127) & ~size_t(127);
    c.red = reinterpret_cast<float *>(smem + off);
    off += ((size_t)2 * kConsumerWarps * kTileRows * p.R * sizeof(float) + 127) & ~size_t(127);
    c.scr = smem + off;
    off += (size_t)p.scratch_smem;
    c.ring = smem + off;
    c.cta = blockIdx.x;
    c.grid = gridDim.x;
    c.tid = threadIdx.x;
    c.warp = threadIdx.x >> 5;
    c.lane = threadIdx.x & 31;
    c.stage = 0;
    c.bar_target = 0;
    c.redbuf = 0;

    if (c.tid == 0) {
        for (int i = 0; i < p.n_stages; ++i) {
            mbar_init(&c.misc->full[i], 1);
            mbar_init(&c.misc->empty[i], kConsumerWarps);
        }
        c.misc->aborted = 0;
        mbar_fence_init();
    }
    // the ring starts zeroed so that never-written tails multiply as finite numbers
    for (size_t i = (size_t)c.tid * 16; i < (size_t)p.n_stages * p.stage_bytes; i += (size_t)kThreads * 16)
        *reinterpret_cast<uint4 *>(c.ring + i) = make_uint4(0, 0, 0, 0);
    fence_proxy_async();
    __syncthreads();

    const bool is_producer = (c.warp == kConsumerWarps);
    const int R = p.R;
    const int n_steps = (p.mode == 0) ? p.K : 1;
    const int n_layers = (p.mode == 0) ? 1 : p.n_layers;

    if (is_producer) {
        // ---------------- producer: the weight stream of every phase, in program order
        for (int step = 0; step < n_steps; ++step) {
            if (p.mode == 0) produce_phase(c, PROJ, p.layers[0]);
            for (int l = 0; l < n_layers; ++l) {
                produce_phase(c, QKV, p.layers[l]);
                produce_phase(c, OPROJ, p.layers[l]);
                produce_phase(c, GATEUP, p.layers[l]);
                produce_phase(c, DOWN, p.layers[l]);
            }
            produce_phase(c, HEAD, p.layers[0]);
        }
        // drain: every copy this warp issued must have landed before the CTA may exit
        if (c.lane == 0) {
            uint32_t issued = c.stage;
            uint32_t first = issued > (uint32_t)p.n_stages ? issued - p.n_stages : 0;
            for (uint32_t s = first; s < issued; ++s) {
                uint64_t *bar = &c.misc->full[s % p.n_stages];
                uint32_t parity = (s / p.n_stages) & 1u;
                unsigned long long t0 = global_timer_ns();
                for (uint32_t n = 0; !mbar_try_wait(bar, parity); ++n)
                    if ((n & 255u) == 255u && global_timer_ns() - t0 > kWaitLimitNs) break;
            }
        }
        return;
    }

    // ---------------- consumers
    bf16_t *s_hi = reinterpret_cast<bf16_t *>(c.scr);
    const int KCd = p.KC;
    auto act_stride = [&](int len) { return ((len + 31) & ~31) + 32; };   // +64 B: rows land in different banks

    for (int step = 0; step < n_steps; ++step) {
        // ============ front end
        if (p.mode == 0) {
            // ---- PROJ: x0 = W_p [ rms(h) ; rms(Emb(tok)) ]
            const int st = act_stride(2 * p.d);
            bf16_t *a_hi = s_hi, *a_lo = s_hi + (size_t)R * st;
            if (c.tid < R) {
                int tok;
                if (step == 0) tok = p.tokens[c.tid];
                else {
                    unsigned long long key = ldcg_u64(p.s.keys + (size_t)(step - 1) * kMaxRows + c.tid);
                    if ((key >> 32) == 0ull) raise(c, kDevAllNan);
                    tok = (int)argmax_key_id(key);
                    if (c.cta == 0) p.out_tokens[(size_t)c.tid * p.K + (step - 1)] = tok;
                }
                if ((unsigned)tok >= (unsigned)p.V) { raise(c, kDevBadToken); tok = 0; }
                c.misc->tok[c.tid] = tok;
            }
            bar_sync(1, kConsumerThreads);
            float sq[kMaxRows][2];
            for (int r = 0; r < R; ++r) { sq[r][0] = 0.f; sq[r][1] = 0.f; }
            for (int r = 0; r < R; ++r) {
                const bf16_t *erow = p.embed + (size_t)c.misc->tok[r] * p.d;
                for (int k = c.tid * 8; k < p.d; k += kConsumerThreads * 8) {
                    uint4 ev = ldnc128(erow + k);
                    uint4 gv = ldnc128(p.g_enorm + k);
                    uint32_t ew[4] = {ev.x, ev.y, ev.z, ev.w}, gw[4] = {gv.x, gv.y, gv.z, gv.w};
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        float e0 = bf16lo_f32(ew[i]), e1 = bf16hi_f32(ew[i]);
                        sq[r][1] += e0 * e0 + e1 * e1;
                        store_split(a_hi, a_lo, (size_t)r * st + p.d + k + 2 * i, e0 * bf16lo_f32(gw[i]));
                        store_split(a_hi, a_lo, (size_t)r * st + p.d + k + 2 * i + 1, e1 * bf16hi_f32(gw[i]));
                    }
                    if (step == 0) {
                        uint4 hv = ldnc128(p.h_last + (size_t)r * p.d + k);
                        uint4 hg = ldnc128(p.g_hnorm + k);
                        uint32_t hw[4] = {hv.x, hv.y, hv.z, hv.w}, hgw[4] = {hg.x, hg.y, hg.z, hg.w};
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            float h0 = bf16lo_f32(hw[i]), h1 = bf16hi_f32(hw[i]);
                            sq[r][0] += h0 * h0 + h1 * h1;
                            store_split(a_hi, a_lo, (size_t)r * st + k + 2 * i, h0 * bf16lo_f32(hgw[i]));
                            store_split(a_hi, a_lo, (size_t)r * st + k + 2 * i + 1, h1 * bf16hi_f32(hgw[i]));
                        }
                    }
                }
            }
            if (step > 0) stage_hilo(c, p.s.actR_hi, p.s.actR_lo, p.dp, p.d, a_hi, a_lo, st, 0);
            block_sum2(c, sq, R);
            if (step > 0 && c.warp < R) {
                // recursed state: h = (x2*g_final) * s_x; rms(h) adds s_h = rsqrt(s_x^2 * mean((x2 g)^2) + eps)
                float sx = rsqrtf(sum_partials(c, p.s.ssC, c.warp) / (float)p.d + p.eps);
                float sy = sum_partials(c, p.s.ssD, c.warp) / (float)p.d;
                if (c.lane == 0) c.misc->scale0[c.warp] = sx * rsqrtf(sx * sx * sy + p.eps);
            }
            if (c.tid < R) {
                if (step == 0) c.misc->scale0[c.tid] = rsqrtf(c.misc->ssred[0][c.tid][0] / (float)p.d + p.eps);
                c.misc->scale1[c.tid] = rsqrtf(c.misc->ssred[0][c.tid][1] / (float)p.d + p.eps);
            }
            bar_sync(1, kConsumerThreads);
            SqAcc sqa;
            ActSrc act{a_hi, a_lo, st, true};
            const LayerPtrs &L0 = p.layers[0];
            consume_phase<PROJ>(c, act, p.d / KCd, [&](int row, int col, float v, float) {
                p.s.x0[(size_t)col * p.d + row] = v;
                store_split(p.s.actD_hi, p.s.actD_lo, (size_t)col * p.dp + row, v * bf16bits_f32(L0.g_in[row]));
                sqa.a += v * v;
            });
            flush_sq(c, sqa, p.s.ssA, nullptr);
            grid_barrier(c);
        } else {
            // ---- EMBED (target): x0 = Emb(tok), CTA-sliced over d
            int r0 = (int)(((long long)c.cta * p.d) / c.grid), r1 = (int)(((long long)(c.cta + 1) * p.d) / c.grid);
            // thread = (row slot tid>>3, activation row tid&7)
            SqAcc sqa;
            for (int row = r0 + (c.tid >> 3); row < r1; row += kTileRows) {
                int col = c.tid & 7;
                if (col < R) {
                    int tok = p.tokens[col];
                    if ((unsigned)tok >= (unsigned)p.V) { raise(c, kDevBadToken); tok = 0; }
                    float v = bf16bits_f32(p.embed[(size_t)tok * p.d + row]);
                    p.s.x0[(size_t)col * p.d + row] = v;
                    store_split(p.s.actD_hi, p.s.actD_lo, (size_t)col * p.dp + row,
                                v * bf16bits_f32(p.layers[0].g_in[row]));
                    sqa.a += v * v;
                }
            }
            flush_sq(c, sqa, p.s.ssA, nullptr);
            grid_barrier(c);
        }

        // ============ decoder layers
        for (int l = 0; l < n_layers; ++l) {
            const LayerPtrs &L = p.layers[l];
            const bool last_layer = (l + 1 == n_layers);
            // ---- QKV
            {
                const int st = act_stride(p.d);
                bf16_t *a_hi = s_hi, *a_lo = s_hi + (size_t)R * st;
                stage_hilo(c, p.s.actD_hi, p.s.actD_lo, p.dp, p.d, a_hi, a_lo, st, 0);
                if (c.warp < R) {
                    float s = rsqrtf(sum_partials(c, p.s.ssA, c.warp) / (float)p.d + p.eps);
                    if (c.lane == 0) c.misc->scale0[c.warp] = s;
                }
                bar_sync(1, kConsumerThreads);
                ActSrc act{a_hi, a_lo, st, true};
                const int nq = p.qdim + 2 * p.kvdim;
                consume_phase<QKV>(c, act, 0, [&](int row, int col, float v, float) {
                    p.s.qkv[(size_t)col * nq + row] = v * c.misc->scale0[col];
                });
                grid_barrier(c);
            }
            // ---- attention
            attention_phase(c, p.kvs[l], (p.mode == 0) ? step : 0);
            grid_barrier(c);
            // ---- O projection + residual
            {
                const int st = act_stride(p.qdim);
                bf16_t *a_hi = s_hi, *a_lo = s_hi + (size_t)R * st;
                stage_hilo(c, p.s.actO_hi, p.s.actO_lo, p.qp, p.qdim, a_hi, a_lo, st, 0);
                bar_sync(1, kConsumerThreads);
                ActSrc act{a_hi, a_lo, st, true};
                SqAcc sqa;
                consume_phase<OPROJ>(c, act, 0, [&](int row, int col, float v, float) {
                    float x = ldcg_f32(p.s.x0 + (size_t)col * p.d + row) + v;
                    p.s.x1[(size_t)col * p.d + row] = x;
                    store_split(p.s.actP_hi, p.s.actP_lo, (size_t)col * p.dp + row, x * bf16bits_f32(L.g_post[row]));
                    sqa.a += x * x;
                });
                flush_sq(c, sqa, p.s.ssB, nullptr);
                grid_barrier(c);
            }
            // ---- gate / up + SwiGLU
            {
                const int st = act_stride(p.d);
                bf16_t *a_hi = s_hi, *a_lo = s_hi + (size_t)R * st;
                stage_hilo(c, p.s.actP_hi, p.s.actP_lo, p.dp, p.d, a_hi, a_lo, st, 0);
                if (c.warp < R) {
                    float s = rsqrtf(sum_partials(c, p.s.ssB, c.warp) / (float)p.d + p.eps);
                    if (c.lane == 0) c.misc->scale0[c.warp] = s;
                }
                bar_sync(1, kConsumerThreads);
                ActSrc act{a_hi, a_lo, st, true};
                consume_phase<GATEUP>(c, act, 0, [&](int row, int col, float gt, float up) {
                    float s = c.misc->scale0[col];
                    gt *= s;
                    up *= s;
                    float a = gt / (1.f + expf(-gt)) * up;
                    store_split(p.s.actF_hi, p.s.actF_lo, (size_t)col * p.Fp + row, a);
                });
                grid_barrier(c);
            }
            // ---- down projection + residual
            {
                ActSrc act;
                if (p.stage_F_in_smem) {
                    const int st = act_stride(p.F);
                    bf16_t *a_hi = s_hi, *a_lo = s_hi + (size_t)R * st;
                    // Fp is a multiple of 32 and the pad beyond F is zero in global scratch
                    stage_hilo(c, p.s.actF_hi, p.s.actF_lo, p.Fp, p.Fp, a_hi, a_lo, st, 0);
                    bar_sync(1, kConsumerThreads);
                    act = ActSrc{a_hi, a_lo, st, true};
                } else {
                    act = ActSrc{p.s.actF_hi, p.s.actF_lo, p.Fp, false};
                }
                SqAcc sqa;
                const bf16_t *gnext = (p.mode == 1 && !last_layer) ? p.layers[l + 1].g_in : p.g_final;
                consume_phase<DOWN>(c, act, 0, [&](int row, int col, float v, float) {
                    float x = ldcg_f32(p.s.x1 + (size_t)col * p.d + row) + v;
                    float y = x * bf16bits_f32(gnext[row]);
                    sqa.a += x * x;
                    if (p.mode == 1 && !last_layer) {
                        p.s.x0[(size_t)col * p.d + row] = x;
                        store_split(p.s.actD_hi, p.s.actD_lo, (size_t)col * p.dp + row, y);
                    } else {
                        store_split(p.s.actH_hi, p.s.actH_lo, (size_t)col * p.dp + row, y);
                        if (p.mode == 0) {
                            store_split(p.s.actR_hi, p.s.actR_lo, (size_t)col * p.dp + row,
                                        y * bf16bits_f32(p.g_hnorm[row]));
                            sqa.b += y * y;
                        }
                    }
                });
                bool to_head = !(p.mode == 1 && !last_layer);
                flush_sq(c, sqa, to_head ? p.s.ssC : p.s.ssA, (p.mode == 0) ? p.s.ssD : nullptr);
                grid_barrier(c);
            }
        }

        // ============ output head
        {
            const int st = act_stride(p.d);
            bf16_t *a_hi = s_hi, *a_lo = s_hi + (size_t)R * st;
            stage_hilo(c, p.s.actH_hi, p.s.actH_lo, p.dp, p.d, a_hi, a_lo, st, 0);
            if (c.warp < R) {
                float s = rsqrtf(sum_partials(c, p.s.ssC, c.warp) / (float)p.d + p.eps);
                if (c.lane == 0) c.misc->scale0[c.warp] = s;
            }
            bar_sync(1, kConsumerThreads);
            if (p.out_h) {   // every CTA writes its slice of the post-final-norm hidden state
                int r0 = (int)(((long long)c.cta * p.d) / c.grid), r1 = (int)(((long long)(c.cta + 1) * p.d) / c.grid);
                for (int i = c.tid; i < R * (r1 - r0); i += kConsumerThreads) {
                    int r = i / (r1 - r0), k = r0 + (i - r * (r1 - r0));
                    float y = bf16bits_f32(a_hi[(size_t)r * st + k]) + bf16bits_f32(a_lo[(size_t)r * st + k]);
                    size_t o = (p.mode == 0) ? ((size_t)r * p.K + step) * p.d + k : (size_t)r * p.d + k;
                    p.out_h[o] = f32_bf16bits(y * c.misc->scale0[r]);
                }
            }
            ActSrc act{a_hi, a_lo, st, true};
            unsigned long long best = 0ull;
            consume_phase<HEAD>(c, act, 0, [&](int row, int col, float v, float) {
                int id = p.ids ? p.ids[row] : row;
                if ((unsigned)id >= (unsigned)p.V) id = 0;
                float lv = v;
                if (p.mode == 1) {
                    // target: the decision is taken on the bf16 logits that cross the boundary
                    uint16_t lb = f32_bf16bits(v * c.misc->scale0[col]);
                    if (p.out_logits_bf16) p.out_logits_bf16[(size_t)col * p.V + row] = lb;
                    lv = bf16bits_f32(lb);
                } else if (p.out_logits_f32) {
                    p.out_logits_f32[((size_t)col * p.K + step) * p.N + row] = v * c.misc->scale0[col];
                }
                unsigned long long key = argmax_key(lv, (uint32_t)id);
                best = key > best ? key : best;
            });
            // reduce the per-thread maxima (thread = (row slot, col)) over the 32 row slots
            {
                unsigned long long k = best;
                unsigned long long o8 = __shfl_xor_sync(0xffffffffu, k, 8);
                k = o8 > k ? o8 : k;
                unsigned long long o16 = __shfl_xor_sync(0xffffffffu, k, 16);
                k = o16 > k ? o16 : k;
                if (c.lane < 8) c.misc->keyred[c.warp][c.lane] = k;
                bar_sync(1, kConsumerThreads);
                if (c.tid < R) {
                    unsigned long long m = 0ull;
                    for (int w = 0; w < kConsumerWarps; ++w) m = c.misc->keyred[w][c.tid] > m ? c.misc->keyred[w][c.tid] : m;
                    if (m != 0ull) atomicMax(p.s.keys + (size_t)step * kMaxRows + c.tid, m);
                }
            }
            grid_barrier(c);
        }
    }

    // ============ publish the last step's tokens and the status word
    if (c.cta == 0 && c.tid < R) {
        int last = n_steps - 1;
        unsigned long long key = ldcg_u64(p.s.keys + (size_t)last * kMaxRows + c.tid);
        if ((key >> 32) == 0ull) raise(c, kDevAllNan);
        int tok = (int)argmax_key_id(key);
        if (p.out_tokens) {
            if (p.mode == 0) p.out_tokens[(size_t)c.tid * p.K + last] = tok;
            else p.out_tokens[c.tid] = tok;
        }
    }
    if (c.cta == 0 && c.tid == 0 && p.user_status) {
        __threadfence();
        uint32_t st = ldcg_u32(p.s.status);
        if (st) atomicOr(p.user_status, st);
    }
}

}  // namespace

size_t mega_smem_bytes(const MegaParams &p) {
    size_t off = (sizeof(Misc) + 127) & ~size_t(127);
    off += ((size_t)2 * kConsumerWarps * kTileRows * p.R * sizeof(float) + 127) & ~size_t(127);
    off += (size_t)p.scratch_smem;
    off += (size_t)p.n_stages * p.stage_bytes;
    return off;
}

size_t mega_fixed_smem(int R) {
    size_t off = (sizeof(Misc) + 127) & ~size_t(127);
    off += ((size_t)2 * kConsumerWarps * kTileRows * R * sizeof(float) + 127) & ~size_t(127);
    return off;
}

int mega_max_grid(size_t smem_bytes, int *err) {
    int dev = 0, sms = 0, per_sm = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(mega_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes);
    if (e == cudaSuccess) e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, mega_kernel, kThreads, smem_bytes);
    if (err) *err = (int)e;
    if (e != cudaSuccess) return 0;
    return sms * (per_sm > 0 ? 1 : 0);
}

int mega_launch(const MegaParams &p, int grid, cudaStream_t stream) {
    size_t smem = mega_smem_bytes(p);
    cudaError_t e = cudaFuncSetAttribute(mega_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return (int)e;
    void *args[] = {const_cast<MegaParams *>(&p)};
    e = cudaLaunchCooperativeKernel((const void *)mega_kernel, dim3(grid), dim3(kThreads), args, smem, stream);
    return (int)e;
}

}  // namespace fmtp
