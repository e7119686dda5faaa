// Weight-streaming GEMM for 5..64 activation rows on the sm_100a tensor cores (tcgen05 + TMEM).
//
//   D[m, n] = sum_k A[m, k] * X[n, k]      m: weight rows (128 per tile, the MMA's M)
//                                          n: activation columns (NB = 16..128, the MMA's N)
//
// The weight matrix is read exactly once from HBM; the activation operand X (bf16, row n = 2r is
// the high part of activation row r and n = 2r + 1 the low part, so the pair carries an fp32
// value) is small and re-read from L2 for every tile. One CTA per SM walks a static list of work
// items (tile, K range). Roles: warps 0-3 epilogue (TMEM -> registers -> global), warp 4 issues
// the MMAs, warps 5-12 copy A into a shared-memory ring with 16-byte cp.async, laid out as
// the MMA's 128-byte-swizzled K-major tiles (64 K elements wide); the X block of a stage comes by
// one TMA tile copy (same swizzle) through the copy engine, which leaves the load/store path's
// ~64 GB/s per SM to the weights: with 64 rows the X bytes equal the weight bytes. A ring stage holds KA such
// 64-wide blocks that are requested back to back, so a weight row is read in pieces of KA x 128
// contiguous bytes. Accumulators are double buffered in TMEM so the epilogue of one item overlaps
// the MMAs of the next.
//
// A stage's barrier counts one asynchronous arrival per copy thread (cp.async.mbarrier.arrive), so a
// stage is published the moment its bytes have landed.
//
// Every wait is time-bounded; on expiry the CTA raises the timeout flag, drains and returns.
#pragma once
#include "umma.cuh"
#include "batched.cuh"
#include <cuda.h>
#include <cstring>

namespace fmtp {

constexpr int kGemmProducers = 256;          // eight copy warps
constexpr int kGemmThreads = 160 + kGemmProducers;
constexpr int kGemmBK = 64;                 // K elements per swizzled block: one 128-byte row
constexpr int kGemmTileM = 128;
constexpr int kGemmMaxStages = 10;

enum GemmEpilogue {
    EPI_PARTIAL = 0,   // fp32 partial sums  partial[split][r][m] = D[m,2r] + D[m,2r+1]
    EPI_SWIGLU = 1,    // a tile holds 64 gate rows and the 64 up rows of the same indices: act = silu(g) * u, written as the
                       // hi/lo operand of the next GEMM
    EPI_ARGMAX = 2,    // per activation row the maximum of (logit, row id) as a packed key (atomicMax), optional fp32 logits
};

struct GemmArgs {
    const bf16_t *a[3];          // up to three matrices whose rows are concatenated (q, k, v); [rows][lda] bf16
    int a_rows[3];
    int n_seg;
    const bf16_t *a_up;          // EPI_SWIGLU: the up matrix (a[0] is the gate matrix, same shape)
    const int32_t *row_ids;      // optional: GEMM row m reads a[0][row_ids[m]] (compressed output head)
    int V;                       // rows of a[0] when row_ids is used (ids outside are clamped and flagged)
    int n_rows, K, lda;          // output rows (EPI_SWIGLU: ffn indices); K % 8 == 0
    const bf16_t *x;             // [NB][ldx] bf16
    int ldx, NB, R;              // NB % 16 == 0, 2R <= NB <= 128
    int splits, kb_per_split;    // K is cut into `splits` ranges of kb_per_split 64-wide blocks
    int epi;
    float *partial;              // [splits][R][ldp]
    int ldp;
    bf16_t *xop_out;             // EPI_SWIGLU: [>= 2R][ld_out]
    int ld_out;
    unsigned long long *keys;    // EPI_ARGMAX: [R]
    float *logits;               // EPI_ARGMAX, optional: row r at logits + r*logits_stride, column m
    long long logits_stride;
    bf16_t *logits_bf16;         // EPI_ARGMAX with round_bf16, optional: the logits as bf16, same indexing
    int round_bf16;              // 1: the argmax is decided on the logits rounded to bf16 (the values a caller sees)
    uint32_t *status;
    int n_stages;
    int force_ka;                // 0: pick the blocks per stage from the shared memory available
    unsigned long long wait_limit_ns;   // every wait of the kernel gives up after this long
    int extra_arrivals;          // self-test only: arrivals a ring stage expects beyond the copies that are made
};

struct GemmSmem {
    uint64_t full[kGemmMaxStages], empty[kGemmMaxStages];
    uint64_t tfull[2], tempty[2], drain;
    uint32_t tmem_base, abort_flag;
    unsigned long long kmax[4][64];
    float exch[64][17];          // EPI_SWIGLU: up-row sums handed to the gate rows' threads
};

__host__ __device__ inline int gemm_kblock_bytes(int NB) { return kGemmTileM * 128 + NB * 128; }
__host__ __device__ inline int gemm_tile_rows(int epi) { return epi == EPI_SWIGLU ? 64 : kGemmTileM; }

__device__ __forceinline__ bool gemm_wait(GemmSmem *sm, uint64_t *bar, uint32_t parity, unsigned long long limit_ns) {
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_timer_ns();
    uint32_t polls = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++polls & 63u) == 0) {
            if (*reinterpret_cast<volatile uint32_t *>(&sm->abort_flag)) return false;
            if (global_timer_ns() - t0 > limit_ns) {
                *reinterpret_cast<volatile uint32_t *>(&sm->abort_flag) = 1u;
                return false;
            }
        }
    }
    return true;
}

// Work items of a CTA: items (tile of 128 rows, K range) are dealt round-robin over the CTAs. (Giving every CTA
// an equal contiguous share of the output head's rows instead -- 221 rows as a full and a partial tile at the 7B
// shape, where 256 tiles are 1.7 rounds of 148 CTAs -- was measured 3 % slower: the second round's 108 CTAs still
// saturate HBM, and partial tiles cost issue slots.)
struct GemmItem { int row0, row_end, split; };
__device__ __forceinline__ int gemm_my_items(const GemmArgs &g, int n_items) {
    return (int)blockIdx.x < n_items ? (n_items - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
}
__device__ __forceinline__ GemmItem gemm_my_item(const GemmArgs &g, int i) {
    GemmItem it;
    const int item = (int)blockIdx.x + i * (int)gridDim.x;
    const int tile = item / g.splits, tile_rows = gemm_tile_rows(g.epi);
    it.split = item - tile * g.splits;
    it.row0 = tile * tile_rows;
    it.row_end = min(it.row0 + tile_rows, g.n_rows);
    return it;
}

// True on all 128 epilogue threads (warps 0-3) if `flag` is set on any of them.
__device__ __forceinline__ bool epi_any(bool flag) {
    uint32_t out;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 p, %1, 0;\n\t"
        "bar.red.or.pred q, 2, 128, p;\n\t"
        "selp.u32 %0, 1, 0, q;\n\t}"
        : "=r"(out)
        : "r"(flag ? 1u : 0u)
        : "memory");
    return out != 0;
}

// One TMA tile copy global -> shared (2-D tensor map, element coordinates x, y); its bytes are counted on `bar`.
// x * element size must be a multiple of 16 bytes.
__device__ __forceinline__ void tma_load_2d(uint32_t dst_smem, const CUtensorMap *map, int x, int y, uint64_t *bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst_smem), "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar))
        : "memory");
}

// State of one producer thread's walk over the ring.
struct GemmProducer {
    uint32_t dst0;            // shared address of this thread's chunk in row r0 of stage 0
    int stage_bytes, kblock_bytes, S, c;
    int stage;
    uint32_t phase;
    bool tma_thread;          // the one producer thread that issues the X tile copies
    uint32_t dst_x;           // shared address of the X tile in block 0 of stage 0
    const CUtensorMap *xmap;
    uint64_t *full;
    uint64_t policy;          // L2 eviction policy of the weight stream
};

// Copies this thread's share of K block kb + J (if it is inside the item) into block J of the
// current stage. Source addresses are the per-row pointers plus the immediate J * 128 bytes, so
// all blocks of a stage go out before a pointer register is rewritten.
// PART: 1 = the weight rows only, 2 = the activation rows only, 3 = both.
template <int J, int PART>
__device__ __forceinline__ void produce_kblock(const GemmArgs &g, const GemmProducer &pr, int kb, int kb1,
                                               const bf16_t *(&ap)[4], const uint32_t (&aok)[4]) {
    if (kb + J >= kb1) return;
    if ((PART & 2) && pr.tma_thread)
        tma_load_2d(pr.dst_x + (uint32_t)pr.stage * pr.stage_bytes + (uint32_t)J * pr.kblock_bytes, pr.xmap, (kb + J) * kGemmBK, 0,
                    pr.full + pr.stage);
    if (!(PART & 1)) return;
    const bool kvalid = (kb + J) * kGemmBK + pr.c * 8 < g.K;
    const uint32_t dst = pr.dst0 + (uint32_t)pr.stage * pr.stage_bytes + (uint32_t)J * pr.kblock_bytes;
    if (kvalid && (aok[0] & aok[1] & aok[2] & aok[3]) != 0u) {      // the common case: plain 16-byte copies
#pragma unroll
        for (int i = 0; i < 4; ++i) cp_async16_full_hint<J * 128>(dst + i * 4096, ap[i], pr.policy);
    } else if (kvalid) {
#pragma unroll
        for (int i = 0; i < 4; ++i) cp_async16_off_hint<J * 128>(dst + i * 4096, ap[i], aok[i], pr.policy);
    } else {   // this chunk column lies beyond K: zeros, nothing is read
#pragma unroll
        for (int i = 0; i < 4; ++i) cp_async16_off<0>(dst + i * 4096, g.a[0], 0u);
    }
}

template <int KA, int PART>
__device__ __forceinline__ void produce_stage(const GemmArgs &g, const GemmProducer &pr, int kb, int kb1,
                                              const bf16_t *(&ap)[4], const uint32_t (&aok)[4]) {
    produce_kblock<0, PART>(g, pr, kb, kb1, ap, aok);
    if constexpr (KA > 1) produce_kblock<1, PART>(g, pr, kb, kb1, ap, aok);
    if constexpr (KA > 2) {
        produce_kblock<2, PART>(g, pr, kb, kb1, ap, aok);
        produce_kblock<3, PART>(g, pr, kb, kb1, ap, aok);
    }
}

// KA 64-wide K blocks per ring stage; every stage of the ring can be in flight.
template <int KA>
__global__ void __launch_bounds__(kGemmThreads, 1) skinny_gemm_kernel(const GemmArgs g, const __grid_constant__ CUtensorMap xmap) {
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    unsigned char *ring = smem_raw + ((1024u - (raw & 1023u)) & 1023u);
    const int S = g.n_stages;
    const int kblock_bytes = gemm_kblock_bytes(g.NB);
    const int stage_bytes = KA * kblock_bytes;
    GemmSmem *sm = reinterpret_cast<GemmSmem *>(ring + (size_t)S * stage_bytes);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    const int buf_cols = (g.NB + 31) & ~31;                 // TMEM columns of one accumulator buffer
    uint32_t alloc_cols = 32;
    while ((int)alloc_cols < 2 * buf_cols) alloc_cols <<= 1;

    if (tid == 0) {
        for (int s = 0; s < S; ++s) { mbar_init(&sm->full[s], kGemmProducers + 1 + g.extra_arrivals); mbar_init(&sm->empty[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&sm->tfull[b], 1); mbar_init(&sm->tempty[b], 128); }
        mbar_init(&sm->drain, 1);
        sm->abort_flag = 0;
        mbar_fence_init();
    }
    if (warp == 4) {
        tmem_alloc(&sm->tmem_base, alloc_cols);
        tmem_relinquish();
        tc_fence_before_sync();
    }
    chain_release();         // the next kernel of the stream may start its own set-up
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t *>(&sm->tmem_base);

    const int tile_rows = gemm_tile_rows(g.epi);
    const int n_tiles = (g.n_rows + tile_rows - 1) / tile_rows;
    const int n_items = n_tiles * g.splits;
    const int n_kb = (g.K + kGemmBK - 1) / kGemmBK;

    if (warp >= 5) {
        // ================= producers: thread pt copies chunk column c of tile rows r0 + 32 i
        const int pt = tid - 160;
        const int c = pt & 7, r0 = pt >> 3;
        GemmProducer pr;
        pr.dst0 = smem_u32(ring) + (uint32_t)(r0 * 128 + ((c ^ (r0 & 7)) << 4));
        pr.stage_bytes = stage_bytes; pr.kblock_bytes = kblock_bytes; pr.S = S; pr.c = c;
        pr.stage = 0; pr.phase = 0;
        pr.policy = l2_evict_first();
        pr.tma_thread = pt == 0; pr.dst_x = smem_u32(ring) + 16384; pr.xmap = &xmap; pr.full = sm->full;
        bool ok_run = true;
        const bf16_t *ap[4];
        uint32_t aok[4];
        int kb0 = 0, kb1 = 0;
        auto setup_item = [&](int i) {
            const GemmItem gi = gemm_my_item(g, i);
            kb0 = gi.split * g.kb_per_split;
            kb1 = kb0 + g.kb_per_split;
            if (kb1 > n_kb) kb1 = n_kb;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int tr = r0 + 32 * i;
                const bf16_t *base = g.a[0];
                int m;
                if (g.epi == EPI_SWIGLU) {             // tile rows 0-63: gate rows, 64-127: the up rows of the same indices
                    m = gi.row0 + (tr & 63);
                    if (tr >= 64) base = g.a_up;
                } else {
                    m = gi.row0 + tr;
                }
                aok[i] = m < gi.row_end ? 16u : 0u;
                if (m >= gi.row_end) m = gi.row_end - 1;
                int row = m;
                if (g.row_ids) {
                    int id = g.row_ids[m];
                    if ((unsigned)id >= (unsigned)g.V) { atomicOr(g.status, 0x1u); id = 0; }
                    row = id;
                } else if (g.n_seg > 1) {
                    if (row >= g.a_rows[0]) {
                        row -= g.a_rows[0];
                        base = g.a[1];
                        if (row >= g.a_rows[1]) { row -= g.a_rows[1]; base = g.a[2]; }
                    }
                }
                ap[i] = base + (size_t)row * g.lda + (size_t)kb0 * kGemmBK + c * 8;
            }
        };
        // The weights do not depend on the predecessor in the stream: the weight part of the first item's first
        // stages goes out before waiting for it.
        const int n_my = gemm_my_items(g, n_items);
        // The gathered head reads its row ids, which a kernel earlier in the same call wrote: that is a real
        // dependency, so those GEMMs wait for the chain first (and give up the early weight requests below).
        if (g.row_ids) chain_wait();
        if (n_my > 0) setup_item(0);
        int pre = 0;
        for (int kb = kb0; kb < kb1 && pre < S; kb += KA, ++pre) {
            pr.stage = pre;
            produce_stage<KA, 1>(g, pr, kb, kb1, ap, aok);
#pragma unroll
            for (int i = 0; i < 4; ++i) ap[i] += KA * kGemmBK;
        }
        pr.stage = 0;
        chain_wait();
        for (int i = 0; i < n_my && ok_run; ++i) {
            if (i > 0) setup_item(i);
            for (int kb = kb0; kb < kb1; kb += KA) {
                if (!gemm_wait(sm, &sm->empty[pr.stage], pr.phase ^ 1u, g.wait_limit_ns)) { ok_run = false; break; }
                if (pr.tma_thread) {   // the X tiles of this stage: their bytes are expected on the stage's barrier
                    const int nv = kb1 - kb < KA ? kb1 - kb : KA;
                    mbar_arrive_expect_tx(&sm->full[pr.stage], (uint32_t)(nv * g.NB * 128));
                }
                if (pre > 0) {      // weight part already in flight: add the activation part
                    --pre;
                    produce_stage<KA, 2>(g, pr, kb, kb1, ap, aok);
                } else {
                    produce_stage<KA, 3>(g, pr, kb, kb1, ap, aok);
#pragma unroll
                    for (int i = 0; i < 4; ++i) ap[i] += KA * kGemmBK;
                }
                // this thread's arrival on the stage's barrier fires when its copies above have landed
                cp_async_arrive(&sm->full[pr.stage]);
                if (++pr.stage == S) { pr.stage = 0; pr.phase ^= 1u; }
            }
        }
        cp_async_wait_all();
    } else if (warp == 4) {
        // ================= MMA issue: one thread
        chain_wait();
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_bf16(g.NB);
            int stage = 0;
            uint32_t phase = 0, tphase[2] = {0, 0};
            int buf = 0;
            bool ok_run = true;
            const int n_my = gemm_my_items(g, n_items);
            for (int i = 0; i < n_my && ok_run; ++i) {
                const int kb0 = gemm_my_item(g, i).split * g.kb_per_split;
                int kb1 = kb0 + g.kb_per_split;
                if (kb1 > n_kb) kb1 = n_kb;
                if (!gemm_wait(sm, &sm->tempty[buf], tphase[buf] ^ 1u, g.wait_limit_ns)) break;
                tc_fence_after_sync();
                const uint32_t d0 = tmem_base + (uint32_t)(buf * buf_cols);
                for (int kb = kb0; kb < kb1; kb += KA) {
                    if (!gemm_wait(sm, &sm->full[stage], phase, g.wait_limit_ns)) { ok_run = false; break; }
                    fence_proxy_async();          // the copies' shared-memory writes, before the tensor core reads them
                    tc_fence_after_sync();
#pragma unroll
                    for (int j = 0; j < KA; ++j) {
                        if (kb + j < kb1) {
                            const uint32_t sa = smem_u32(ring) + (uint32_t)stage * stage_bytes + (uint32_t)j * kblock_bytes;
                            const uint32_t sb = sa + 16384;
#pragma unroll
                            for (int ks = 0; ks < 4; ++ks)
                                umma_bf16(d0, umma_smem_desc(sa + ks * 32), umma_smem_desc(sb + ks * 32), idesc,
                                          (kb + j > kb0) || (ks > 0));
                        }
                    }
                    umma_commit(&sm->empty[stage]);
                    if (++stage == S) { stage = 0; phase ^= 1u; }
                }
                if (!ok_run) break;
                umma_commit(&sm->tfull[buf]);
                tphase[buf] ^= 1u;
                buf ^= 1;
            }
            // every MMA issued above has completed once this arrival lands
            umma_commit(&sm->drain);
            gemm_wait(sm, &sm->drain, 0, g.wait_limit_ns);
        }
        __syncwarp();
    } else {
        // ================= epilogue: thread = one row of the tile (TMEM lane 32*warp + lane)
        chain_wait();
        uint32_t tphase[2] = {0, 0};
        int buf = 0;
        const int n_my = gemm_my_items(g, n_items);
        for (int i = 0; i < n_my; ++i) {
            const GemmItem gi = gemm_my_item(g, i);
            const int split = gi.split;
            // the 128 epilogue threads agree on the outcome of the wait before any of them moves on
            if (epi_any(!gemm_wait(sm, &sm->tfull[buf], tphase[buf], g.wait_limit_ns))) break;
            tc_fence_after_sync();
            const int tr = warp * 32 + lane;
            const int m = g.epi == EPI_SWIGLU ? gi.row0 + (tr & 63) : gi.row0 + tr;
            const bool m_ok = m < gi.row_end;
            const uint32_t t0 = tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)(buf * buf_cols);
            uint32_t row_id = (uint32_t)m;
            if (g.epi == EPI_ARGMAX && g.row_ids && m_ok) {
                int id = g.row_ids[m];
                row_id = ((unsigned)id >= (unsigned)g.V) ? 0u : (uint32_t)id;
            }
            for (int c0 = 0; c0 < g.NB; c0 += 32) {
                float v[32];
                tmem_ld32(t0 + c0, v);
                if (g.epi == EPI_PARTIAL) {
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const int r = (c0 >> 1) + j;
                        if (r < g.R && m_ok) g.partial[((size_t)split * g.R + r) * g.ldp + m] = v[2 * j] + v[2 * j + 1];
                    }
                } else if (g.epi == EPI_SWIGLU) {
                    if (warp >= 2) {
#pragma unroll
                        for (int j = 0; j < 16; ++j) sm->exch[tr - 64][j] = v[2 * j] + v[2 * j + 1];
                    }
                    bar_sync(1, 128);
                    if (warp < 2) {
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            const int r = (c0 >> 1) + j;
                            if (r < g.R && m_ok) {
                                const float gv = v[2 * j] + v[2 * j + 1], uv = sm->exch[tr][j];
                                const float act = gv / (1.0f + expf(-gv)) * uv;
                                uint16_t hi, lo;
                                split_bf16(act, hi, lo);
                                g.xop_out[(size_t)(2 * r) * g.ld_out + m] = hi;
                                g.xop_out[(size_t)(2 * r + 1) * g.ld_out + m] = lo;
                            }
                        }
                    }
                    bar_sync(1, 128);
                } else {
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const int r = (c0 >> 1) + j;           // warp-uniform
                        if (r < g.R) {
                            float logit = v[2 * j] + v[2 * j + 1];
                            if (g.logits && m_ok) g.logits[(size_t)r * g.logits_stride + m] = logit;
                            if (g.round_bf16) {
                                const uint16_t b = f32_bf16bits(logit);
                                if (g.logits_bf16 && m_ok) g.logits_bf16[(size_t)r * g.logits_stride + m] = b;
                                logit = bf16bits_f32(b);
                            }
                            unsigned long long key = m_ok ? argmax_key(logit, row_id) : 0ull;
#pragma unroll
                            for (int o = 16; o > 0; o >>= 1) {
                                const unsigned long long other = __shfl_xor_sync(0xffffffffu, key, o);
                                key = other > key ? other : key;
                            }
                            if (lane == 0) sm->kmax[warp][r] = key;
                        }
                    }
                }
            }
            tc_fence_before_sync();
            mbar_arrive(&sm->tempty[buf]);
            tphase[buf] ^= 1u;
            buf ^= 1;
            if (g.epi == EPI_ARGMAX) {
                bar_sync(1, 128);
                if (tid < g.R && g.keys) {
                    unsigned long long k = sm->kmax[0][tid];
#pragma unroll
                    for (int w = 1; w < 4; ++w) k = sm->kmax[w][tid] > k ? sm->kmax[w][tid] : k;
                    atomicMax(&g.keys[tid], k);
                }
                bar_sync(1, 128);
            }
        }
    }
    __syncthreads();
    if (tid == 0 && *reinterpret_cast<volatile uint32_t *>(&sm->abort_flag)) atomicOr(g.status, 0x8u);
    if (warp == 4) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, alloc_cols);
    }
}

// Tensor map of the activation operand X [NB][ldx] (bf16): tiles of 64 K elements x NB rows, 128-byte
// swizzle (the layout the MMA reads), zeros beyond K. Returns 0 or a cudaError_t.
inline int gemm_encode_xmap(CUtensorMap *map, const bf16_t *x, int ldx, int K, int NB) {
    typedef CUresult (*encode_fn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    static encode_fn encode = nullptr;
    if (!encode) {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qr;
        cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qr);
        if (e != cudaSuccess) return (int)e;
        if (!fn || qr != cudaDriverEntryPointSuccess) return (int)cudaErrorNotSupported;
        encode = reinterpret_cast<encode_fn>(fn);
    }
    const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)NB};
    const cuuint64_t strides[1] = {(cuuint64_t)ldx * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kGemmBK, (cuuint32_t)NB};
    const cuuint32_t estr[2] = {1, 1};
    CUresult r = encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<bf16_t *>(x), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? 0 : (int)cudaErrorInvalidValue;
}

// Launches the GEMM on `stream` with one CTA per SM (fewer when there are fewer work items).
// Returns the cudaError_t of the launch.
inline int skinny_gemm_launch(GemmArgs g, int n_sm, int smem_optin, cudaStream_t stream, TmapCache *cache) {
    const int avail = smem_optin - 1024 - (int)sizeof(GemmSmem);
    const int kbb = gemm_kblock_bytes(g.NB);
    // blocks per stage: as many as still leave a ring of three stages
    int ka = g.force_ka > 0 ? g.force_ka : (avail / (4 * kbb) >= 3 ? 4 : avail / (2 * kbb) >= 3 ? 2 : 1);
    int stages = avail / (ka * kbb);
    if (stages > kGemmMaxStages) stages = kGemmMaxStages;
    if (stages < 3) return (int)cudaErrorInvalidConfiguration;
    g.n_stages = stages;
    const size_t smem = 1024 + (size_t)stages * ka * kbb + sizeof(GemmSmem);
    const int tile_rows = gemm_tile_rows(g.epi);
    const int n_items = ((g.n_rows + tile_rows - 1) / tile_rows) * g.splits;
    const int grid = n_items < n_sm ? n_items : n_sm;
    void (*kern)(const GemmArgs, const CUtensorMap) = ka == 4 ? skinny_gemm_kernel<4> : ka == 2 ? skinny_gemm_kernel<2> : skinny_gemm_kernel<1>;
    if (ka != 1 && ka != 2 && ka != 4) return (int)cudaErrorInvalidConfiguration;
    cudaError_t e = cudaSuccess;
    int &limit = cache->gemm_smem[ka == 4 ? 2 : ka == 2 ? 1 : 0];
    if ((int)smem > limit) {                  // raise the kernel's shared-memory limit once per footprint
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return (int)e;
        limit = (int)smem;
    }
    // the operand's tensor map depends on (address, row pitch, K, rows) only: encoded once, then reused
    CUtensorMap xmap;
    static_assert(sizeof(CUtensorMap) == 128, "tensor map size");
    TmapEntry *hit = nullptr;
    for (int i = 0; i < cache->n; ++i)
        if (cache->e[i].x == g.x && cache->e[i].ldx == g.ldx && cache->e[i].K == g.K && cache->e[i].NB == g.NB) { hit = &cache->e[i]; break; }
    if (hit) std::memcpy(&xmap, hit->map, sizeof(xmap));
    else {
        int rc = gemm_encode_xmap(&xmap, g.x, g.ldx, g.K, g.NB);
        if (rc) return rc;
        const int cap = (int)(sizeof(cache->e) / sizeof(cache->e[0]));
        TmapEntry &dst = cache->e[cache->n < cap ? cache->n++ : (cache->next++ % cap)];
        dst.x = g.x; dst.ldx = g.ldx; dst.K = g.K; dst.NB = g.NB;
        std::memcpy(dst.map, &xmap, sizeof(xmap));
    }
    e = launch_chained(kern, dim3(grid), dim3(kGemmThreads), smem, stream, g, xmap);
    return (int)e;
}

}  // namespace fmtp
