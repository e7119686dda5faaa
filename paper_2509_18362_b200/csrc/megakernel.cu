// Persistent decoder kernel: one cooperative launch runs every phase of K recursive MTP draft
// steps (or of one target-decoder step) with grid barriers in between, so a draft call never
// returns to the host between steps.
//
// Structure of a CTA (one per SM): 8 consumer warps + 4 producer warps.
//   * The producers stream bf16 weight rows from HBM into a ring of shared-memory stages with
//     16-byte cp.async copies whose completion is counted on mbarriers (on B200 this path sustains
//     ~65 GB/s per SM where 1 KB bulk copies reach ~25 GB/s and large ones ~47 GB/s). Weight addresses do not depend on activations, so the producers
//     run ahead of the grid barriers: while the consumers wait for the previous phase's vector,
//     HBM keeps streaming the next phase's rows.
//   * A matrix-vector phase gives every CTA a contiguous range of output rows. A stage holds up
//     to 32 rows x KC columns; the two halves of the consumer warps take alternate stages, each
//     warp a fixed k-slice, and multiply with mma.sync m16n8k16 (weights = A operand, activation
//     rows = B operand columns), then reduce across warps in a fixed order. The activation vector
//     is fp32 carried as two bf16 numbers (hi + lo, two adjacent MMA columns), so products are
//     exact and the sum is fp32-accurate; every activation row has its own column pair, so a
//     row's result does not depend on how many other rows the call carries.
//   * RMSNorm is folded: the producing phase stores x*g (split hi/lo) plus per-CTA partial sums of
//     x^2; the consuming phase multiplies its accumulators by rsqrt(mean(x^2)+eps).
//   * Attention splits the context into fixed 64-token chunks (work items over sequence x KV head
//     x chunk) whose committed K/V the producers stream through the same ring; scores and the weighted sum
//     run on mma.sync with the query heads (and the probabilities) split into bf16 high and low parts, fp32 softmax
//     per chunk; after a grid barrier a merge phase, spread over all CTAs, combines a head's chunk
//     partials in ascending order -- no float atomics anywhere, results are reproducible.
//   * Producers and consumers each walk the phase program from ONE loop with a runtime phase
//     kind: the code is much larger than the instruction cache, and straight-line code that runs
//     once per step is fetched from L2 (measured: 3-10x slower than the same code in a loop).
//   * Tensor memory as a second staging level (large shapes with at most four activation rows): the ring of
//     shared-memory stages holds 4 us of the stream, a phase end (epilogue, grid barrier, the wait for the slowest
//     CTA, staging of the next input vector) lasts 5-7 us, so HBM idled at every phase end. A mover thread copies
//     the first eight stages of every phase, as they land, into the eight slots of the SM's 256 KB tensor memory
//     (tcgen05.cp, 32 KB per stage; measured 0.47 us per stage, faster than the 0.67 us at which stages arrive but
//     slower than the consumers, hence only the head of a phase) and frees their shared-memory stages at once; the
//     consumers read those stages' MMA fragments from tensor memory (tcgen05.ld), the rest from shared memory.
//     The producers then run up to 14 stages (9 us) ahead of the consumers.
//   * The output head gathers rows W[ids[j]] (Eq. 3 of the paper), keeps a running (value, id)
//     maximum per activation row and publishes it with one 64-bit atomicMax per CTA; logits are
//     never written unless a debug buffer is passed.
#include "mega.cuh"
#include "ptx.cuh"
#include "umma.cuh"

#include <cooperative_groups.h>

namespace fmtp {

namespace {

constexpr uint32_t kDevBadToken = 0x1u, kDevBadPage = 0x2u, kDevBadPos = 0x4u, kDevTimeout = 0x8u,
                   kDevAllNan = 0x10u;


enum Kind { PROJ = 0, QKV = 1, OPROJ = 2, GATEUP = 3, DOWN = 4, HEAD = 5, ATTN = 6, EMBED = 7, MERGE = 8, DONE = 9 };

// The phase program of a launch. Draft: K x (PROJ, QKV, ATTN, MERGE, OPROJ, GATEUP, DOWN, HEAD).
// Target step: EMBED, n_layers x (QKV, ATTN, MERGE, OPROJ, GATEUP, DOWN), HEAD. Producers and consumers
// walk it independently with this iterator, each from a single loop.
struct Prog { int step, layer, kind; };

struct Misc {   // small shared-memory block
    uint64_t full[kMaxStages];
    uint64_t empty[kMaxStages];
    uint64_t tfull[kTmSlots];     // tensor-memory slots: filled by the mover's copies / read out by the four owning warps
    uint64_t tempty[kTmSlots];
    uint64_t tdrain;              // the mover's last copies, before the tensor memory is freed
    uint32_t tmem_base;
    uint32_t use_done[kMaxStages];   // per ring slot: uses whose data has been taken out (read by consumers or moved)
    float scale0[kMaxRows];
    float scale1[kMaxRows];
    float ssred[kConsumerWarps][kMaxRows][2];
    float colred[kTileRows][kMaxRows];
    unsigned long long keyred[kConsumerWarps][kMaxRows];
    int tok[kMaxRows];
    int outrow[kMaxRows];   // where the head publishes activation row r (out_row), set when the head's input is staged
    int seqlen[kMaxRows];   // committed length of every sequence and its number of extend rows, read once at kernel start:
    int next[kMaxRows];     // neither changes during a launch, and every phase that needs them saves an L2 round trip
    unsigned long long rowptr[kProducerWarps][32];   // tile row pointers, one line per producer warp
    int flag;
    uint32_t aborted;
};

// Development aid, compiled only with -DFMTP_PROF: consumer thread 0 of every CTA stamps the
// global timer at phase boundaries, and warp 0 of each role accumulates the cycles it spends
// waiting / working, into device arrays the host reads with fmtp_prof_read() / fmtp_prof_wait().
#ifdef FMTP_PROF
constexpr int kProfMarks = 512;
__device__ unsigned long long g_prof[160][kProfMarks];
__device__ long long g_wait[160][8];   // consumer wait-full, consumer stage body, producer wait-empty, producer issue
#define PROF(c, tag) do { if ((c).tid == 0 && (c).nprof < kProfMarks) g_prof[(c).cta][(c).nprof++] = ((unsigned long long)(tag) << 48) | (global_timer_ns() & 0xffffffffffffull); } while (0)
#define PROF_T0() long long prof_t0 = clock64()
#define PROF_ACC(c, slot, cond) do { if (cond) { long long prof_t1 = clock64(); (c).pacc[slot] += prof_t1 - prof_t0; prof_t0 = prof_t1; } } while (0)
#define PROF_FLUSH(c, lo, hi, cond) do { if (cond) for (int q_ = lo; q_ < hi; ++q_) atomicAdd((unsigned long long *)&g_wait[(c).cta][q_], (unsigned long long)(c).pacc[q_]); } while (0)
#else
#define PROF(c, tag) do { } while (0)
#define PROF_T0() do { } while (0)
#define PROF_ACC(c, slot, cond) do { } while (0)
#define PROF_FLUSH(c, lo, hi, cond) do { } while (0)
#endif

// Per-thread view of the CTA's state. Every function that takes it is force-inlined: if its address
// escaped into a real call the whole struct would live in local memory and each field access
// would queue behind the cp.async traffic in the load/store unit.
struct Cta {
#ifdef FMTP_PROF
    int nprof;
    long long pacc[5];
#endif
    const MegaParams *p;
    Misc *misc;
    float *red;            // [2][8 warps][32 rows][R]
    unsigned char *scr;    // per-phase scratch (activation staging / attention)
    unsigned char *ring;
    int cta, grid, tid, warp, lane;
    int R, M;              // activation rows and rows per sequence of the current step (see set_step_rows)
    int slot;              // ring slot of the next stage (same sequence in producer and consumers)
    uint32_t parity;       // mbarrier phase parity of that slot
    int tslot;             // tensor-memory slot of the next matrix stage (same sequence in mover and consumers)
    uint32_t tparity;
    uint32_t tmem;         // base address of the CTA's tensor memory
    uint32_t bar_target;   // grid barrier generation
    int redbuf;
};

__device__ __forceinline__ void next_stage(Cta &c) {
    if (++c.slot == c.p->n_stages) { c.slot = 0; c.parity ^= 1u; }
}
__device__ __forceinline__ void next_tslot(Cta &c) {
    if (++c.tslot == kTmSlots) { c.tslot = 0; c.tparity ^= 1u; }
}
__device__ __forceinline__ void raise(const Cta &c, uint32_t bits) { atomicOr(c.p->s.status, bits); }

__device__ __forceinline__ bool aborted(const Cta &c) { return *((volatile uint32_t *)&c.misc->aborted) != 0; }

// Bounded wait on an mbarrier phase (kept inline: a real call makes ptxas ignore setmaxnreg), called
// from every ring wait. Returns false on timeout or abort, after setting the status bits.
__device__ __forceinline__ bool wait_bar_impl(Misc *misc, uint64_t *bar, uint32_t parity, uint32_t *abort_flag, uint32_t *status,
                                              unsigned long long limit_ns) {
    if (*((volatile uint32_t *)&misc->aborted) != 0) return false;
    unsigned long long t0 = 0;
    for (uint32_t n = 0;; ++n) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((n & 255u) == 255u) {
            if (ldcg_u32(abort_flag) != 0) {
                misc->aborted = 1;
                return false;
            }
            unsigned long long now = global_timer_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > limit_ns) break;
        }
    }
    misc->aborted = 1;
    atomicOr(status, kDevTimeout);
    atomicExch(abort_flag, 1u);
    return false;
}
__device__ __forceinline__ bool wait_bar(const Cta &c, uint64_t *bar, uint32_t parity) {
    if (mbar_try_wait(bar, parity)) return true;          // fast path: already complete
    return wait_bar_impl(c.misc, bar, parity, c.p->s.abort_flag, c.p->s.status, c.p->wait_limit_ns);
}
// The same wait for a thread that is in no hurry (the mover of the tensor-memory path): it sleeps between polls, so
// that its spinning does not take issue slots and load/store bandwidth from the producer and consumer warps that
// share its scheduler.
__device__ __forceinline__ bool wait_bar_idle(const Cta &c, uint64_t *bar, uint32_t parity) {
    if (aborted(c)) return false;
    unsigned long long t0 = 0;
    for (uint32_t n = 0;; ++n) {
        if (mbar_try_wait(bar, parity)) return true;
        __nanosleep(64);
        if ((n & 63u) == 63u) {
            if (ldcg_u32(c.p->s.abort_flag) != 0) { c.misc->aborted = 1; return false; }
            const unsigned long long now = global_timer_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > c.p->wait_limit_ns) break;
        }
    }
    c.misc->aborted = 1;
    atomicOr(c.p->s.status, kDevTimeout);
    atomicExch(c.p->s.abort_flag, 1u);
    return false;
}
__device__ __forceinline__ void do_abort(const Cta &c) {
    c.misc->aborted = 1;
    atomicOr(c.p->s.status, kDevTimeout);
    atomicExch(c.p->s.abort_flag, 1u);
}

// Grid-wide barrier among the consumer threads of all CTAs (the producer warp never joins).
__device__ __forceinline__ void grid_barrier(Cta &c) {
    bar_sync(1, kConsumerThreads);
    c.bar_target += (uint32_t)(c.grid + c.p->extra_arrivals);     // extra_arrivals: 0, or 1 in the wait-timeout self-test
    if (c.tid == 0) {
        // the arrival is a release at device scope: it orders every write the CTA made before the bar.sync above
        // (the waiting side reads with acquire), so no separate fences are needed
        asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(c.p->s.barrier) : "memory");
        if (!aborted(c)) {
            uint32_t n = 0;
            unsigned long long t0 = 0;
            while ((int32_t)(ld_acquire_u32(c.p->s.barrier) - c.bar_target) < 0) {
                if ((++n & 255u) == 255u) {
                    if (ldcg_u32(c.p->s.abort_flag) != 0) { c.misc->aborted = 1; break; }
                    unsigned long long now = global_timer_ns();
                    if (t0 == 0) t0 = now;
                    else if (now - t0 > c.p->wait_limit_ns) { do_abort(c); break; }
                }
            }
        }
    }
    bar_sync(1, kConsumerThreads);
}

__device__ __forceinline__ void prog_begin(const MegaParams &p, Prog &g) {
    g.step = 0; g.layer = 0; g.kind = (p.mode == 0) ? PROJ : EMBED;
}
__device__ __forceinline__ void prog_next(const MegaParams &p, Prog &g) {
    switch (g.kind) {
        case PROJ: case EMBED: g.kind = QKV; break;
        case QKV: g.kind = ATTN; break;
        case ATTN: g.kind = MERGE; break;
        case MERGE: g.kind = OPROJ; break;
        case OPROJ: g.kind = GATEUP; break;
        case GATEUP: g.kind = DOWN; break;
        case DOWN:
            if (p.mode == 1 && g.layer + 1 < p.n_layers) { g.layer++; g.kind = QKV; }
            else g.kind = HEAD;
            break;
        default:   // HEAD
            g.step++; g.layer = 0;
            g.kind = (p.mode == 0 && g.step < p.K) ? PROJ : DONE;
            break;
    }
}

// ---- rows of a step --------------------------------------------------------------------------
// Target step: every sequence carries p.M rows at positions L .. L+M-1. Draft: step 0 carries up to p.M
// "extend" rows per sequence -- the pairs (target hidden state, next token) of the positions committed
// since the last call, causal among themselves at positions L .. L+n-1, n = n_ext[b] -- of which the
// last one is draft step 1 (Sec. 2.3 "Drafting phase": step k = 1 runs over the shifted sequence with
// the target's hidden states); the rows beyond n are padding: computed, never stored or published.
// Every later step carries one row per sequence at position L + n - 1 + step.
__device__ __forceinline__ void set_step_rows(Cta &c, int step) {
    c.M = (c.p->mode == 0 && step > 0) ? 1 : c.p->M;
    c.R = c.p->B * c.M;
}
__device__ __forceinline__ int seq_next(const Cta &c, int b) { return c.misc->next[b]; }
__device__ __forceinline__ int step_rows(const Cta &c, int b, int step) {      // rows of sequence b that count
    return c.p->mode == 1 ? c.p->M : (step == 0 ? seq_next(c, b) : 1);
}
// Row of the previous step whose output row r of this draft step continues (step >= 1).
__device__ __forceinline__ int src_row(const Cta &c, int r, int step) {
    return step == 1 ? r * c.p->M + seq_next(c, r) - 1 : r;
}
// Output index (sequence in a draft, row in a target step) of activation row r, -1 if it publishes nothing.
__device__ __forceinline__ int out_row(const Cta &c, int r, int step) {
    if (c.p->mode == 1 || step > 0) return r;
    const int b = r / c.p->M;
    return (r - b * c.p->M == seq_next(c, b) - 1) ? b : -1;
}

// ---- phase geometry ----------------------------------------------------------------------
// rows x K of the phase's matrix, tile height, this CTA's row range, and how K is cut into ring stages:
// into segments of seglen (the projection has two, one per input vector; every other phase one) and each
// segment into nks_seg stages of kc = KC elements (the last one shorter).
struct Geom { int rows, K, cap, nks, v0, v1, kc, rs, seglen, nks_seg; };
struct StageK { int koff, klen; };
__device__ __forceinline__ StageK stage_k(const Geom &g, int ks) {
    const int seg = ks / g.nks_seg, j = ks - seg * g.nks_seg;
    StageK s;
    s.koff = seg * g.seglen + j * g.kc;
    s.klen = min(g.kc, g.seglen - j * g.kc);
    return s;
}

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
    g.v0 = (int)(((long long)c.cta * g.rows) / c.grid);
    g.v1 = (int)(((long long)(c.cta + 1) * g.rows) / c.grid);
    g.kc = p.KC;
    g.rs = g.kc * 2;
    g.seglen = (kind == PROJ) ? p.d : g.K;
    g.nks_seg = (g.seglen + g.kc - 1) / g.kc;
    g.nks = ((kind == PROJ) ? 2 : 1) * g.nks_seg;
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
// The producer warps copy a stage with 16-byte cp.async instructions: warp `pw` takes tile rows
// pw, pw + 4, pw + 8, ...; its 32 lanes cover 512 contiguous bytes of a row per instruction.
// Each thread then posts an asynchronous arrival on the stage's `full` barrier that fires when its
// own copies have landed. The copies of a stage are issued from fully unrolled code with one
// address register pair per instruction: a cp.async reads its address operands only when it
// leaves the memory-instruction queue, so reusing an address register for the next copy would
// stall the warp on every instruction (measured: 4.2 instead of 7.0 TB/s). Row pointers of the
// next tile are computed one tile ahead so the subset-id lookup of the output head is off the
// issue path.
constexpr int kRowsPerProducer = kTileRows / kProducerWarps;   // 8

// Row pointers of a tile for one producer warp: lane j computes the pointer of tile row j (one
// subset-id lookup per lane, all in parallel), the warp exchanges them through its own line of a
// small shared-memory table and every lane keeps the eight rows its warp copies in registers.
// (No shuffles here or in the issue path: they would queue behind the cp.async traffic.)
__device__ __forceinline__ void tile_ptrs(Cta &c, int kind, const LayerPtrs &L, int vr0, int nv, int pw,
                                          const unsigned char *(&out)[kRowsPerProducer]) {
    unsigned long long *tbl = c.misc->rowptr[pw];
    __syncwarp();
    tbl[c.lane] = reinterpret_cast<unsigned long long>(tile_row_ptr(c, kind, L, vr0, nv, c.lane));
    __syncwarp();
#pragma unroll
    for (int i = 0; i < kRowsPerProducer; ++i) out[i] = reinterpret_cast<const unsigned char *>(tbl[pw + i * kProducerWarps]);
}

// Stage layout with tensor-memory staging (TM): the stage is the image of its tensor-memory slot, 128 lane rows x
// 256 bytes, stored as two 16 KB tiles of 128-byte rows with the 128-byte swizzle the tcgen05 descriptors describe
// (16-byte piece c of lane row L at c ^ (L & 7)). Lane row 32*wi + 4*g + t belongs to thread (g, t) of the consumer
// warps wi and wi + 4 and holds, in fragment order, the sixteen 16-byte pieces that thread multiplies: piece
// 4*j + rb = weight row g + 8*rb, k elements [32*ch + 8*t, +8) with ch = 8*(j >> 1) + 2*wi + (j & 1). A producer
// instruction still copies 512 contiguous bytes of one weight row; the eight lanes of a quarter-warp land in eight
// different 16-byte bank groups.
template <bool TM>
__device__ __forceinline__ void produce_phase(Cta &c, int kind, const LayerPtrs &L) {
    const MegaParams &p = *c.p;
    const Geom g = geom(c, kind);
    const int pw = c.warp - kConsumerWarps;
    const unsigned char *cur[kRowsPerProducer], *nxt[kRowsPerProducer];
#pragma unroll
    for (int i = 0; i < kRowsPerProducer; ++i) nxt[i] = nullptr;
    uint32_t toff[kRowsPerProducer];
    if (TM) {
        const int t = c.lane & 3, jlow = (c.lane >> 2) & 1, wq = c.lane >> 3;
#pragma unroll
        for (int i = 0; i < kRowsPerProducer; ++i) {
            const int gr = pw + 4 * (i & 1), rb = i >> 1;            // tile row pw + 4*i = gr + 8*rb
            const int lrow = 32 * wq + 4 * gr + t;
            toff[i] = (uint32_t)(lrow * 128 + ((4 * (jlow ^ (pw & 1)) + (rb ^ t)) << 4));
        }
    }
    // rows are stored without padding; in odd rows the two 64-byte halves of every 128 bytes are
    // swapped, which keeps the consumers' 128-bit fragment loads free of bank conflicts. All rows of a
    // producer warp have the parity of pw.
    const uint32_t lane16 = (uint32_t)c.lane * 16u;
    const uint32_t lane16d = (uint32_t)(c.lane ^ ((pw & 1) << 2)) * 16u;
    const uint32_t rs = (uint32_t)g.rs;
    // weights are read once per step: they enter L2 marked evict-first, so that the stream does not push out what
    // the step keeps re-reading (activation vectors, partial sums, barrier words and the kernel's own code)
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    // the loop starts one tile early: iteration t fetches the pointers of tile t + 1
#pragma unroll 1
    for (int vr0 = g.v0 - g.cap; vr0 < g.v1; vr0 += g.cap) {
#pragma unroll
        for (int i = 0; i < kRowsPerProducer; ++i) cur[i] = nxt[i];
        if (vr0 + g.cap < g.v1) tile_ptrs(c, kind, L, vr0 + g.cap, min(g.cap, g.v1 - vr0 - g.cap), pw, nxt);
        if (vr0 < g.v0) continue;
#pragma unroll 1
        for (int ks = 0; ks < g.nks; ++ks) {
            const int slot = c.slot;
            const uint32_t parity = c.parity;
            bool ok = true;
            PROF_T0();
            if (c.lane == 0) ok = wait_bar(c, &c.misc->empty[slot], parity ^ 1u);
            ok = __shfl_sync(0xffffffffu, ok, 0);
            PROF_ACC(c, 2, pw == 0 && c.lane == 0);
            if (!ok) return;   // abort: stop issuing copies
            const StageK sk = stage_k(g, ks);
            const int klen = sk.klen;
            const uint32_t dst0 = smem_u32(c.ring + (size_t)slot * p.stage_bytes) + (uint32_t)pw * rs + lane16d;
            const size_t koff = (size_t)sk.koff * 2 + lane16;
            if (TM) {
                // every stage is 512 wide here: the second piece of a row (k elements 256..511) belongs to the second
                // 16 KB tile of the stage
                const uint32_t sbase = smem_u32(c.ring + (size_t)slot * p.stage_bytes);
                uint32_t d[kRowsPerProducer];
                const unsigned char *q[kRowsPerProducer];
#pragma unroll
                for (int i = 0; i < kRowsPerProducer; ++i) {
                    q[i] = cur[i] + koff;
                    d[i] = sbase + toff[i];
                }
#pragma unroll
                for (int i = 0; i < kRowsPerProducer; ++i) {
                    if (cur[i] != nullptr) {
                        asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2;" ::"r"(d[i]), "l"(q[i]), "l"(pol) : "memory");
                        asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0+16384], [%1+512], 16, %2;" ::"r"(d[i]), "l"(q[i]), "l"(pol) : "memory");
                    }
                }
            } else if (klen == 512) {
                // the stage width of the large shapes, from fully unrolled code: two 512-byte pieces per row, one
                // instruction per piece and lane, all with their own address registers (the piece offsets are
                // immediates). The loop is this tight on purpose: a predicate or branch per instruction costs
                // several per cent of the stream rate (measured: -5 % with three predicated pieces per row).
                uint32_t d[kRowsPerProducer];
                const unsigned char *q[kRowsPerProducer];
#pragma unroll
                for (int i = 0; i < kRowsPerProducer; ++i) {
                    q[i] = cur[i] + koff;
                    d[i] = dst0 + (uint32_t)(i * kProducerWarps) * rs;
                }
#pragma unroll
                for (int i = 0; i < kRowsPerProducer; ++i) {
                    if (cur[i] != nullptr) {
                        asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2;" ::"r"(d[i]), "l"(q[i]), "l"(pol) : "memory");
                        asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0+512], [%1+512], 16, %2;" ::"r"(d[i]), "l"(q[i]), "l"(pol) : "memory");
                    }
                }
            } else {
                // other stage widths (small or odd geometries): generic loop; a row's tail up to the next
                // multiple of 32 elements is filled with zeros (source size 0: nothing is read)
                const int n16 = klen >> 3, n16z = ((klen + 31) & ~31) >> 3;
#pragma unroll
                for (int i = 0; i < kRowsPerProducer; ++i) {
                    const unsigned char *rp = cur[i];
                    if (rp != nullptr) {
                        for (int u = c.lane; u < n16z; u += 32) {
                            const uint32_t nbytes = u < n16 ? 16u : 0u;
                            asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2, %3;" ::"r"(dst0 + (uint32_t)(i * kProducerWarps) * rs + (uint32_t)(u - c.lane) * 16u),
                                         "l"(u < n16 ? rp + koff + (size_t)(u - c.lane) * 16 : rp), "r"(nbytes), "l"(pol) : "memory");
                        }
                    }
                }
            }
            cp_async_arrive(&c.misc->full[slot]);
            PROF_ACC(c, 3, pw == 0 && c.lane == 0);
            next_stage(c);
        }
    }
}

// ---- consumer: matrix-vector core --------------------------------------------------------------
struct ActSrc {          // where the B operand (activations) is read from
    const bf16_t *hi, *lo;   // shared-memory staging area, or global scratch written by other CTAs
    int stride;              // elements per activation row
    bool in_smem;
};

// Per-thread accumulation of v^2 per activation row across the tiles of a phase, reduced over
// the CTA's rows at phase end and written to this CTA's line of a partial table.
struct SqAcc {
    float a, b;
};

// What the per-row epilogue of a matrix phase needs besides the value.
struct EpiCtx {
    SqAcc sq;
    unsigned long long best;     // running (logit, id) maximum of this thread (output head)
    const LayerPtrs *L;
    const bf16_t *gnext;         // gain applied after the down projection (next layer's or the final norm's)
    int step;
    bool to_next_layer;          // target mode, not the last layer: the result feeds the next layer
};

__device__ __forceinline__ void store_split(bf16_t *hi, bf16_t *lo, size_t idx, float v) {
    uint16_t h, l;
    split_bf16(v, h, l);
    hi[idx] = h;
    lo[idx] = l;
}

// Operands of the epilogue that do not depend on the dot product (residual value, norm gains, the
// token id of a head row): loaded when the tile starts, so their latency hides behind the stream.
struct EpiPre { float resid, g0, g1; int id; };
__device__ __forceinline__ EpiPre epi_prefetch(const Cta &c, int kind, const EpiCtx &x, int row, int col, bool valid) {
    const MegaParams &p = *c.p;
    EpiPre e;
    e.resid = 0.f; e.g0 = 0.f; e.g1 = 0.f; e.id = row;
    if (!valid) return e;
    switch (kind) {
        case PROJ: e.g0 = bf16bits_f32(x.L->g_in[row]); break;
        case OPROJ:
            e.resid = ldcg_f32(p.s.x0 + (size_t)col * p.d + row);
            e.g0 = bf16bits_f32(x.L->g_post[row]);
            break;
        case DOWN:
            e.resid = ldcg_f32(p.s.x1 + (size_t)col * p.d + row);
            e.g0 = bf16bits_f32(x.gnext[row]);
            if (p.mode == 0) e.g1 = bf16bits_f32(p.g_hnorm[row]);
            break;
        case HEAD:
            if (p.ids) e.id = p.ids[row];
            break;
        default: break;
    }
    return e;
}

// Epilogue of one (virtual row, activation row): what the phase does with the finished dot product.
__device__ __forceinline__ void epilogue(const Cta &c, int kind, EpiCtx &x, const EpiPre &pre, int row, int col, float v, float up) {
    const MegaParams &p = *c.p;
    const Scratch &s = p.s;
    switch (kind) {
        case PROJ: {
            s.x0[(size_t)col * p.d + row] = v;
            store_split(s.actD_hi, s.actD_lo, (size_t)col * p.dp + row, v * pre.g0);
            x.sq.a += v * v;
            break;
        }
        case QKV:
            s.qkv[(size_t)col * (p.qdim + 2 * p.kvdim) + row] = v * c.misc->scale0[col];
            break;
        case OPROJ: {
            float r = pre.resid + v;
            s.x1[(size_t)col * p.d + row] = r;
            store_split(s.actP_hi, s.actP_lo, (size_t)col * p.dp + row, r * pre.g0);
            x.sq.a += r * r;
            break;
        }
        case GATEUP: {
            float sc = c.misc->scale0[col];
            float gt = v * sc, u = up * sc;
            store_split(s.actF_hi, s.actF_lo, (size_t)col * p.Fp + row, gt / (1.f + expf(-gt)) * u);
            break;
        }
        case DOWN: {
            float r = pre.resid + v;
            float y = r * pre.g0;
            x.sq.a += r * r;
            if (x.to_next_layer) {
                s.x0[(size_t)col * p.d + row] = r;
                store_split(s.actD_hi, s.actD_lo, (size_t)col * p.dp + row, y);
            } else {
                store_split(s.actH_hi, s.actH_lo, (size_t)col * p.dp + row, y);
                if (p.mode == 0) {
                    store_split(s.actR_hi, s.actR_lo, (size_t)col * p.dp + row, y * pre.g1);
                    x.sq.b += y * y;
                }
            }
            break;
        }
        default: {   // HEAD
            int id = pre.id;
            if ((unsigned)id >= (unsigned)p.V) id = 0;
            float lv = v;
            if (p.mode == 1) {
                // target: the decision is taken on the bf16 logits that cross the boundary
                uint16_t lb = f32_bf16bits(v * c.misc->scale0[col]);
                if (p.out_logits_bf16) p.out_logits_bf16[(size_t)col * p.V + row] = lb;
                lv = bf16bits_f32(lb);
            } else if (p.out_logits_f32) {
                const int orow = c.misc->outrow[col];
                if (orow >= 0) p.out_logits_f32[((size_t)orow * p.K + x.step) * p.N + row] = v * c.misc->scale0[col];
            }
            unsigned long long key = argmax_key(lv, (uint32_t)id);
            x.best = key > x.best ? key : x.best;
            break;
        }
    }
}

// One chunk (32 weight rows x 32 k) of a stage: four MMAs per activation set.
struct Frag { uint4 u0, v0, u1, v1; };
__device__ __forceinline__ void mma_chunk(float (&acc)[2][2][4], const Frag &f, const uint4 &b) {
    mma_bf16(acc[0][0], f.u0.x, f.v0.x, f.u0.y, f.v0.y, b.x, b.y);
    mma_bf16(acc[1][0], f.u1.x, f.v1.x, f.u1.y, f.v1.y, b.x, b.y);
    mma_bf16(acc[0][1], f.u0.z, f.v0.z, f.u0.w, f.v0.w, b.z, b.w);
    mma_bf16(acc[1][1], f.u1.z, f.v1.z, f.u1.w, f.v1.w, b.z, b.w);
}
__device__ __forceinline__ Frag load_frag(uint32_t a, uint32_t rs) {
    Frag f;
    f.u0 = lds128_u32(a);
    f.v0 = lds128_u32(a + 8 * rs);
    f.u1 = lds128_u32(a + 16 * rs);
    f.v1 = lds128_u32(a + 24 * rs);
    return f;
}

// Moves the running sums of the first input segment aside (the projection scales its two input
// segments with different RMSNorm factors).
template <bool two_sets>
__device__ __forceinline__ void park(float (&acc)[2][2][4], float (&acd)[2][2][4], float (&acc0)[2][4], float (&acd0)[2][4]) {
#pragma unroll
    for (int i = 0; i < 2; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            acc0[i][j] = acc[i][0][j] + acc[i][1][j];
            acc[i][0][j] = acc[i][1][j] = 0.f;
            if (two_sets) {
                acd0[i][j] = acd[i][0][j] + acd[i][1][j];
                acd[i][0][j] = acd[i][1][j] = 0.f;
            }
        }
}

// Runs all tiles of one matrix phase for this CTA and calls epilogue() once per valid (virtual
// row, activation row), by exactly one thread. The kernel has a single call site per template
// argument, so the streaming loop exists once in the instruction stream: this kernel is far
// larger than the instruction cache and anything not in a loop is fetched from L2.
//
// MMA mapping: A = 16 weight rows x 16 k, B column 2r holds the hi part and column 2r+1 the lo
// part of activation row r, so one MMA covers four activation rows exactly (the two columns are
// added at the end); rows 4..7 use a second set of accumulators. The two halves of the consumer
// warps (warps 0-3 / 4-7) take alternate stages, so each warp does four chunks per barrier wait
// and two stages are in work at once.
//
// With tensor-memory staging (TM) the stage has the layout of a tensor-memory slot (see the producer): the thread's
// sixteen 16-byte pieces, already in fragment order, come by two tcgen05.ld of 32 registers each (the first eight
// stages of a phase) or by sixteen conflict-free 128-bit loads from the shared-memory stage (the rest), and the
// warp's four k chunks of a stage are 8*(j >> 1) + 2*wi + (j & 1), j = 0..3.
template <bool two_sets, bool TM>
__device__ __forceinline__ void consume_tiles(Cta &c, const int kind, const ActSrc &act, EpiCtx &ex) {
    const MegaParams &p = *c.p;
    const Geom geo = geom(c, kind);
    const int R = c.R;
    const int g = c.lane >> 2, t = c.lane & 3;
    const int grp = c.warp >> 2, wi = c.warp & 3;
    const int arow = g >> 1;
    const bf16_t *abase = (g & 1) ? act.lo : act.hi;
    const bool has0 = arow < R, has1 = two_sets && (arow + 4 < R);
    const size_t aoff0 = (size_t)arow * act.stride + t * 8, aoff1 = (size_t)(arow + 4) * act.stride + t * 8;
    const uint32_t rs = (uint32_t)geo.rs;
    const uint4 zero = make_uint4(0, 0, 0, 0);
    for (int vr0 = geo.v0; vr0 < geo.v1; vr0 += geo.cap) {
        const int nv = min(geo.cap, geo.v1 - vr0);
        const int erow = c.tid >> 3, ecol = c.tid & 7;               // this thread's epilogue element
        const bool evalid = erow < ((kind == GATEUP) ? min(nv, 16) : nv) && ecol < R;
        const EpiPre pre = epi_prefetch(c, kind, ex, vr0 + erow, ecol, evalid);
        float acc[2][2][4], acd[2][2][4], acc0[2][4], acd0[2][4];
#pragma unroll
        for (int i = 0; i < 2; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                acc[i][0][j] = acc[i][1][j] = acd[i][0][j] = acd[i][1][j] = 0.f;
                acc0[i][j] = acd0[i][j] = 0.f;
            }
        // Activations read from global memory (the ffn-wide vector of the down projection is not staged whole in
        // shared memory). A warp needs 512 bytes of it per stage and activation row -- its four 32-element chunks,
        // hi and lo part -- and fetches them one owned stage ahead with ONE 16-byte cp.async per lane into a small
        // ring in the (otherwise unused) staging area, then reads its fragments from there: per-lane global loads
        // straight into the fragment registers were four load instructions per stage and warp, a third on top of the
        // producers' copies in the same load/store path, and held this phase a quarter below the others' stream rate.
        constexpr int kCpw = 4;                                       // chunks a warp has in a full stage: wi, wi + 4, wi + 8, wi + 12
        uint32_t xo[8];                                               // TM: where this lane's piece s of a 16 KB tile sits in its row
#pragma unroll
        for (int s8 = 0; s8 < 8; ++s8) xo[s8] = (uint32_t)(32 * wi + c.lane) * 128u + (((uint32_t)s8 ^ ((uint32_t)c.lane & 7u)) << 4);
        const bool gfast = !two_sets && !act.in_smem && 16 * R * 512 <= p.scratch_smem;      // the slice ring must fit the staging area
        // which half of the warps takes a stage depends only on the stage's index within the phase,
        // never on how many stages the CTA has seen before: the summation order of a row must not
        // depend on the batch or on earlier calls
        const int stage0 = ((vr0 - geo.v0) / geo.cap) * geo.nks;
        // slice ring: slot (stage index mod 4) x warp of the owning group x activation row x 512 bytes
        const uint32_t slice_base = smem_u32(c.scr) + (uint32_t)(wi * R) * 512u;
        auto slice_slot = [&](int sa) -> uint32_t { return slice_base + (uint32_t)((sa & 3) * 4 * R) * 512u; };
        auto slice_fetch = [&](int sa, const StageK &sk) {           // lane = (chunk j, hi/lo, 16-byte piece)
            const int j = c.lane >> 3, hl = (c.lane >> 2) & 1, tp = c.lane & 3;
            const int ch = TM ? 8 * (j >> 1) + 2 * wi + (j & 1) : wi + 4 * j;
            const bf16_t *src = (hl ? act.lo : act.hi) + (size_t)sk.koff + ch * 32 + tp * 8;
            const uint32_t dst = slice_slot(sa) + (uint32_t)c.lane * 16u;
#pragma unroll 1
            for (int r = 0; r < R; ++r)
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + (uint32_t)r * 512u), "l"(src + (size_t)r * act.stride) : "memory");
            asm volatile("cp.async.commit_group;" ::: "memory");
        };
        if (gfast) {
            const int ks0 = ((stage0 & 1) == grp) ? 0 : 1;          // first stage this warp owns
            if (ks0 < geo.nks) {
                const StageK s0 = stage_k(geo, ks0);
                if (s0.klen == 512) slice_fetch(stage0 + ks0, s0);
            }
        }
#pragma unroll 1
        for (int ks = 0; ks < geo.nks; ++ks) {
            if (kind == PROJ && ks == geo.nks_seg) {
                // the second input segment starts: every warp parks the sums of the first (whichever stages of it
                // the warp owned)
                park<two_sets>(acc, acd, acc0, acd0);
            }
            if (TM) {
                // the first kTmSlots stages of a phase come through tensor memory (they land while the consumers are still
                // busy with the previous phase's end), the rest is read from the shared-memory stage directly
                const bool via_tmem = stage0 + ks < kTmSlots;
                if (((stage0 + ks) & 1) == grp) {
                    const StageK sk = stage_k(geo, ks);
                    uint32_t w0[32], w1[32];
                    const int ts = c.tslot, slot = c.slot;
                    PROF_T0();
                    if (via_tmem) {
                        wait_bar(c, &c.misc->tfull[ts], c.tparity);
                        PROF_ACC(c, 0, c.tid == 0);
                        tc_fence_after_sync();
                        const uint32_t ta = c.tmem + ((uint32_t)(32 * wi) << 16) + (uint32_t)(ts * kTmSlotCols);
                        tmem_ld32_issue(ta, w0);
                        tmem_ld32_issue(ta + 32, w1);
                    } else {
                        wait_bar(c, &c.misc->full[slot], c.parity);
                        PROF_ACC(c, 0, c.tid == 0);
                    }
                    uint4 bq[kCpw];
                    if (act.in_smem) {
                        const uint32_t ab = smem_u32(abase + aoff0 + (size_t)sk.koff);
#pragma unroll
                        for (int j = 0; j < kCpw; ++j) bq[j] = has0 ? lds128_u32(ab + (8 * (j >> 1) + 2 * wi + (j & 1)) * 64) : zero;
                    } else {
                        if (ks + 2 < geo.nks) slice_fetch(stage0 + ks + 2, stage_k(geo, ks + 2));
                        if (ks + 2 < geo.nks) asm volatile("cp.async.wait_group 1;" ::: "memory");
                        else asm volatile("cp.async.wait_group 0;" ::: "memory");
                        __syncwarp();
                        const uint32_t sl = slice_slot(stage0 + ks) + (uint32_t)(arow * 512 + ((g & 1) * 4 + t) * 16);
#pragma unroll
                        for (int j = 0; j < kCpw; ++j) bq[j] = has0 ? lds128_u32(sl + j * 128) : zero;
                    }
                    if (via_tmem) {
                        tmem_ld_wait();
                        tc_fence_before_sync();
                        __syncwarp();
                        if (c.lane == 0) mbar_arrive(&c.misc->tempty[ts]);       // the slot's data is in registers
                    } else {
                        // the stage has the slot's layout: lane row 32*wi + lane, piece s of it at (s & 7) ^ (lane & 7) in tile s >> 3
                        const uint32_t lb = smem_u32(c.ring + (size_t)slot * p.stage_bytes);
#pragma unroll
                        for (int s8 = 0; s8 < 8; ++s8) {
                            const uint4 a = lds128_u32(lb + xo[s8]);
                            const uint4 b = lds128_u32(lb + xo[s8] + 16384u);
                            w0[4 * s8] = a.x; w0[4 * s8 + 1] = a.y; w0[4 * s8 + 2] = a.z; w0[4 * s8 + 3] = a.w;
                            w1[4 * s8] = b.x; w1[4 * s8 + 1] = b.y; w1[4 * s8 + 2] = b.z; w1[4 * s8 + 3] = b.w;
                        }
                    }
#pragma unroll
                    for (int j = 0; j < 2; ++j) {
                        Frag f;
                        f.u0 = make_uint4(w0[16 * j + 0], w0[16 * j + 1], w0[16 * j + 2], w0[16 * j + 3]);
                        f.v0 = make_uint4(w0[16 * j + 4], w0[16 * j + 5], w0[16 * j + 6], w0[16 * j + 7]);
                        f.u1 = make_uint4(w0[16 * j + 8], w0[16 * j + 9], w0[16 * j + 10], w0[16 * j + 11]);
                        f.v1 = make_uint4(w0[16 * j + 12], w0[16 * j + 13], w0[16 * j + 14], w0[16 * j + 15]);
                        mma_chunk(acc, f, bq[j]);
                    }
#pragma unroll
                    for (int j = 0; j < 2; ++j) {
                        Frag f;
                        f.u0 = make_uint4(w1[16 * j + 0], w1[16 * j + 1], w1[16 * j + 2], w1[16 * j + 3]);
                        f.v0 = make_uint4(w1[16 * j + 4], w1[16 * j + 5], w1[16 * j + 6], w1[16 * j + 7]);
                        f.u1 = make_uint4(w1[16 * j + 8], w1[16 * j + 9], w1[16 * j + 10], w1[16 * j + 11]);
                        f.v1 = make_uint4(w1[16 * j + 12], w1[16 * j + 13], w1[16 * j + 14], w1[16 * j + 15]);
                        mma_chunk(acc, f, bq[2 + j]);
                    }
                    if (!via_tmem) {
                        __syncwarp();
                        if (c.lane == 0) {
                            // counted before the arrival, so that the count of a use is never written after the slot's next use
                            if (wi == 0) { volatile uint32_t *ud = &c.misc->use_done[slot]; *ud = *ud + 1; }   // see the mover
                            mbar_arrive(&c.misc->empty[slot]);
                        }
                    }
                    PROF_ACC(c, 1, c.tid == 0);
                }
                if (via_tmem) next_tslot(c);
            } else if (((stage0 + ks) & 1) == grp) {
                const int slot = c.slot;
                const uint32_t parity = c.parity;
                PROF_T0();
                wait_bar(c, &c.misc->full[slot], parity);
                PROF_ACC(c, 0, c.tid == 0);

                const StageK sk = stage_k(geo, ks);
                const int nchunk = (sk.klen + 31) >> 5;
                const uint32_t sb = smem_u32(c.ring + (size_t)slot * p.stage_bytes) + t * 16 + g * rs;
                const int par = g & 1;                    // odd rows: 64-byte halves swapped
                const size_t kbase = (size_t)sk.koff;
                if (!two_sets && nchunk == 16 && (act.in_smem || gfast)) {
                    // the stage width of the large shapes with at most four activation rows: this warp's chunks
                    // wi, wi + 4, wi + 8, wi + 12 in two batches of two, all loads of a batch issued before its MMAs,
                    // nothing predicated (see the producer: this loop sets the stream rate)
                    uint4 bq[kCpw];
                    if (act.in_smem) {
                        const uint32_t ab = smem_u32(abase + aoff0 + kbase);
#pragma unroll
                        for (int j = 0; j < kCpw; ++j) bq[j] = has0 ? lds128_u32(ab + (wi + 4 * j) * 64) : zero;
                    } else {
                        // request the slices of the next owned stage, then wait for this stage's (requested one owned
                        // stage ago) and read the fragments from the slice ring
                        bool more = false;
                        if (ks + 2 < geo.nks) {
                            const StageK s2 = stage_k(geo, ks + 2);
                            if (s2.klen == 512) { slice_fetch(stage0 + ks + 2, s2); more = true; }   // (a shorter last stage is read directly by the loop below)
                        }
                        if (more) asm volatile("cp.async.wait_group 1;" ::: "memory");
                        else asm volatile("cp.async.wait_group 0;" ::: "memory");
                        __syncwarp();
                        const uint32_t sl = slice_slot(stage0 + ks) + (uint32_t)(arow * 512 + ((g & 1) * 4 + t) * 16);
#pragma unroll
                        for (int j = 0; j < kCpw; ++j) bq[j] = has0 ? lds128_u32(sl + j * 128) : zero;
                    }
#pragma unroll
                    for (int b2 = 0; b2 < 2; ++b2) {
                        const int ch = wi + 8 * b2;
                        Frag f0 = load_frag(sb + (ch ^ par) * 64, rs);
                        Frag f1 = load_frag(sb + ((ch + 4) ^ par) * 64, rs);
                        mma_chunk(acc, f0, bq[2 * b2]);
                        mma_chunk(acc, f1, bq[2 * b2 + 1]);
                    }
                } else {
#pragma unroll 1
                    for (int ch = wi; ch < nchunk; ch += 4) {
                        Frag f0 = load_frag(sb + (ch ^ par) * 64, rs);
                        uint4 b0 = zero, d0 = zero;
                        if (has0) b0 = act.in_smem ? lds128(abase + aoff0 + kbase + ch * 32) : ldcg128(abase + aoff0 + kbase + ch * 32);
                        if (has1) d0 = act.in_smem ? lds128(abase + aoff1 + kbase + ch * 32) : ldcg128(abase + aoff1 + kbase + ch * 32);
                        mma_chunk(acc, f0, b0);
                        if (two_sets) mma_chunk(acd, f0, d0);
                    }
                }
                __syncwarp();
                if (c.lane == 0) mbar_arrive(&c.misc->empty[slot]);
                PROF_ACC(c, 1, c.tid == 0);
            }
            next_stage(c);
        }
        // cross-warp reduction in a fixed order
        PROF_T0();
        float *red = c.red + (size_t)c.redbuf * kConsumerWarps * kTileRows * R + (size_t)c.warp * kTileRows * R;
#pragma unroll
        for (int i = 0; i < 2; ++i) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int row = i * 16 + g + h * 8;
                // activation row t (set 0) / t + 4 (set 1): hi column + lo column
                if (t < R) {
                    float v = (acc[i][0][2 * h] + acc[i][0][2 * h + 1]) + (acc[i][1][2 * h] + acc[i][1][2 * h + 1]);
                    if (kind == PROJ) v = (acc0[i][2 * h] + acc0[i][2 * h + 1]) * c.misc->scale0[t] + v * c.misc->scale1[t];
                    red[row * R + t] = v;
                }
                if (two_sets && t + 4 < R) {
                    float v = (acd[i][0][2 * h] + acd[i][0][2 * h + 1]) + (acd[i][1][2 * h] + acd[i][1][2 * h + 1]);
                    if (kind == PROJ) v = (acd0[i][2 * h] + acd0[i][2 * h + 1]) * c.misc->scale0[t + 4] + v * c.misc->scale1[t + 4];
                    red[row * R + t + 4] = v;
                }
            }
        }
        bar_sync(1, kConsumerThreads);
        {
            const float *rb = c.red + (size_t)c.redbuf * kConsumerWarps * kTileRows * R;
            const int row = erow, col = ecol;
            if (evalid) {
                float a = 0.f, b = 0.f;
#pragma unroll
                for (int w = 0; w < kConsumerWarps; ++w) a += rb[(size_t)w * kTileRows * R + row * R + col];
                if (kind == GATEUP) {
#pragma unroll
                    for (int w = 0; w < kConsumerWarps; ++w) b += rb[(size_t)w * kTileRows * R + (row + 16) * R + col];
                }
                epilogue(c, kind, ex, pre, vr0 + row, col, a, b);
            }
        }
        c.redbuf ^= 1;
        PROF_ACC(c, 4, c.tid == 0);
    }
}

// Sum over CTAs of a per-CTA partial-sums-of-squares table [grid][8], for activation row `col`,
// by one full warp in a fixed reduction tree (reproducible). Split in two so that the loads can be
// issued before other work and consumed after it (grid <= 32 * kPartialRegs).
constexpr int kPartialRegs = 5;
__device__ __forceinline__ void load_partials(const Cta &c, const float *tbl, int col, float (&v)[kPartialRegs]) {
#pragma unroll
    for (int q = 0; q < kPartialRegs; ++q) {
        int i = c.lane + 32 * q;
        v[q] = (i < c.grid) ? ldcg_f32(tbl + (size_t)i * kMaxRows + col) : 0.f;
    }
}
__device__ __forceinline__ float reduce_partials(const float (&v)[kPartialRegs]) {
    float s = 0.f;
#pragma unroll
    for (int q = 0; q < kPartialRegs; ++q) s += v[q];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    return s;
}

// Copies R rows of a hi/lo activation pair from global scratch into the shared staging area.
// `len` elements per row (multiple of 8), rows `stride_s` apart in shared memory, starting at
// element offset `dst_off`.
// With remap_step >= 1 row r is read from global row src_row(r, remap_step): the projection of draft step 1
// continues each sequence's last extend row.
template <int U>
__device__ __forceinline__ void stage_hilo_impl(const Cta &c, const bf16_t *ghi, const bf16_t *glo, int gstride, int len, bf16_t *shi,
                                                bf16_t *slo, int sstride, int dst_off, int remap_step) {
    const int per_row = len / 8;
    const int total = c.R * per_row;
    // U units per thread and round: 2 U loads in flight before the first store waits
#pragma unroll 1
    for (int i0 = c.tid; i0 < total; i0 += U * kConsumerThreads) {
        uint4 a[U], b[U];
#pragma unroll
        for (int q = 0; q < U; ++q) {
            int i = min(i0 + q * kConsumerThreads, total - 1);
            int r = i / per_row, k = (i - r * per_row) * 8;
            const int rs = remap_step > 0 ? src_row(c, r, remap_step) : r;
            a[q] = ldcg128(ghi + (size_t)rs * gstride + k);
            b[q] = ldcg128(glo + (size_t)rs * gstride + k);
        }
#pragma unroll
        for (int q = 0; q < U; ++q) {
            int i = i0 + q * kConsumerThreads;
            if (i < total) {
                int r = i / per_row, k = (i - r * per_row) * 8;
                *reinterpret_cast<uint4 *>(shi + (size_t)r * sstride + dst_off + k) = a[q];
                *reinterpret_cast<uint4 *>(slo + (size_t)r * sstride + dst_off + k) = b[q];
            }
        }
    }
}
__device__ __forceinline__ void stage_hilo(const Cta &c, const bf16_t *ghi, const bf16_t *glo, int gstride, int len, bf16_t *shi,
                                           bf16_t *slo, int sstride, int dst_off, int remap_step = 0) {
    // several rows: twice as many loads per round, so that the copy stays at one or two L2 round trips
    if (c.R * (len / 8) > 4 * kConsumerThreads) stage_hilo_impl<8>(c, ghi, glo, gstride, len, shi, slo, sstride, dst_off, remap_step);
    else stage_hilo_impl<4>(c, ghi, glo, gstride, len, shi, slo, sstride, dst_off, remap_step);
}

__device__ __forceinline__ void flush_sq(const Cta &c, const SqAcc &q, float *tblA, float *tblB) {
    // thread (row slot = tid>>3, col = tid&7): the four row slots of a warp are added by shuffle, the
    // eight warps in ascending order by the first eight threads
    float a = q.a, b = q.b;
    a += __shfl_xor_sync(0xffffffffu, a, 8);
    a += __shfl_xor_sync(0xffffffffu, a, 16);
    b += __shfl_xor_sync(0xffffffffu, b, 8);
    b += __shfl_xor_sync(0xffffffffu, b, 16);
    if (c.lane < kMaxRows) {
        c.misc->colred[c.warp][c.lane] = a;
        c.misc->colred[kConsumerWarps + c.warp][c.lane] = b;
    }
    bar_sync(1, kConsumerThreads);
    if (c.tid < kMaxRows) {
        float sa = 0.f, sb = 0.f;
#pragma unroll
        for (int w = 0; w < kConsumerWarps; ++w) {
            sa += c.misc->colred[w][c.tid];
            sb += c.misc->colred[kConsumerWarps + w][c.tid];
        }
        if (tblA) tblA[(size_t)c.cta * kMaxRows + c.tid] = sa;
        if (tblB) tblB[(size_t)c.cta * kMaxRows + c.tid] = sb;
    }
}

// ---- attention phase -------------------------------------------------------------------------
// Rows r = b*M + m sit at position step_base(b) + m (see "rows of a step"). The context of a sequence is cut
// into fixed 64-token chunks from position 0; a work item is (sequence, KV head, chunk) and items
// are dealt round-robin over the CTAs. A row's result therefore depends on its own position only.
//
// The producers stream the committed part of a chunk (positions below seq_lens[b], which nothing
// in this launch writes) through the same ring as the weights: K rows at token*dh, V rows after
// the 64 K rows. The consumers add the positions this launch produced (earlier draft steps from
// the pages, this call's rows from the QKV scratch, rotated and rounded to bf16 exactly as they
// are stored) into the same stage buffer and then work from shared memory only.
// Scratch: qs[M*Gq][dh] rotated, pre-scaled queries of one KV head, then the per-warp partials (o, m, l) of the
// working warp groups.

// One chunk of one KV head on the tensor cores, for every row of the call. K and V stay in the stage (16-byte piece w
// of token row t stored at piece w ^ (t & 7), so that ldmatrix reads without bank conflicts). The consumer warps
// form two groups of four; group g takes the rows m = g, g + 2, ..., so a row's arithmetic does not depend on how
// many rows the call carries. Within a group warp wi owns tokens 16*wi .. 16*wi+15 of the chunk. Scores: the query
// heads are the A operand (rows 0-7 the bf16 high parts of up to eight heads, rows 8-15 the low parts: products with
// the bf16 keys are exact), K fragments by ldmatrix; softmax statistics per warp; P*V with the probabilities split
// the same way, V fragments by transposing ldmatrix. The four warps' (o, m, l) are merged in warp order, then the
// chunks in ascending order by the merge phase.
template <int DH>
__device__ __forceinline__ void attn_rows_mma(Cta &c, const bf16_t *sk, const bf16_t *sv, const float *qs, float *part,
                                              int b, int kvh, int chunk, int base, int max_tokens, int rows) {
    const MegaParams &p = *c.p;
    constexpr int wstride = DH + 2;
    const int Gq = p.Hq / p.Hkv, M = c.M;
    const int c0 = chunk * kAttnChunk;
    const int grp = c.warp >> 2, wi = c.warp & 3;
    const int hrow = c.lane >> 2, kq = (c.lane & 3) * 2;
    const int tw = wi * 16;                                  // first token (within the chunk) of this warp
    float *wp = part + (size_t)grp * (4 * 8 * wstride + 64);  // this group's [4 warps][8 heads][DH + 2], then 32 weights, 8 x (m, l)
    float *fw = wp + 4 * 8 * wstride;
    const uint32_t sk_u = smem_u32(sk), sv_u = smem_u32(sv);
    // ldmatrix row addresses (see the batched attention kernel): K: matrices (tokens 0-7, dims 0-7), (0-7, 8-15),
    // (8-15, 0-7), (8-15, 8-15) of a 16-dim slice; V (transposed): (tokens 0-7, dims 0-7), (8-15, 0-7), (0-7, 8-15), (8-15, 8-15)
    const int ktok = tw + (c.lane & 7) + ((c.lane >> 4) << 3), kpc = (c.lane >> 3) & 1;
    const int vtok = tw + (c.lane & 7) + (((c.lane >> 3) & 1) << 3), vpc = c.lane >> 4;
    const uint32_t krow = sk_u + (uint32_t)ktok * (DH * 2), vrow = sv_u + (uint32_t)vtok * (DH * 2);
    const uint32_t ksw = (uint32_t)(ktok & 7), vsw = (uint32_t)(vtok & 7);
#pragma unroll 1
    for (int m = grp; m < M; m += 2) {
        const int npos = min(base + min(m, rows - 1), max_tokens - 1);   // last visible position of this row
#pragma unroll 1
        for (int h0 = 0; h0 < Gq; h0 += 8) {                             // eight query heads per pass
            const int nh = min(8, Gq - h0);
            // query fragments from the fp32 vectors: hi parts in rows 0-7, lo parts in rows 8-15
            uint32_t qa[DH / 16][4];
            {
                const float *qh = qs + ((size_t)(m * Gq + h0 + hrow)) * DH;
#pragma unroll
                for (int ks = 0; ks < DH / 16; ++ks) {
                    float2 x0 = make_float2(0.f, 0.f), x1 = make_float2(0.f, 0.f);
                    if (hrow < nh) {
                        x0 = *reinterpret_cast<const float2 *>(qh + ks * 16 + kq);
                        x1 = *reinterpret_cast<const float2 *>(qh + ks * 16 + kq + 8);
                    }
                    uint16_t h0a, l0a, h0b, l0b, h1a, l1a, h1b, l1b;
                    split_bf16(x0.x, h0a, l0a); split_bf16(x0.y, h0b, l0b);
                    split_bf16(x1.x, h1a, l1a); split_bf16(x1.y, h1b, l1b);
                    qa[ks][0] = (uint32_t)h0a | ((uint32_t)h0b << 16);
                    qa[ks][1] = (uint32_t)l0a | ((uint32_t)l0b << 16);
                    qa[ks][2] = (uint32_t)h1a | ((uint32_t)h1b << 16);
                    qa[ks][3] = (uint32_t)l1a | ((uint32_t)l1b << 16);
                }
            }
            // scores of this warp's 16 tokens (two n-tiles of 8)
            float s[2][4];
            s[0][0] = s[0][1] = s[0][2] = s[0][3] = 0.f;
            s[1][0] = s[1][1] = s[1][2] = s[1][3] = 0.f;
#pragma unroll
            for (int ks = 0; ks < DH / 16; ++ks) {
                uint32_t b00, b01, b10, b11;
                asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                             : "=r"(b00), "=r"(b01), "=r"(b10), "=r"(b11) : "r"(krow + ((((uint32_t)(ks * 2 + kpc)) ^ ksw) << 4)));
                mma_bf16(s[0], qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3], b00, b01);
                mma_bf16(s[1], qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3], b10, b11);
            }
            // thread: head hrow, tokens tw + nt*8 + kq + {0,1}; hi-part product in [0],[1], lo-part in [2],[3]
            float sc[4], mx = -INFINITY;
#pragma unroll
            for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                    float v = s[nt][j] + s[nt][j + 2];
                    if (c0 + tw + nt * 8 + kq + j > npos) v = -INFINITY;
                    sc[nt * 2 + j] = v;
                    mx = fmaxf(mx, v);
                }
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
            float psum = 0.f;
            uint32_t pa[4];
            {
                float pr[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) { pr[i] = (sc[i] == -INFINITY) ? 0.f : expf(sc[i] - mx); psum += pr[i]; }
                uint16_t h0, l0, h1, l1, h2, l2, h3, l3;
                split_bf16(pr[0], h0, l0); split_bf16(pr[1], h1, l1); split_bf16(pr[2], h2, l2); split_bf16(pr[3], h3, l3);
                pa[0] = (uint32_t)h0 | ((uint32_t)h1 << 16);      // row hrow,     tokens kq, kq+1
                pa[1] = (uint32_t)l0 | ((uint32_t)l1 << 16);      // row hrow + 8
                pa[2] = (uint32_t)h2 | ((uint32_t)h3 << 16);      // row hrow,     tokens 8+kq, 8+kq+1
                pa[3] = (uint32_t)l2 | ((uint32_t)l3 << 16);
            }
            psum += __shfl_xor_sync(0xffffffffu, psum, 1);
            psum += __shfl_xor_sync(0xffffffffu, psum, 2);
            // o[head][dim] = sum over the warp's tokens of p * V
            float o[DH / 8][4];
#pragma unroll
            for (int nt = 0; nt < DH / 8; ++nt) o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f;
#pragma unroll
            for (int nt = 0; nt < DH / 8; nt += 2) {
                uint32_t b00, b01, b10, b11;
                asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                             : "=r"(b00), "=r"(b01), "=r"(b10), "=r"(b11) : "r"(vrow + ((((uint32_t)(nt + vpc)) ^ vsw) << 4)));
                mma_bf16(o[nt], pa[0], pa[1], pa[2], pa[3], b00, b01);
                mma_bf16(o[nt + 1], pa[0], pa[1], pa[2], pa[3], b10, b11);
            }
            // ---- merge the group's four warps (fixed order) -> chunk partial in global memory
            {
                float *w = wp + ((size_t)wi * 8 + hrow) * wstride;
#pragma unroll
                for (int nt = 0; nt < DH / 8; ++nt) { w[nt * 8 + kq] = o[nt][0] + o[nt][2]; w[nt * 8 + kq + 1] = o[nt][1] + o[nt][3]; }
                if ((c.lane & 3) == 0) { w[DH] = mx; w[DH + 1] = psum; }
            }
            bar_sync(3 + grp, 128);
            const int gt = c.tid & 127;                      // thread within the group
            if (gt < 32) {                                   // thread = (head gt >> 2, warp gt & 3): the warp's weight
                const int h = gt >> 2, w = gt & 3;
                float mm = -INFINITY;
#pragma unroll
                for (int q = 0; q < 4; ++q) mm = fmaxf(mm, wp[((size_t)q * 8 + h) * wstride + DH]);
                const float mw = wp[((size_t)w * 8 + h) * wstride + DH];
                fw[w * 8 + h] = (mw == -INFINITY) ? 0.f : expf(mw - mm);
                if (w == 0) fw[32 + 2 * h] = mm;
            }
            bar_sync(3 + grp, 128);
            for (int i = gt; i < nh * DH; i += 128) {
                const int h = i / DH, e = i - h * DH;
                float ov = 0.f, l = 0.f;
#pragma unroll
                for (int w = 0; w < 4; ++w) {
                    const float *pw = wp + ((size_t)w * 8 + h) * wstride;
                    const float f = fw[w * 8 + h];
                    ov += f * pw[e];
                    l += f * pw[DH + 1];
                }
                const int r = b * M + m, hq = kvh * Gq + h0 + h;
                float *dst = p.s.att_part + (((size_t)r * p.Hq + hq) * p.max_chunks + chunk) * wstride;
                dst[e] = ov;
                if (e == 0) { dst[DH] = fw[32 + 2 * h]; dst[DH + 1] = l; }
            }
            bar_sync(3 + grp, 128);                          // the group's buffer is free for its next pass
        }
    }
}

struct AttnItem { int b, kvh, chunk, Lb, nch, base, rows; };

// Positions the cache of `kv` has slots for (positions beyond are flagged, never touched), the committed
// length of a sequence brought into that range, the position of its row 0 in `step` and the chunks its
// rows can see: every index the attention and merge phases form from seq_lens stays inside the block
// table and the partial buffer, whatever the caller put there.
__device__ __forceinline__ int kv_max_tokens(const MegaParams &p, const KvPtrs &kv) { return min(kv.max_pages * p.page, p.max_ctx); }
__device__ __forceinline__ int committed_len(const Cta &c, const KvPtrs &kv, int b) {
    return min(max(c.misc->seqlen[b], 0), kv_max_tokens(*c.p, kv));
}
__device__ __forceinline__ int step_base(const Cta &c, const KvPtrs &kv, int b, int step) {
    return committed_len(c, kv, b) + ((c.p->mode == 0 && step > 0) ? seq_next(c, b) - 1 + step : 0);
}
__device__ __forceinline__ int visible_chunks(const Cta &c, const KvPtrs &kv, int b, int step) {
    const int last = min(step_base(c, kv, b, step) + step_rows(c, b, step) - 1, kv_max_tokens(*c.p, kv) - 1);
    return min(last / kAttnChunk + 1, c.p->max_chunks);
}

__device__ __forceinline__ int attn_total(const Cta &c, const KvPtrs &kv, int step) {
    int total = 0;
    for (int b = 0; b < c.p->B; ++b) total += c.p->Hkv * visible_chunks(c, kv, b, step);
    return total;
}
__device__ __forceinline__ AttnItem attn_item(const Cta &c, const KvPtrs &kv, int step, int item) {
    const MegaParams &p = *c.p;
    AttnItem it;
    int b = 0, rem = item, nch = 1;
    for (; b < p.B; ++b) {
        nch = visible_chunks(c, kv, b, step);
        if (rem < p.Hkv * nch) break;
        rem -= p.Hkv * nch;
    }
    if (b >= p.B) b = p.B - 1;
    it.b = b; it.Lb = committed_len(c, kv, b); it.nch = nch;
    it.base = step_base(c, kv, b, step);
    it.rows = step_rows(c, b, step);
    it.kvh = rem / nch;
    it.chunk = rem - it.kvh * nch;
    return it;
}

__device__ __forceinline__ void produce_attention(Cta &c, const KvPtrs &kv, int step) {
    const MegaParams &p = *c.p;
    const int ptid = c.tid - kConsumerThreads;               // 0 .. 127
    const int upt = p.dh >> 3;                                // 16-byte units per token row
    const int total = attn_total(c, kv, step);
    for (int item = c.cta; item < total; item += c.grid) {
        const AttnItem it = attn_item(c, kv, step, item);
        const int c0 = it.chunk * kAttnChunk;
        const int n_old = max(0, min(kAttnChunk, it.Lb - c0));   // committed tokens of this chunk
        const int32_t *bt = kv.block_table + (size_t)it.b * kv.max_pages;
        const int slot = c.slot;
        const uint32_t parity = c.parity;
        bool ok = true;
        if (c.lane == 0) ok = wait_bar(c, &c.misc->empty[slot], parity ^ 1u);
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) return;
        const uint32_t dst0 = smem_u32(c.ring + (size_t)slot * p.stage_bytes);
        const int nunits = n_old * upt;
        // four units per round so that the copies in flight use distinct address registers
        for (int u0 = ptid; u0 < nunits; u0 += 4 * kProducerWarps * 32) {
            uint32_t d[4];
            const unsigned char *qk[4], *qv[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                int u = u0 + i * kProducerWarps * 32;
                int tok = min(u / upt, n_old - 1), w = u % upt;
                int j = c0 + tok;
                int page = bt[j / p.page];
                if ((unsigned)page >= (unsigned)kv.num_pages) { raise(c, kDevBadPage); page = 0; }
                size_t off = ((((size_t)page * p.Hkv + it.kvh) * p.page + (j % p.page)) * p.dh) * 2 + (size_t)w * 16;
                d[i] = dst0 + (uint32_t)(tok * p.dh * 2 + ((w ^ (tok & 7)) << 4));      // piece w of token row tok at w ^ (tok & 7)
                qk[i] = reinterpret_cast<const unsigned char *>(kv.k_pages) + off;
                qv[i] = reinterpret_cast<const unsigned char *>(kv.v_pages) + off;
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                if (u0 + i * kProducerWarps * 32 < nunits) {
                    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d[i]), "l"(qk[i]) : "memory");
                    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d[i] + (uint32_t)(kAttnChunk * p.dh * 2)), "l"(qv[i]) : "memory");
                }
            }
        }
        cp_async_arrive(&c.misc->full[slot]);
        next_stage(c);
    }
}

template <int DH>
__device__ __forceinline__ void attention_phase(Cta &c, const KvPtrs &kv, int step) {
    const MegaParams &p = *c.p;
    constexpr int dh = DH, half = DH >> 1;
    const int Gq = p.Hq / p.Hkv, M = c.M;
    float *qs = reinterpret_cast<float *>(c.scr);
    const float qscale = rsqrtf((float)dh);
    const int max_tokens = min(kv.max_pages * p.page, p.max_ctx);   // positions beyond are flagged, not touched
    const int upt = dh >> 3;

    const int total = attn_total(c, kv, step);
    for (int item = c.cta; item < total; item += c.grid) {
        const AttnItem it = attn_item(c, kv, step, item);
        const int b = it.b, kvh = it.kvh, chunk = it.chunk, Lb = it.Lb;
        const int base = it.base;                  // position of row m = 0
        const int rows = it.rows;                  // rows of this sequence that count (the rest is padding)
        const int c0 = chunk * kAttnChunk;
        const int32_t *bt = kv.block_table + (size_t)b * kv.max_pages;
        const int slot = c.slot;
        const uint32_t parity = c.parity;
        bf16_t *sk = reinterpret_cast<bf16_t *>(c.ring + (size_t)slot * p.stage_bytes);
        bf16_t *sv = sk + (size_t)kAttnChunk * dh;

        // -- rotated, pre-scaled queries of this KV head (independent of the stage); two elements per thread and
        // round, all eight loads of a round issued before the first use (they are L2 round trips)
        for (int i0 = c.tid; i0 < M * Gq * half; i0 += 2 * kConsumerThreads) {
            float x[2], y[2], cs[2], sn[2];
            int qi[2], e[2];
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                const int i = min(i0 + u * kConsumerThreads, M * Gq * half - 1);
                qi[u] = i / half; e[u] = i - qi[u] * half;
                const int m = qi[u] / Gq, hq = kvh * Gq + (qi[u] - m * Gq);
                const int r = b * M + m;
                int pos = base + min(m, rows - 1);
                if (pos >= max_tokens) pos = max_tokens - 1;
                const float *q = p.s.qkv + (size_t)r * (p.qdim + 2 * p.kvdim) + hq * dh;
                x[u] = ldcg_f32(q + e[u]); y[u] = ldcg_f32(q + e[u] + half);
                cs[u] = p.s.rope_cos[(size_t)pos * half + e[u]]; sn[u] = p.s.rope_sin[(size_t)pos * half + e[u]];
            }
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                if (i0 + u * kConsumerThreads < M * Gq * half) {
                    qs[qi[u] * dh + e[u]] = (x[u] * cs[u] - y[u] * sn[u]) * qscale;
                    qs[qi[u] * dh + e[u] + half] = (y[u] * cs[u] + x[u] * sn[u]) * qscale;
                }
            }
        }
        PROF(c, ATTN * 8 + 3);
        wait_bar(c, &c.misc->full[slot], parity);
        PROF(c, ATTN * 8 + 4);
        // -- positions written earlier in this launch (previous draft steps): from the pages
        {
            const int lo = max(Lb, c0), hi = min(min(base, c0 + kAttnChunk), max_tokens);
            for (int i = c.tid; i < (hi - lo) * upt; i += kConsumerThreads) {
                int tk = i / upt, w = i - tk * upt, j = lo + tk;
                int page = bt[j / p.page];
                if ((unsigned)page >= (unsigned)kv.num_pages) { raise(c, kDevBadPage); page = 0; }
                size_t off = (((size_t)page * p.Hkv + kvh) * p.page + (j % p.page)) * dh + (size_t)w * 8;
                const int ws = w ^ ((j - c0) & 7);                       // the stage's piece order (see attn_rows_mma)
                *reinterpret_cast<uint4 *>(sk + (size_t)(j - c0) * dh + ws * 8) = ldcg128(kv.k_pages + off);
                *reinterpret_cast<uint4 *>(sv + (size_t)(j - c0) * dh + ws * 8) = ldcg128(kv.v_pages + off);
            }
        }
        // -- this call's rows: rotate, round to bf16, put into the stage and append to the cache
        for (int i = c.tid; i < M * half; i += kConsumerThreads) {
            int m = i / half, e = i - m * half;
            if (m >= rows) continue;                              // padding row: nothing to store
            int r = b * M + m, pos = base + m;
            if (pos >= max_tokens) { if (chunk == 0) raise(c, kDevBadPos); continue; }
            if (pos < c0 || pos >= c0 + kAttnChunk) continue;     // another chunk's item owns it
            const float *kk = p.s.qkv + (size_t)r * (p.qdim + 2 * p.kvdim) + p.qdim + kvh * dh;
            const float *vv = kk + p.kvdim;
            float x = ldcg_f32(kk + e), y = ldcg_f32(kk + e + half);
            float cs = p.s.rope_cos[(size_t)pos * half + e], sn = p.s.rope_sin[(size_t)pos * half + e];
            uint16_t k0 = f32_bf16bits(x * cs - y * sn), k1 = f32_bf16bits(y * cs + x * sn);
            uint16_t v0 = f32_bf16bits(ldcg_f32(vv + e)), v1 = f32_bf16bits(ldcg_f32(vv + e + half));
            bf16_t *dk = sk + (size_t)(pos - c0) * dh, *dv = sv + (size_t)(pos - c0) * dh;
            const int sw = (pos - c0) & 7;
            const int ea = (((e >> 3) ^ sw) << 3) + (e & 7), eb = ((((e + half) >> 3) ^ sw) << 3) + ((e + half) & 7);
            dk[ea] = k0; dk[eb] = k1; dv[ea] = v0; dv[eb] = v1;
            int page = bt[pos / p.page];
            if ((unsigned)page >= (unsigned)kv.num_pages) { raise(c, kDevBadPage); page = 0; }
            size_t o = (((size_t)page * p.Hkv + kvh) * p.page + (pos % p.page)) * dh;
            kv.k_pages[o + e] = k0;
            kv.k_pages[o + e + half] = k1;
            kv.v_pages[o + e] = v0;
            kv.v_pages[o + e + half] = v1;
        }
        // -- value rows of the chunk's positions that nothing has written (beyond the last row of this call): zeros, so
        // that a masked probability of 0 meets a finite number in the tensor-core product
        {
            const int last = min(base + rows - 1, max_tokens - 1);
            const int nfill = max(0, min(kAttnChunk, last + 1 - c0));
            for (int i = c.tid; i < (kAttnChunk - nfill) * upt; i += kConsumerThreads)
                *reinterpret_cast<uint4 *>(sv + (size_t)nfill * dh + (size_t)i * 8) = make_uint4(0, 0, 0, 0);
        }
        bar_sync(1, kConsumerThreads);
        PROF(c, ATTN * 8 + 5);

        float *part = qs + (((size_t)M * Gq * dh + 3) & ~(size_t)3);
        attn_rows_mma<DH>(c, sk, sv, qs, part, b, kvh, chunk, base, max_tokens, rows);
        bar_sync(1, kConsumerThreads);   // every warp has read what it needs from the stage
        if (c.tid == 0) { volatile uint32_t *ud = &c.misc->use_done[slot]; *ud = *ud + 1; }   // see the mover of the tensor-memory path
        if (c.warp < kConsumerWarps / 2 && c.lane == 0) mbar_arrive(&c.misc->empty[slot]);
        next_stage(c);
        bar_sync(1, kConsumerThreads);   // the query / partial scratch is reused by the next item
    }
}

// ---- merge of the chunk partials ------------------------------------------------------------------
// After the grid barrier that ends the attention phase every (row, query head) has one partial
// (o, m, l) per visible chunk. A unit of work is a quarter of one head's output vector; units are
// dealt round-robin over the CTAs. Thread = (output element, chunk group): it adds its chunks in
// ascending order, the chunk groups are then added in ascending order, so the summation order
// depends only on the number of visible chunks, i.e. on the row's position.
__device__ __forceinline__ void merge_phase(Cta &c, const KvPtrs &kv, int step) {
    const MegaParams &p = *c.p;
    const int dh = p.dh, M = c.M, wstride = dh + 2;
    const int qe = dh >> 2;                          // output elements per unit (32 or 16)
    const int ncg = kConsumerThreads / qe;           // chunk groups (8 or 16)
    const int max_tokens = min(kv.max_pages * p.page, p.max_ctx);
    float *ms = reinterpret_cast<float *>(c.scr);    // [max_chunks] chunk maxima
    float *ls = ms + p.max_chunks;                   // [max_chunks] chunk denominators
    float *red = ls + p.max_chunks;                  // [ncg][qe + 1] partial sums (+ denominators)
    const int units = c.R * p.Hq * 4;
    const int el = c.tid % qe, cg = c.tid / qe;
    for (int u = c.cta; u < units; u += c.grid) {
        const int r = u / (p.Hq * 4), rem = u - r * (p.Hq * 4);
        const int hq = rem >> 2, e = (rem & 3) * qe + el;
        const int b = r / M, m = r - b * M;
        const int pos = min(step_base(c, kv, b, step) + min(m, step_rows(c, b, step) - 1), max_tokens - 1);
        const int ncm = min(pos / kAttnChunk + 1, p.max_chunks);        // chunks visible to this row
        const float *src = p.s.att_part + ((size_t)r * p.Hq + hq) * p.max_chunks * wstride;
        for (int i = c.tid; i < ncm; i += kConsumerThreads) {
            ms[i] = ldcg_f32(src + (size_t)i * wstride + dh);
            ls[i] = ldcg_f32(src + (size_t)i * wstride + dh + 1);
        }
        bar_sync(1, kConsumerThreads);
        float mx = -INFINITY;
        for (int i = 0; i < ncm; ++i) mx = fmaxf(mx, ms[i]);
        float ov = 0.f, l = 0.f;
#pragma unroll 4
        for (int ch = cg; ch < ncm; ch += ncg) {
            const float mc = ms[ch];
            const float f = (mc == -INFINITY) ? 0.f : expf(mc - mx);
            ov += f * ldcg_f32(src + (size_t)ch * wstride + e);
            l += f * ls[ch];
        }
        red[cg * (qe + 1) + el] = ov;
        if (el == 0) red[cg * (qe + 1) + qe] = l;
        bar_sync(1, kConsumerThreads);
        if (c.tid < qe) {
            float so = 0.f, sl = 0.f;
            for (int i = 0; i < ncg; ++i) { so += red[i * (qe + 1) + c.tid]; sl += red[i * (qe + 1) + qe]; }
            store_split(p.s.actO_hi, p.s.actO_lo, (size_t)r * p.qp + hq * dh + e, so / sl);
        }
        bar_sync(1, kConsumerThreads);
    }
}

// ---- the kernel --------------------------------------------------------------------------------
// One instantiation per (more than four activation rows?, head dimension): each contains only the
// code it runs, which keeps it near the size of the instruction cache.
template <bool TWO, int DH, bool TM>
__global__ void __launch_bounds__(TM ? kTmThreads : kThreads, 1) mega_kernel(const __grid_constant__ MegaParams p) {
    static_assert(!(TM && TWO), "tensor-memory staging serves at most four activation rows");
    extern __shared__ __align__(128) unsigned char smem[];
    Cta c;
    c.p = &p;
    c.misc = reinterpret_cast<Misc *>(smem);
    size_t off = (sizeof(Misc) + 127) & ~size_t(127);
    c.red = reinterpret_cast<float *>(smem + off);
    off += ((size_t)2 * kConsumerWarps * kTileRows * p.R * sizeof(float) + 127) & ~size_t(127);
    c.scr = smem + off;
    off += (size_t)p.scratch_smem;
    if (TM) off = (size_t)(((smem_u32(smem) + (uint32_t)off + 1023u) & ~1023u) - smem_u32(smem));   // swizzled tiles: 1024-byte aligned
    c.ring = smem + off;
    c.cta = blockIdx.x;
    c.grid = gridDim.x;
    c.tid = threadIdx.x;
    c.warp = threadIdx.x >> 5;
    c.lane = threadIdx.x & 31;
    c.slot = 0;
    c.parity = 0;
    c.tslot = 0;
    c.tparity = 0;
    c.tmem = 0;
    c.bar_target = 0;
    c.redbuf = 0;
#ifdef FMTP_PROF
    c.nprof = 0;
    for (int i = 0; i < 5; ++i) c.pacc[i] = 0;
#endif

    if (c.tid == 0) {
        for (int i = 0; i < p.n_stages; ++i) {
            mbar_init(&c.misc->full[i], kProducerWarps * 32);
            mbar_init(&c.misc->empty[i], kConsumerWarps / 2);   // the four warps that own the stage (or the mover in their place)
        }
        if (TM) {
            for (int i = 0; i < kTmSlots; ++i) {
                mbar_init(&c.misc->tfull[i], 1);
                mbar_init(&c.misc->tempty[i], kConsumerWarps / 2);
            }
            mbar_init(&c.misc->tdrain, 1);
        }
        for (int i = 0; i < kMaxStages; ++i) c.misc->use_done[i] = 0;
        c.misc->aborted = 0;
        mbar_fence_init();
    }
    if (c.tid < p.B) {
        c.misc->seqlen[c.tid] = p.kvs[0].seq_lens[c.tid];
        c.misc->next[c.tid] = (p.mode == 0 && p.n_ext) ? min(max(p.n_ext[c.tid], 1), p.M) : p.M;
    }
    // the ring starts zeroed so that never-written tails multiply as finite numbers
    for (size_t i = (size_t)c.tid * 16; i < (size_t)p.n_stages * p.stage_bytes; i += (size_t)blockDim.x * 16)
        *reinterpret_cast<uint4 *>(c.ring + i) = make_uint4(0, 0, 0, 0);
    constexpr int kMoverWarp = kConsumerWarps + kProducerWarps;
    if (TM) {
        if (c.warp == kMoverWarp) {          // the whole tensor memory of the SM (this kernel has the SM to itself)
            tmem_alloc(&c.misc->tmem_base, 512);
            tmem_relinquish();
        }
        tc_fence_before_sync();
    }
    __syncthreads();
    if (TM) {
        tc_fence_after_sync();
        c.tmem = c.misc->tmem_base;
    }

#ifdef FMTP_PROF
    const long long prof_c0 = clock64();
    const unsigned long long prof_n0 = global_timer_ns();
#endif
    const bool is_producer = (c.warp >= kConsumerWarps);
    const int n_steps = (p.mode == 0) ? p.K : 1;
    set_step_rows(c, 0);

    if (TM && c.warp >= kMoverWarp) {
        // ---------------- fourth warpgroup: one thread moves landed weight stages into tensor memory, in program
        // order; the other warps only give their registers back
        setmaxnreg_dec<kTmMoverRegs>();
        if (c.warp == kMoverWarp) {
            if (c.lane == 0) {
                bool ok = true;
                uint32_t wraps = 0;            // times the ring position has wrapped = earlier uses of the current slot
                Prog g;
#pragma unroll 1
                for (prog_begin(p, g); g.kind != DONE && ok; prog_next(p, g)) {
                    set_step_rows(c, g.step);
                    if (g.kind == EMBED || g.kind == MERGE) continue;
                    if (g.kind == ATTN) {      // K/V stages stay in shared memory: skip this CTA's items
                        const int total = attn_total(c, p.kvs[g.layer], g.step);
                        for (int item = c.cta; item < total; item += c.grid) { if (c.slot + 1 == p.n_stages) ++wraps; next_stage(c); }
                        continue;
                    }
                    const Geom geo = geom(c, g.kind);
                    const int tiles = (geo.v1 - geo.v0 + geo.cap - 1) / geo.cap;
                    const int total = tiles * geo.nks;
#pragma unroll 1
                    for (int n = 0; n < total && ok; ++n) {
                        if (n < kTmSlots) {           // the head of the phase goes through tensor memory
                            const int slot = c.slot, ts = c.tslot;
                            // A wait names a barrier phase by its parity only, so it must not be asked more than one phase
                            // ahead of the barrier; this thread skips the stages the consumers read themselves, possibly
                            // many uses of a slot. It therefore first waits until every earlier use of the slot has been
                            // taken out (counted by whoever took it), which puts the slot's barrier in this use's phase.
                            {
                                volatile uint32_t *ud = &c.misc->use_done[slot];
                                unsigned long long t0 = 0;
                                for (uint32_t it = 0; *ud < wraps; ++it) {
                                    __nanosleep(128);
                                    if ((it & 63u) == 63u) {
                                        if (ldcg_u32(p.s.abort_flag) != 0) { c.misc->aborted = 1; ok = false; break; }
                                        const unsigned long long now = global_timer_ns();
                                        if (t0 == 0) t0 = now;
                                        else if (now - t0 > p.wait_limit_ns) { do_abort(c); ok = false; break; }
                                    }
                                }
                                __threadfence_block();
                            }
                            ok = ok && wait_bar_idle(c, &c.misc->full[slot], c.parity) && wait_bar_idle(c, &c.misc->tempty[ts], c.tparity ^ 1u);
                            if (!ok) break;
                            fence_proxy_async();          // the copies' shared-memory writes, before the tensor core reads them
                            tc_fence_after_sync();
                            const uint32_t sa = smem_u32(c.ring + (size_t)slot * p.stage_bytes);
                            const uint32_t ta = c.tmem + (uint32_t)(ts * kTmSlotCols);
#pragma unroll
                            for (int h = 0; h < 2; ++h)
#pragma unroll
                                for (int q = 0; q < 4; ++q)
                                    tmem_cp_128x256b(ta + (uint32_t)(h * 32 + q * 8), umma_smem_desc(sa + (uint32_t)(h * 16384 + q * 32)));
                            // the stage may be overwritten once the copies have read it: the arrivals of the four warps that
                            // would have read it
#pragma unroll
                            for (int q = 0; q < kConsumerWarps / 2; ++q) umma_commit(&c.misc->empty[slot]);
                            umma_commit(&c.misc->tfull[ts]);
                            c.misc->use_done[slot] = wraps + 1;
                            next_tslot(c);
                        }
                        if (c.slot + 1 == p.n_stages) ++wraps;
                        next_stage(c);
                    }
                }
                // every copy issued has completed before the tensor memory is freed
                umma_commit(&c.misc->tdrain);
                for (uint32_t n = 0; n < (1u << 22) && !mbar_try_wait(&c.misc->tdrain, 0u); ++n) { }
            }
            __syncwarp();
            bar_sync(2, kConsumerThreads + 32);       // the consumers have read their last slot
            tc_fence_after_sync();
            tmem_dealloc(c.tmem, 512);
        }
        return;
    }
    if (is_producer) {
        setmaxnreg_dec<kProducerRegs>();
        // ---------------- producers: the weight / KV stream of every phase, in program order
        Prog g;
        for (prog_begin(p, g); g.kind != DONE; prog_next(p, g)) {
            set_step_rows(c, g.step);
            if (g.kind == ATTN) produce_attention(c, p.kvs[g.layer], g.step);
            else if (g.kind != EMBED && g.kind != MERGE) produce_phase<TM>(c, g.kind, p.layers[g.layer]);
        }
        cp_async_wait_all();   // every copy this thread issued has landed before the CTA may exit
        PROF_FLUSH(c, 2, 4, c.warp == kConsumerWarps && c.lane == 0);
        return;
    }

    // ---------------- consumers: one loop over the phase program; every phase ends in a grid barrier
    setmaxnreg_inc<TM ? kTmConsumerRegs : kConsumerRegs>();
    bf16_t *s_hi = reinterpret_cast<bf16_t *>(c.scr);
    EpiCtx ex;
    ex.best = 0ull;
    Prog g;
#pragma unroll 1
    for (prog_begin(p, g); g.kind != DONE; prog_next(p, g)) {
        const int kind = g.kind, step = g.step;
        set_step_rows(c, step);
        const int R = c.R;
        const LayerPtrs &L = p.layers[g.layer];
        const bool last_layer = (p.mode == 0) || (g.layer + 1 == p.n_layers);
        ex.sq.a = 0.f; ex.sq.b = 0.f;
        ex.L = &L;
        ex.step = step;
        ex.to_next_layer = (p.mode == 1) && !last_layer;
        ex.gnext = ex.to_next_layer ? p.layers[g.layer + 1].g_in : p.g_final;
        PROF(c, kind * 8);
        if (kind == ATTN) {
            attention_phase<DH>(c, p.kvs[g.layer], step);
            PROF(c, kind * 8 + 2);
            grid_barrier(c);
            continue;
        }
        if (kind == MERGE) {
            merge_phase(c, p.kvs[g.layer], step);
            PROF(c, kind * 8 + 2);
            grid_barrier(c);
            continue;
        }
        if (kind == EMBED) {
            // ---- target: x0 = Emb(tok), CTA-sliced over d; thread = (row slot tid>>3, activation row tid&7)
            int r0 = (int)(((long long)c.cta * p.d) / c.grid), r1 = (int)(((long long)(c.cta + 1) * p.d) / c.grid);
            for (int row = r0 + (c.tid >> 3); row < r1; row += kTileRows) {
                int col = c.tid & 7;
                if (col < R) {
                    int tok = p.tokens[col];
                    if ((unsigned)tok >= (unsigned)p.V) { raise(c, kDevBadToken); tok = 0; }
                    float v = bf16bits_f32(p.embed[(size_t)tok * p.d + row]);
                    p.s.x0[(size_t)col * p.d + row] = v;
                    store_split(p.s.actD_hi, p.s.actD_lo, (size_t)col * p.dp + row, v * bf16bits_f32(L.g_in[row]));
                    ex.sq.a += v * v;
                }
            }
            flush_sq(c, ex.sq, p.s.ssA, nullptr);
            PROF(c, kind * 8 + 2);
            grid_barrier(c);
            continue;
        }

        // ============ matrix phases: stage the input vector(s) in shared memory ...
        const int klen = (kind == PROJ) ? 2 * p.d : (kind == OPROJ) ? p.qdim : (kind == DOWN) ? p.F : p.d;
        const int st = ((klen + 31) & ~31) + 32;      // +64 B: rows land in different banks
        bf16_t *a_hi = s_hi, *a_lo = s_hi + (size_t)R * st;
        ActSrc act{a_hi, a_lo, st, true};
        if (kind == PROJ) {
            // ---- x0 = W_p [ rms(h) ; rms(Emb(tok)) ]
            // loads that do not depend on each other are issued first: the previous step's argmax key,
            // the partial sums that normalise the recursed state, and that state itself
            unsigned long long key = 0ull;
            if (step > 0 && c.tid < R) key = ldcg_u64(p.s.keys + (size_t)(step - 1) * kMaxRows + c.tid);
            float pvc[kPartialRegs], pvd[kPartialRegs];
            const bool renorm = step > 0 && c.warp < R;
            if (renorm) {
                const int col = src_row(c, c.warp, step);      // step 1 continues each sequence's last extend row
                load_partials(c, p.s.ssC, col, pvc);
                load_partials(c, p.s.ssD, col, pvd);
            }
            if (step > 0) stage_hilo(c, p.s.actR_hi, p.s.actR_lo, p.dp, p.d, a_hi, a_lo, st, 0, step);
            if (renorm) {
                // recursed state: h = (x2*g_final) * s_x; rms(h) adds s_h = rsqrt(s_x^2 * mean((x2 g)^2) + eps)
                float sx = rsqrtf(reduce_partials(pvc) / (float)p.d + p.eps);
                float sy = reduce_partials(pvd) / (float)p.d;
                if (c.lane == 0) c.misc->scale0[c.warp] = sx * rsqrtf(sx * sx * sy + p.eps);
            }
            if (c.tid < R) {
                int tok;
                if (step == 0) {
                    const int b = c.tid / p.M;         // a padding row's token is never looked at
                    tok = (c.tid - b * p.M < seq_next(c, b)) ? p.tokens[c.tid] : 0;
                } else {
                    if ((key >> 32) == 0ull) raise(c, kDevAllNan);
                    tok = (int)argmax_key_id(key);
                    if (c.cta == 0) p.out_tokens[(size_t)c.tid * p.K + (step - 1)] = tok;
                }
                if ((unsigned)tok >= (unsigned)p.V) { raise(c, kDevBadToken); tok = 0; }
                c.misc->tok[c.tid] = tok;
            }
            bar_sync(1, kConsumerThreads);
#pragma unroll 1
            for (int r = 0; r < R; ++r) {
                float sqh = 0.f, sqe = 0.f;
                const bf16_t *erow = p.embed + (size_t)c.misc->tok[r] * p.d;
                for (int k = c.tid * 8; k < p.d; k += kConsumerThreads * 8) {
                    uint4 ev = ldnc128(erow + k);
                    uint4 gv = ldnc128(p.g_enorm + k);
                    uint32_t ew[4] = {ev.x, ev.y, ev.z, ev.w}, gw[4] = {gv.x, gv.y, gv.z, gv.w};
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        float e0 = bf16lo_f32(ew[i]), e1 = bf16hi_f32(ew[i]);
                        sqe += e0 * e0 + e1 * e1;
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
                            sqh += h0 * h0 + h1 * h1;
                            store_split(a_hi, a_lo, (size_t)r * st + k + 2 * i, h0 * bf16lo_f32(hgw[i]));
                            store_split(a_hi, a_lo, (size_t)r * st + k + 2 * i + 1, h1 * bf16hi_f32(hgw[i]));
                        }
                    }
                }
                // block sums of the two squared norms of row r
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    sqh += __shfl_xor_sync(0xffffffffu, sqh, o);
                    sqe += __shfl_xor_sync(0xffffffffu, sqe, o);
                }
                if (c.lane == 0) { c.misc->ssred[c.warp][r][0] = sqh; c.misc->ssred[c.warp][r][1] = sqe; }
            }
            bar_sync(1, kConsumerThreads);
            if (c.tid < R) {
                float sh = 0.f, se = 0.f;
                for (int i = 0; i < kConsumerWarps; ++i) { sh += c.misc->ssred[i][c.tid][0]; se += c.misc->ssred[i][c.tid][1]; }
                if (step == 0) c.misc->scale0[c.tid] = rsqrtf(sh / (float)p.d + p.eps);
                c.misc->scale1[c.tid] = rsqrtf(se / (float)p.d + p.eps);
            }
        } else {
            // ---- the previous phase's output vector (hi/lo) and the sum of squares that normalises it
            const bf16_t *ghi, *glo;
            const float *sstab = nullptr;
            int gstride = p.dp, glen = p.d;
            switch (kind) {
                case QKV:    ghi = p.s.actD_hi; glo = p.s.actD_lo; sstab = p.s.ssA; break;
                case OPROJ:  ghi = p.s.actO_hi; glo = p.s.actO_lo; gstride = p.qp; glen = p.qdim; break;
                case GATEUP: ghi = p.s.actP_hi; glo = p.s.actP_lo; sstab = p.s.ssB; break;
                case DOWN:   ghi = p.s.actF_hi; glo = p.s.actF_lo; gstride = p.Fp; glen = p.Fp; break;   // pad beyond F is zero
                default:     ghi = p.s.actH_hi; glo = p.s.actH_lo; sstab = p.s.ssC; break;               // HEAD
            }
            float pv[kPartialRegs];
            const bool norm = sstab != nullptr && c.warp < R;
            if (norm) load_partials(c, sstab, c.warp, pv);       // in flight while the vector is staged
            if (kind == DOWN) act = ActSrc{ghi, glo, gstride, false};     // read from global memory inside the loop
            else stage_hilo(c, ghi, glo, gstride, glen, a_hi, a_lo, st, 0);
            if (norm) {
                float sc = rsqrtf(reduce_partials(pv) / (float)p.d + p.eps);
                if (c.lane == 0) c.misc->scale0[c.warp] = sc;
            }
        }
        if (kind == HEAD && c.tid < R) c.misc->outrow[c.tid] = out_row(c, c.tid, step);
        bar_sync(1, kConsumerThreads);
        if (kind == HEAD && p.out_h) {   // every CTA writes its slice of the post-final-norm hidden state
            int r0 = (int)(((long long)c.cta * p.d) / c.grid), r1 = (int)(((long long)(c.cta + 1) * p.d) / c.grid);
            for (int i = c.tid; i < R * (r1 - r0); i += kConsumerThreads) {
                int r = i / (r1 - r0), k = r0 + (i - r * (r1 - r0));
                const int orow = c.misc->outrow[r];
                if (orow < 0) continue;                    // an extend row that is not its sequence's last
                float y = bf16bits_f32(a_hi[(size_t)r * st + k]) + bf16bits_f32(a_lo[(size_t)r * st + k]);
                size_t o = (p.mode == 0) ? ((size_t)orow * p.K + step) * p.d + k : (size_t)orow * p.d + k;
                p.out_h[o] = f32_bf16bits(y * c.misc->scale0[r]);
            }
        }
        PROF(c, kind * 8 + 1);

        // ============ ... stream the weights ...
        consume_tiles<TWO, TM>(c, kind, act, ex);

        // ============ ... and publish what the next phase needs besides the vector
        if (kind == PROJ) flush_sq(c, ex.sq, p.s.ssA, nullptr);
        else if (kind == OPROJ) flush_sq(c, ex.sq, p.s.ssB, nullptr);
        else if (kind == DOWN) flush_sq(c, ex.sq, ex.to_next_layer ? p.s.ssA : p.s.ssC, (p.mode == 0) ? p.s.ssD : nullptr);
        else if (kind == HEAD) {
            // reduce the per-thread maxima (thread = (row slot, col)) over the 32 row slots
            unsigned long long k = ex.best;
            unsigned long long o8 = __shfl_xor_sync(0xffffffffu, k, 8);
            k = o8 > k ? o8 : k;
            unsigned long long o16 = __shfl_xor_sync(0xffffffffu, k, 16);
            k = o16 > k ? o16 : k;
            if (c.lane < 8) c.misc->keyred[c.warp][c.lane] = k;
            bar_sync(1, kConsumerThreads);
            if (c.tid < R) {
                unsigned long long m = 0ull;
                for (int w = 0; w < kConsumerWarps; ++w) m = c.misc->keyred[w][c.tid] > m ? c.misc->keyred[w][c.tid] : m;
                const int orow = c.misc->outrow[c.tid];
                if (m != 0ull && orow >= 0) atomicMax(p.s.keys + (size_t)step * kMaxRows + orow, m);
            }
            ex.best = 0ull;
        }
        PROF(c, kind * 8 + 2);
        grid_barrier(c);
    }
    PROF(c, DONE * 8);
    if (TM) {                                  // lets the mover's warp free the tensor memory
        tc_fence_before_sync();
        bar_arrive(2, kConsumerThreads + 32);
    }

    PROF_FLUSH(c, 0, 2, c.tid == 0);
    PROF_FLUSH(c, 4, 5, c.tid == 0);
#ifdef FMTP_PROF
    if (c.tid == 0) {
        atomicAdd((unsigned long long *)&g_wait[c.cta][5], (unsigned long long)(clock64() - prof_c0));
        atomicAdd((unsigned long long *)&g_wait[c.cta][6], global_timer_ns() - prof_n0);
    }
#endif
    // ============ publish the last step's tokens and the status word
    if (c.cta == 0 && c.tid < ((p.mode == 0) ? p.B : p.R)) {
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

#ifdef FMTP_PROF
extern "C" int fmtp_prof_wait(long long *host, int reset) {
    int e = (int)cudaMemcpyFromSymbol(host, g_wait, sizeof(g_wait));
    if (reset) { static long long z[160][8]; cudaMemcpyToSymbol(g_wait, z, sizeof(z)); }
    return e;
}
extern "C" int fmtp_prof_read(unsigned long long *host, size_t bytes) {
    return (int)cudaMemcpyFromSymbol(host, g_prof, bytes < sizeof(g_prof) ? bytes : sizeof(g_prof));
}
#endif

size_t mega_smem_bytes(const MegaParams &p) {
    size_t off = (sizeof(Misc) + 127) & ~size_t(127);
    off += ((size_t)2 * kConsumerWarps * kTileRows * p.R * sizeof(float) + 127) & ~size_t(127);
    off += (size_t)p.scratch_smem;
    if (p.use_tmem) off = ((off + 1023) & ~size_t(1023)) + 1024;      // the ring starts on a 1024-byte boundary, wherever the base lies
    off += (size_t)p.n_stages * p.stage_bytes;
    return off;
}

size_t mega_fixed_smem(int R) {
    size_t off = (sizeof(Misc) + 127) & ~size_t(127);
    off += ((size_t)2 * kConsumerWarps * kTileRows * R * sizeof(float) + 127) & ~size_t(127);
    return off;
}

namespace {
const void *kernel_for(int R, int dh, int tm) {
    if (tm) return dh == 128 ? (const void *)mega_kernel<false, 128, true> : (const void *)mega_kernel<false, 64, true>;
    if (dh == 128) return R > 4 ? (const void *)mega_kernel<true, 128, false> : (const void *)mega_kernel<false, 128, false>;
    return R > 4 ? (const void *)mega_kernel<true, 64, false> : (const void *)mega_kernel<false, 64, false>;
}
}  // namespace

int mega_kernel_index(const MegaParams &p) {
    if (p.use_tmem) return 4 + (p.dh == 128 ? 1 : 0);
    return (p.dh == 128 ? 2 : 0) + (p.R > 4 ? 1 : 0);
}

int mega_max_grid(const MegaParams &p, size_t smem_bytes, int *err) {
    int dev = 0, sms = 0, per_sm = 0;
    const void *fn = kernel_for(p.R, p.dh, p.use_tmem);
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes);
    if (e == cudaSuccess) e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fn, p.use_tmem ? kTmThreads : kThreads, smem_bytes);
    if (err) *err = (int)e;
    if (e != cudaSuccess) return 0;
    return sms * (per_sm > 0 ? 1 : 0);
}

int mega_launch(const MegaParams &p, int grid, cudaStream_t stream) {
    size_t smem = mega_smem_bytes(p);
    const void *fn = kernel_for(p.R, p.dh, p.use_tmem);
    void *args[] = {const_cast<MegaParams *>(&p)};
    return (int)cudaLaunchCooperativeKernel(fn, dim3(grid), dim3(p.use_tmem ? kTmThreads : kThreads), args, smem, stream);
}

}  // namespace fmtp
