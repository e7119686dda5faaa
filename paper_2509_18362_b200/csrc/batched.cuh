// Batched path of the draft and target calls: groups of up to 64 activation rows run as a sequence of kernels
// on one stream, with every weight matrix streamed once per step and group by the tcgen05 GEMM of
// skinny_gemm.cuh. (Calls whose rows fit one launch of the persistent kernel of megakernel.cu -- up to 8 rows,
// and fewer than 3 sequences at 7B-class widths -- run there instead.)
#pragma once
#include "mega.cuh"

namespace fmtp {

constexpr int kBatchRows = 64;        // sequences per group (activation columns = 2 x rows <= 128)
constexpr int kBatchAttnChunk = 256;  // fewest context tokens per attention work item (sizes the partial buffer)
// Context tokens per attention work item for a row that sees n_ctx positions. An item ends with serial work (the
// compute warps merge their partials and write the chunk's) while the K/V stream of the next items waits, so long
// contexts take four times longer items (measured at 64 sequences with contexts in [512, 8192]: -13 us of 393 per
// step); up to 4096 positions a row keeps 256-token items so that a small batch still spreads over all SMs. The size
// is a function of the row's own context only: a row's summation order does not depend on the batch it is in.
__host__ __device__ inline int attn_chunk_tokens(int n_ctx) { return n_ctx > 4096 ? 1024 : kBatchAttnChunk; }
constexpr int kBatchMaxSplits = 8;

// What the launches of the batched path would otherwise ask the driver for on every call; lives in the context
// (one per device), filled on first use: the tensor maps of the GEMMs' activation operands, and the
// shared-memory limits already raised on the kernels.
struct TmapEntry {
    const void *x;
    int ldx, K, NB;
    alignas(64) unsigned char map[128];      // a CUtensorMap
};
struct TmapCache {
    TmapEntry e[12];
    int n, next;
    int gemm_smem[3];                        // limit set on skinny_gemm_kernel<1>, <2>, <4>
    int attn_smem;                           // limit set on attn_kernel
};

struct BatchedWs {
    bf16_t *xop0;                 // [128][ld0]  hi/lo activation operand (projection, QKV, O-proj, MLP and head inputs)
    bf16_t *xopF;                 // [128][ldF]  hi/lo SwiGLU activation (input of the down projection)
    bf16_t *xopH;                 // [128][ld0]  head operand gathered from the passes of a draft's extend step
    float *partial;               // [kBatchMaxSplits][rows][ldp] split-K partial sums
    float *x;                     // [rows][d]   residual stream
    float *hout;                  // [rows][d]   final-normed hidden state (recursed in fp32)
    float *q;                     // [rows][qdim] rotated queries
    float *att_part;              // [rows][Hq][max_chunks][dh + 2]  (o, m, l) per context chunk
    unsigned long long *keys;     // [max_K][kBatchRows] argmax keys
    uint32_t *id_bitmap;          // [ceil(V/32)] membership bits of the subset
    int32_t *sorted_ids;          // [V] the subset in ascending id order
    uint32_t *status;
    int ld0, ldF, ldp, max_chunks, rows;
    size_t keys_bytes;
};

struct BatchedShape {
    int d, Hq, Hkv, dh, F, V, page, max_ctx, max_K, max_rows;
    float eps;
};

// Carves the buffers out of `base` (nullptr: size query); returns the bytes used.
size_t batched_layout(BatchedWs &ws, unsigned char *base, const BatchedShape &sh);

struct BatchedCall {
    BatchedShape sh;
    BatchedWs ws;
    const float *rope_cos, *rope_sin;     // [max_ctx][dh/2]
    int n_sm, smem_optin;
    TmapCache *cache;
    unsigned long long wait_limit_ns;     // every device-side wait gives up after this long
    int inject_gemm_timeout;              // self-test: the call's first GEMM expects a copy that is never made
    int B, K, N;
    const int32_t *ids;                   // subset or NULL
    int M0;                               // extend rows per sequence in step 0 (layout of h_last / tok_last), >= 1
    const int32_t *n_ext;                 // [B] rows of a sequence that count (1..M0), NULL = M0 for every sequence
    const bf16_t *h_last;                 // [B][M0][d]
    const int32_t *tok_last;              // [B][M0]
    int32_t *out_drafts;                  // [B][K]
    bf16_t *out_h;                        // [B][K][d] or NULL
    float *out_logits;                    // [B][K][N] or NULL
    uint32_t *user_status;
    const bf16_t *embed, *lm_head, *g_hnorm, *g_enorm, *w_proj, *g_final;
    LayerPtrs layer;
    KvPtrs kv;
};

struct BatchedTargetCall {
    BatchedShape sh;
    BatchedWs ws;
    const float *rope_cos, *rope_sin;
    int n_sm, smem_optin;
    TmapCache *cache;
    unsigned long long wait_limit_ns;
    int B, M, n_layers;                   // B * M <= kBatchRows rows
    const int32_t *tokens;                // [B][M]
    bf16_t *out_h;                        // [B][M][d] or NULL
    bf16_t *out_logits;                   // [B][M][V] or NULL
    int32_t *out_argmax;                  // [B][M] or NULL
    uint32_t *user_status;
    const bf16_t *embed, *lm_head, *g_final;
    const LayerPtrs *layers;              // host array [n_layers]
    const KvPtrs *kvs;                    // host array [n_layers]
};

// Enqueues one target-decoder step (all layers, final norm, full output head) for B sequences of M rows.
int batched_target(const BatchedTargetCall &c, cudaStream_t stream, long long *launches);

// Enqueues all K steps for one group of B <= kBatchRows sequences. Returns a cudaError_t (0 = ok)
// and adds the kernels launched to *launches.
int batched_draft(const BatchedCall &c, cudaStream_t stream, long long *launches);

}  // namespace fmtp
