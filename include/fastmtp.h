/*
 * fastmtp.h -- C ABI of the B200 (sm_100a) FastMTP draft / verify library.
 *
 * The library implements the inference hot path of FastMTP (arXiv 2509.18362): the
 * recursive K-step draft of one position-shared Multi-Token-Prediction head with a
 * compressed-vocabulary output head, the greedy verification that consumes the drafts,
 * and a target-decoder step that reuses the same decoder-layer kernels.
 *
 * Conventions shared by every call
 *   - All tensors are dense, row-major, caller-owned. "dev" = device (HBM) pointer,
 *     "host" = host pointer. bf16 values are passed as raw 16-bit patterns (fmtp_bf16).
 *   - Matrices are [out, in]. Token ids, lengths and indices are int32.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *     Device-pointer entry points only enqueue work on `stream`; they never synchronise
 *     and never read device memory on the host. The *_host entry points copy their
 *     per-step inputs host->device, run, copy results device->host and synchronise
 *     `stream` before returning.
 *   - Return value: FMTP_OK (0) or a negative fmtp_status. On a negative return nothing
 *     was enqueued. Errors only a kernel can see (token id >= vocab, page index out of
 *     range, position beyond the block table, a bounded wait that ran out) never fault:
 *     the access is clamped or skipped, a bit is OR-ed into the caller's `dev_status`
 *     word (FMTP_DEV_* flags) and the kernel runs to completion.
 *   - The library allocates no device memory of its own except where stated: the caller
 *     sizes a workspace with fmtp_workspace_bytes() and hands it over with
 *     fmtp_set_workspace(). One context must not be used from two streams at once.
 */
#ifndef FASTMTP_H
#define FASTMTP_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef uint16_t fmtp_bf16;
typedef struct fmtp_ctx fmtp_ctx;

typedef enum {
    FMTP_OK = 0,
    FMTP_EINVAL = -1,       /* null pointer, non-positive size, misaligned pointer        */
    FMTP_ESHAPE = -2,       /* shape outside what the kernels support (see fmtp_create)   */
    FMTP_EUNSUPPORTED = -3, /* valid request that this build does not implement           */
    FMTP_ENOMEM = -4,       /* workspace missing or too small                             */
    FMTP_ECUDA = -5,        /* a CUDA runtime call failed (see fmtp_last_cuda_error)       */
    FMTP_ETIMEOUT = -6,
    FMTP_EBOUNDS = -7
} fmtp_status;

/* Bits OR-ed into *dev_status by kernels. */
#define FMTP_DEV_BAD_TOKEN   0x1u  /* a token id or subset id outside [0, vocab) was clamped  */
#define FMTP_DEV_BAD_PAGE    0x2u  /* a block-table entry outside [0, num_pages) was clamped  */
#define FMTP_DEV_BAD_POS     0x4u  /* a position beyond max_pages_per_seq*page_size: KV write skipped */
#define FMTP_DEV_TIMEOUT     0x8u  /* a bounded device-side wait gave up; outputs are invalid */
#define FMTP_DEV_ALL_NAN     0x10u /* an argmax row held no comparable value; id 0 / lowest id returned */

/* Model geometry and capacity limits (fixed for the life of a context).
 * Supported: head_dim in {64, 128}; d, n_q_heads*head_dim and ffn multiples of 16 with
 * d a multiple of 64; n_q_heads a multiple of n_kv_heads with at most 8 query heads per
 * KV head; max_rows <= 4096 (rows = batch x rows-per-sequence handled in one call).
 *
 * Two kernel paths sit behind the draft and target calls, chosen by the call's number of
 * sequences B alone (never by rows per sequence, so a position scored as one of 1 or of K+1 rows
 * gives the same bits):
 *   - few sequences (as many as fit one launch: up to 8 rows; at most 2 sequences for models that
 *     stream >= 256 MB of layer weights per step): one persistent kernel launch per call, or per
 *     group of whole sequences when the rows exceed one launch;
 *   - more sequences: groups of up to 64 rows, each step a sequence of kernels on the caller's
 *     stream that read every weight once per group (tensor-core GEMMs).
 * Within a path a sequence's results do not depend on the batch it is in; between the two paths
 * results agree within the documented tolerances, not bit for bit (different summation order).
 * The environment variable FMTP_BATCHED_MIN (read at fmtp_create) overrides the switch point; FMTP_TMEM=1 (also read
 * at fmtp_create) lets the persistent kernel stage weights through tensor memory where the shape allows (results agree
 * with the default within the tolerances of the tests, not bit for bit: the k chunks are dealt to the warps differently). */
typedef struct {
    int32_t d, n_q_heads, n_kv_heads, head_dim, ffn, vocab;
    int32_t n_layers;      /* target decoder depth (fastmtp_target_step); the MTP head has 1 */
    float rms_eps, rope_theta;
    int32_t page_size;     /* tokens per KV page */
    int32_t max_rows;      /* largest batch x rows-per-sequence of any call                 */
    int32_t max_K;         /* largest number of draft steps                                  */
    int32_t max_ctx;       /* largest position + 1 any sequence may reach                    */
} fmtp_shape;

/* One pre-norm decoder layer (Sec. 2.1 of the paper: the transformer block inside the MTP
 * module; also each target layer). All dev, bf16. RMSNorm gains g_* are [d];
 * wq [Hq*dh, d], wk/wv [Hkv*dh, d], wo [d, Hq*dh], w_gate/w_up [ffn, d], w_down [d, ffn]. */
typedef struct {
    const fmtp_bf16 *g_in, *wq, *wk, *wv, *wo, *g_post, *w_gate, *w_up, *w_down;
} fmtp_layer_w;

/* The MTP head (Sec. 2.1 "Architecture Design"): embed [vocab, d] and lm_head [vocab, d] are
 * the main model's (shared, Sec. 2.2); g_hnorm / g_enorm [d] normalise the incoming hidden
 * state and the token embedding; w_proj [d, 2d] projects their concatenation
 * [norm(h) ; norm(emb)]; g_final [d] is the norm before the output head. */
typedef struct {
    const fmtp_bf16 *embed, *lm_head, *g_hnorm, *g_enorm, *w_proj, *g_final;
    fmtp_layer_w layer;
} fmtp_mtp_w;

/* The target decoder: `layers` is a HOST array of n_layers entries holding dev pointers. */
typedef struct {
    const fmtp_bf16 *embed, *lm_head, *g_final;
    const fmtp_layer_w *layers;
} fmtp_target_w;

/* Paged bf16 KV cache of one layer. k_pages / v_pages: dev [num_pages, Hkv, page_size, dh]
 * (keys stored after the rotary embedding). block_table: dev [B, max_pages_per_seq] page
 * indices; seq_lens: dev [B] committed tokens per sequence. Calls read seq_lens on the
 * device (so a replayed launch sees current values) and never modify it. */
typedef struct {
    fmtp_bf16 *k_pages, *v_pages;
    const int32_t *block_table;
    const int32_t *seq_lens;
    int32_t num_pages, max_pages_per_seq;
} fmtp_kv;

/* ---- context ------------------------------------------------------------------------ */

/* Validates `shape` for the current device and creates a context (host memory only).
 * FMTP_ESHAPE if the geometry is unsupported, FMTP_ECUDA if no sm_100 device is current. */
int fmtp_create(const fmtp_shape *shape, fmtp_ctx **out);
int fmtp_destroy(fmtp_ctx *ctx);

/* Bytes of device scratch the context needs (activations between phases, attention
 * partials, rotary table, control words). */
size_t fmtp_workspace_bytes(const fmtp_ctx *ctx);

/* Hands `bytes` of 256-byte-aligned device memory to the context; the context clears it,
 * builds its rotary cos/sin table in it (computed on the host in double precision) and
 * synchronises the device once. The caller keeps ownership and must keep it alive and
 * untouched while the context is used. */
int fmtp_set_workspace(fmtp_ctx *ctx, void *dev, size_t bytes);

const char *fmtp_strerror(int status);
/* cudaError_t of the most recent failing CUDA call made through this context (0 if none). */
int fmtp_last_cuda_error(const fmtp_ctx *ctx);
/* Number of kernel launches this context has enqueued so far. */
long long fmtp_launch_count(const fmtp_ctx *ctx);
/* Of those, launches of the persistent kernel that staged weights through tensor memory (opt-in: environment
 * variable FMTP_TMEM=1 when the context is created; used only for shapes whose contraction lengths are all
 * multiples of 512 and calls of at most four activation rows). */
long long fmtp_tmem_launch_count(const fmtp_ctx *ctx);

/* Diagnostic (no counterpart in the paper): runs a one-warp kernel that waits, with the library's
 * bounded wait loop and a limit of `limit_ms` milliseconds (1..1000), for an event that never comes.
 * On expiry the kernel ORs FMTP_DEV_TIMEOUT into *dev_status (dev, 1 word), optionally stores the
 * nanoseconds it waited in *dev_waited_ns (dev, may be NULL) and returns normally: nothing hangs,
 * traps or faults, and later calls on the same device work as before. The decoder kernel's own waits
 * (ring stages, grid barriers) use the same loop with a 2 s limit. */
int fmtp_selftest_wait_timeout(uint32_t *dev_status, int limit_ms, unsigned long long *dev_waited_ns, void *stream);

/* Diagnostic (no counterpart in the paper): arms the NEXT fastmtp_draft call on this context so that one of its own
 * device-side waits cannot end, with every wait of that call limited to `limit_ms` milliseconds (1..1000):
 *   which = 1  the persistent kernel's grid barrier expects one arrival more than there are CTAs
 *              (takes effect if that call runs on the persistent path);
 *   which = 2  the first ring stage of the call's first tensor-core GEMM expects one copy more than is made
 *              (takes effect if that call runs on the batched path).
 * The wait runs out, the kernel ORs FMTP_DEV_TIMEOUT into the status word, every other CTA / role sees the abort
 * flag and stops waiting, copies in flight are drained, tensor memory is freed, and the launch -- and the rest of
 * the call's launches, on garbage that stays inside the caller's buffers -- ends normally: nothing hangs, traps or
 * faults. The call's outputs are invalid; the context and the device stay usable and the next call is unaffected. */
int fmtp_selftest_inject_wait_timeout(fmtp_ctx *ctx, int limit_ms, int which);

/* ---- draft: Sec. 2.3 "Drafting phase", Sec. 2.1 steps k=1 / k>1, Sec. 2.2 Eq. 3 -------- */

/* Recursive K-step draft for B sequences.
 *
 * Extend rows. Since its last draft call sequence b has committed n = n_ext[b] new positions (n = accepted
 * drafts + 1 after a verification, the prompt after a prefill). For each of them the caller passes the pair
 * (h_last[b][m], tok_last[b][m]): the target's hidden state at that position (the post-final-norm vector
 * that feeds the target's output head) and the token that follows it. The pairs take MTP-cache positions
 * L_b .. L_b + n - 1 (L_b = mtp_kv->seq_lens[b]) and run through the MTP module in ONE pass over its
 * weights, causal among themselves: this is step k = 1 of the paper, which runs the head over the shifted
 * sequence with the target's hidden states. Only the last pair feeds the output head and gives draft 1.
 * max_ext = 1 with n_ext = NULL is the plain form: one pair (h_last[b], tok_last[b]) per sequence.
 *
 * Each step embeds the token, RMS-normalises hidden state and embedding, projects their concatenation
 * 2d -> d, runs one decoder layer (appending this position's K/V to the MTP cache and attending over
 * positions 0..pos), applies the final norm, and takes the argmax of the output head restricted to rows
 * `vocab_subset` (Eq. 3) -- ties go to the lowest token id; no logits are written. Step k >= 2 consumes the
 * head's own previous output hidden state (kept in fp32) and the previous draft at position
 * L_b + n - 1 + (k - 1). All K steps are enqueued without returning to the host (one kernel launch on the
 * persistent path, a fixed sequence of launches on the batched path).
 *
 *   h_last        dev [B, max_ext, d] bf16   tok_last     dev [B, max_ext] int32
 *   n_ext         dev [B] int32 in [1, max_ext] (values outside are clamped), or NULL: every sequence has
 *                 max_ext pairs. Rows m >= n_ext[b] of h_last / tok_last are padding and are never used.
 *   vocab_subset  dev [N] int32 distinct ids in [0, vocab), any order; NULL => full vocab (N ignored)
 *   out_drafts    dev [B, K] int32           out_h        dev [B, K, d] bf16 or NULL (post-final-norm)
 *   out_logits    dev [B, K, N] fp32 or NULL: debug copy of the subset logits (defeats the
 *                 "no logits written" property; leave NULL in production)
 *   dev_status    dev 1 word, OR-ed with FMTP_DEV_* flags; may be NULL
 *
 * The call writes MTP-cache slots L_b .. L_b + n + K - 2 and does not change seq_lens; the caller commits
 * by advancing seq_lens by n (the extend rows are final; the K - 1 slots after them are speculative and
 * are overwritten by the next call). Extending in one call gives the same bits as n calls with one pair
 * each on the persistent path, and agrees within the tolerances on the batched path.
 * Requires B * max_ext <= max_rows, max_ext <= 64, K <= max_K, L_b + n + K - 1 <= max_ctx. The persistent
 * kernel takes the call when B is below the switch point and the B * max_ext rows fit one launch (8 rows;
 * 4 at the 7B-class width), the batched path otherwise.
 */
int fastmtp_draft(fmtp_ctx *ctx, const fmtp_mtp_w *w,
                  const fmtp_bf16 *h_last, const int32_t *tok_last, const int32_t *n_ext, int max_ext,
                  const fmtp_kv *mtp_kv, int B, int K,
                  const int32_t *vocab_subset, int N,
                  int32_t *out_drafts, fmtp_bf16 *out_h, float *out_logits,
                  uint32_t *dev_status, void *stream);

/* Same operation with the per-step inputs and the result in HOST memory: h_last host
 * [B,max_ext,d] bf16, tok_last host [B,max_ext] and n_ext host [B] (or NULL) are copied to the device, the
 * draft runs, out_drafts host [B,K] is copied back and `stream` is synchronised. Weights, subset and KV
 * cache stay on the device. Returns FMTP_EBOUNDS / FMTP_ETIMEOUT if the kernels flagged a problem. */
int fastmtp_draft_host(fmtp_ctx *ctx, const fmtp_mtp_w *w,
                       const fmtp_bf16 *h_last_host, const int32_t *tok_last_host, const int32_t *n_ext_host, int max_ext,
                       const fmtp_kv *mtp_kv, int B, int K,
                       const int32_t *vocab_subset, int N,
                       int32_t *out_drafts_host, void *stream);

/* ---- verification: Sec. 2.3 "Verification phase" (greedy, Sec. 3.1) --------------------- */

/* g[b,j] = argmax over the full vocabulary of target_logits[b,j,:] (ties to the lowest id,
 * NaN never wins); accept_len[b] = number of leading drafts with drafts[b,j] == g[b,j];
 * bonus[b] = g[b, accept_len[b]]: the token the target emits after the accepted prefix, so
 * a round emits accept_len + 1 tokens.
 *
 *   target_logits dev [B, K+1, V] bf16     drafts       dev [B, K] int32 (ignored if K == 0)
 *   out_accept_len, out_bonus dev [B]      out_argmax   dev [B, K+1] or NULL
 * Requires B*(K+1) <= 4096 rows. Uses the context workspace for per-row keys.
 */
int fastmtp_verify_accept(fmtp_ctx *ctx, const fmtp_bf16 *target_logits, const int32_t *drafts,
                          int B, int K, int V,
                          int32_t *out_accept_len, int32_t *out_bonus, int32_t *out_argmax,
                          uint32_t *dev_status, void *stream);

/* The acceptance step of Sec. 2.3 "Verification phase" on token ids: for callers whose target step already
 * returned the greedy token of every verification row (fastmtp_target_step with out_argmax and
 * out_logits = NULL), so that no [B, K+1, V] logits are ever written or read. Same rule and same results as
 * fastmtp_verify_accept given g = target_argmax: accept_len[b] = number of leading drafts equal to g[b, j],
 * bonus[b] = g[b, accept_len[b]].
 *
 *   target_argmax dev [B, K+1] int32       drafts dev [B, K] int32 (ignored if K == 0)
 *   out_accept_len, out_bonus dev [B]
 * Uses no workspace; any B. */
int fastmtp_accept_ids(fmtp_ctx *ctx, const int32_t *target_argmax, const int32_t *drafts, int B, int K,
                       int32_t *out_accept_len, int32_t *out_bonus, void *stream);

/* Host-buffer form: logits and drafts are copied in, accept_len / bonus copied out. */
int fastmtp_verify_accept_host(fmtp_ctx *ctx, const fmtp_bf16 *target_logits_host,
                               const int32_t *drafts_host, int B, int K, int V,
                               int32_t *out_accept_len_host, int32_t *out_bonus_host, void *stream);

/* ---- verification without a context or any allocation ------------------------------------ */

/* The paper has no counterpart for this call; it exists for hosts that cannot allocate. Same
 * operation and same results as fastmtp_verify_accept, but it takes no context and no workspace:
 * the per-row scratch lives in a fixed array inside the library (8.3 KB of device memory on every
 * GPU that loads the library, held until the process exits). Meant for callers that only hold raw
 * device pointers, or that run where creating device memory is impossible or would stall the GPU
 * (an allocator that already owns all of it, a latency-critical decode loop). The call itself
 * performs no cudaMalloc / cudaFree and uses no allocating library routine.
 *
 *   Limit: B * (K + 1) <= FMTP_STATIC_VERIFY_MAX_ROWS, otherwise FMTP_ESHAPE and nothing is enqueued.
 *   The first call on a device looks up the array's device address (once per device, with that
 *   device current); make that first call outside any stream capture.
 *   All calls share the one array: it is cleared on `stream` at the start of every call, and two
 *   calls whose work overlaps on the GPU (different streams, no ordering) race on it.
 *   The looked-up address is kept for the life of the process: after a cudaDeviceReset on that device it is
 *   stale, so a process that resets a device must not call this entry point on it again.
 * Arguments, layouts and the meaning of dev_status are those of fastmtp_verify_accept. */
#define FMTP_STATIC_VERIFY_MAX_ROWS 1024
int fastmtp_verify_accept_static(const fmtp_bf16 *target_logits, const int32_t *drafts,
                                 int B, int K, int V,
                                 int32_t *out_accept_len, int32_t *out_bonus, int32_t *out_argmax,
                                 uint32_t *dev_status, void *stream);

/* ---- target decoder step (Sec. 2.1: embedding, transformer layers F, output head W) ----- */

/* Runs M new tokens per sequence through the n_layers-deep target stack with the same
 * decoder-layer kernels as the draft: rows are causal among themselves and sit at cache
 * positions L_b .. L_b+M-1 (L_b = layer_kvs[0].seq_lens[b]); K/V of those positions are
 * written to every layer's cache, seq_lens is not changed. M = 1 is plain decoding,
 * M = K+1 scores [last token, drafts] for verification.
 *
 *   tokens      dev [B, M] int32           layer_kvs   HOST array [n_layers] of fmtp_kv
 *   out_h       dev [B, M, d] bf16 (post-final-norm hidden states) or NULL
 *   out_logits  dev [B, M, V] bf16 full-vocabulary logits or NULL
 *   out_argmax  dev [B, M] int32 greedy token of every row (decided on the bf16-rounded
 *               logits, ties to the lowest id) or NULL
 * Requires B*M <= max_rows (and M <= 8 on the persistent path, M <= 64 on the batched one). Within a path a
 * row's results do not depend on B or M.
 */
int fastmtp_target_step(fmtp_ctx *ctx, const fmtp_target_w *w, const int32_t *tokens,
                        const fmtp_kv *layer_kvs, int B, int M,
                        fmtp_bf16 *out_h, fmtp_bf16 *out_logits, int32_t *out_argmax,
                        uint32_t *dev_status, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* FASTMTP_H */
