// Parameter block and launch interface of the persistent decoder kernel.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace fmtp {

constexpr int kMaxLayers = 64;
constexpr int kMaxRows = 8;          // activation rows (batch x rows-per-sequence) per launch
constexpr int kConsumerWarps = 8;
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kProducerWarps = 4;       // one warpgroup
constexpr int kThreads = kConsumerThreads + kProducerWarps * 32;
// Registers per thread after the warpgroups split (setmaxnreg): the kernel launches with
// 65536 / 384 = 168 per thread; the producer warpgroup hands 72 x 128 back to the two consumer ones.
constexpr int kProducerRegs = 96;
constexpr int kConsumerRegs = 200;
constexpr int kTileRows = 32;        // weight rows per pipeline stage (two 16-row MMA tiles)
constexpr int kAttnChunk = 64;       // context tokens per attention work item
constexpr int kMaxStages = 8;
// Second staging level in tensor memory (see the kernel): a fourth warpgroup (one warp of it works) moves every landed
// 32 KB weight stage from the shared-memory ring into one of eight 64-column slots of the SM's 256 KB tensor memory,
// the consumers read their fragments from there. 512 threads launch with 128 registers each; the mover's warpgroup
// and the producers hand back what takes the consumers to 192.
constexpr int kTmThreads = 512;
constexpr int kTmMoverRegs = 32;
constexpr int kTmConsumerRegs = 192;
constexpr int kTmSlots = 8;
constexpr int kTmSlotCols = 64;

typedef uint16_t bf16_t;

struct LayerPtrs {
    const bf16_t *g_in, *wq, *wk, *wv, *wo, *g_post, *w_gate, *w_up, *w_down;
};
struct KvPtrs {
    bf16_t *k_pages, *v_pages;
    const int32_t *block_table, *seq_lens;
    int32_t num_pages, max_pages;
};

// Global scratch carved out of the caller's workspace. "hi/lo" buffers hold an fp32 value as
// two bf16 numbers (hi = bf16(x), lo = bf16(x - hi)) in two separate row-major arrays.
struct Scratch {
    float *x0, *x1;                   // [R][d] residual stream before / after attention
    float *qkv;                       // [R][qdim + 2 kvdim]
    bf16_t *actD_hi, *actD_lo;        // [R][dp]  input of QKV            (x * g_in, unnormalised)
    bf16_t *actP_hi, *actP_lo;        // [R][dp]  input of gate/up        (x * g_post)
    bf16_t *actH_hi, *actH_lo;        // [R][dp]  input of the head       (x * g_final)
    bf16_t *actR_hi, *actR_lo;        // [R][dp]  recursed hidden state   (x * g_final * g_hnorm)
    bf16_t *actO_hi, *actO_lo;        // [R][qp]  attention output
    bf16_t *actF_hi, *actF_lo;        // [R][Fp]  SwiGLU activation
    float *ssA, *ssB, *ssC, *ssD;     // [grid][8] per-CTA partial sums of squares
    float *att_part;                  // [R][Hq][max_chunks][dh + 2] (o, m, l) per context chunk
    unsigned long long *keys;         // [max_K or 1][8] argmax keys
    const float *rope_cos, *rope_sin; // [max_ctx][dh/2]
    uint32_t *barrier;                // grid barrier counter
    uint32_t *abort_flag;             // set when a bounded wait gave up
    uint32_t *status;                 // internal status word (OR of FMTP_DEV_*), merged to the caller's
};

struct MegaParams {
    // geometry
    int d, Hq, Hkv, dh, F, V, qdim, kvdim, page;
    int dp, qp, Fp;                   // padded row lengths of the hi/lo buffers (multiples of 32)
    float eps;
    int KC;                           // k elements per pipeline stage
    int n_stages, stage_bytes;        // ring geometry: stages of stage_bytes (32 weight rows x KC elements, or one K/V chunk)
    int scratch_smem;                 // bytes of the per-phase shared scratch region
    int max_chunks;                   // capacity of att_part's chunk dimension
    int max_ctx;                      // rows of the rotary table
    unsigned long long wait_limit_ns; // every device-side wait gives up after this long (2 s outside the self-test)
    int extra_arrivals;               // self-test only: arrivals the grid barrier expects beyond the CTAs that exist
    int use_tmem;                     // weight stages pass through tensor memory (stage = 32 rows x 512, every K a multiple of 512, R <= 4)
    // call
    int mode;                         // 0: MTP draft, 1: target step
    int B, M, R;                      // sequences, rows per sequence (draft: extend rows of step 0), R = B*M
    int K;                            // draft steps (mode 0)
    int n_layers;                     // mode 1
    int N;                            // head rows (subset size or V)
    const int32_t *ids;               // subset or NULL
    const bf16_t *h_last;             // [B][M][d] (mode 0)
    const int32_t *tokens;            // mode 0: tok_last [B][M]; mode 1: [B][M]
    const int32_t *n_ext;             // mode 0: [B] extend rows per sequence (1..M), NULL = M for every sequence
    int32_t *out_tokens;              // mode 0: drafts [B][K]; mode 1: argmax [B][M] or NULL
    bf16_t *out_h;                    // mode 0: [B][K][d]; mode 1: [B][M][d]; or NULL
    float *out_logits_f32;            // mode 0 debug [B][K][N] or NULL
    bf16_t *out_logits_bf16;          // mode 1 [R][V] or NULL
    uint32_t *user_status;            // caller's status word or NULL
    // weights
    const bf16_t *embed, *lm_head, *g_hnorm, *g_enorm, *w_proj, *g_final;
    LayerPtrs layers[kMaxLayers];
    KvPtrs kvs[kMaxLayers];
    Scratch s;
};

// Shared-memory bytes the kernel needs for these parameters.
size_t mega_smem_bytes(const MegaParams &p);
// Shared memory used besides the per-phase scratch and the ring, for R activation rows.
size_t mega_fixed_smem(int R);
// Cooperative launch on `stream` with `grid` CTAs (one per SM). The kernel's shared-memory limit must have been
// raised to this footprint by mega_max_grid. Returns the cudaError_t.
int mega_launch(const MegaParams &p, int grid, cudaStream_t stream);
// Raises the shared-memory limit of the kernel these parameters select and returns the largest co-resident
// grid for this footprint on the current device. The answer depends on (kernel, footprint) only: callers cache it.
int mega_max_grid(const MegaParams &p, size_t smem_bytes, int *err);
// Which of the kernel's instantiations (head dimension, more than four activation rows, tensor-memory staging) the
// parameters select: 0..5.
int mega_kernel_index(const MegaParams &p);

// Verification kernel (verify.cu).
int verify_launch(const bf16_t *logits, const int32_t *drafts, int B, int K, int V,
                  int32_t *accept_len, int32_t *bonus, int32_t *out_argmax,
                  unsigned long long *keys, uint32_t *counter, uint32_t *status, uint32_t *user_status,
                  int n_sm, cudaStream_t stream);

// Acceptance on token ids (verify.cu): accept_len / bonus from the target's per-row greedy tokens [B][K+1].
int accept_ids_launch(const int32_t *target_argmax, const int32_t *drafts, int B, int K, int32_t *accept_len, int32_t *bonus,
                      cudaStream_t stream);

}  // namespace fmtp
