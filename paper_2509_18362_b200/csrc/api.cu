// C ABI of the library: context, workspace layout, argument validation and the entry points
// declared in include/fastmtp.h. Host code only marshals; every step of the path runs in the
// kernels of megakernel.cu and verify.cu.
#include "../../include/fastmtp.h"
#include "mega.cuh"
#include "batched.cuh"

#include <cmath>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

using namespace fmtp;

struct fmtp_ctx {
    fmtp_shape shape;
    int n_sm;
    int smem_optin;
    int KC;
    int dp, qp, Fp;
    int max_chunks;
    // workspace
    unsigned char *ws;
    size_t ws_bytes, ws_need;
    Scratch s;
    size_t ctrl_off, ctrl_bytes;
    unsigned long long *vkeys;
    uint32_t *vcounter;
    // staging for the *_host entry points (device side inside the workspace, host side pinned)
    bf16_t *st_h;
    int32_t *st_tok, *st_next, *st_out;
    uint32_t *st_status;
    void *pinned;
    size_t pinned_bytes;
    void *vstage;              // grow-only device staging of fastmtp_verify_accept_host
    size_t vstage_bytes;
    int last_cuda;
    long long launches;
    // batched draft path (more sequences than one persistent-kernel launch takes)
    BatchedShape bsh;
    BatchedWs bws;
    int batched_min;           // calls with at least this many sequences take the batched path (env FMTP_BATCHED_MIN)
    long long tmem_launches;
    int tmem_staging;          // the persistent kernel stages weights through tensor memory where the shape allows (env FMTP_TMEM=1)
    // answers that depend on the geometry only, kept so that the hot calls make no CUDA attribute / occupancy query:
    struct { size_t smem; int grid; } mega_cfg[6];                 // per kernel instantiation: footprint its limit was raised to
    struct { int mode, B, M, G; } group_memo[16];                  // sequences per launch for (mode, B, M)
    int n_group_memo;
    TmapCache tmaps;                                               // tensor maps of the batched path's GEMM operands
    // fmtp_selftest_inject_wait_timeout: the next draft call runs with this wait limit and one wait that cannot end
    unsigned long long inject_limit_ns;
    int inject_which;                                              // 0 none, 1 grid barrier of the persistent kernel, 2 ring stage of a GEMM
};

namespace {

constexpr int kVerifyMaxRows = 4096;
constexpr unsigned long long kDefaultWaitNs = 2000000000ull;     // a device-side wait gives up after 2 s

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct Carver {
    size_t off = 0;
    unsigned char *base = nullptr;
    template <typename T>
    T *take(size_t n) {
        off = align_up(off, 256);
        T *p = base ? reinterpret_cast<T *>(base + off) : nullptr;
        off += n * sizeof(T);
        return p;
    }
};

// Lays the scratch buffers out inside the workspace (base == nullptr: size query only).
size_t layout(fmtp_ctx *c, unsigned char *base) {
    const fmtp_shape &sh = c->shape;
    const int R = sh.max_rows < kMaxRows ? sh.max_rows : kMaxRows;   // rows of one launch
    const int RB = sh.max_rows;                                     // rows of one call (host staging)
    const int d = sh.d;
    const int qdim = sh.n_q_heads * sh.head_dim, kvdim = sh.n_kv_heads * sh.head_dim;
    Carver cv;
    cv.base = base;
    Scratch &s = c->s;
    s.x0 = cv.take<float>((size_t)R * d);
    s.x1 = cv.take<float>((size_t)R * d);
    s.qkv = cv.take<float>((size_t)R * (qdim + 2 * kvdim));
    s.actD_hi = cv.take<bf16_t>((size_t)R * c->dp);  s.actD_lo = cv.take<bf16_t>((size_t)R * c->dp);
    s.actP_hi = cv.take<bf16_t>((size_t)R * c->dp);  s.actP_lo = cv.take<bf16_t>((size_t)R * c->dp);
    s.actH_hi = cv.take<bf16_t>((size_t)R * c->dp);  s.actH_lo = cv.take<bf16_t>((size_t)R * c->dp);
    s.actR_hi = cv.take<bf16_t>((size_t)R * c->dp);  s.actR_lo = cv.take<bf16_t>((size_t)R * c->dp);
    s.actO_hi = cv.take<bf16_t>((size_t)R * c->qp);  s.actO_lo = cv.take<bf16_t>((size_t)R * c->qp);
    s.actF_hi = cv.take<bf16_t>((size_t)R * c->Fp);  s.actF_lo = cv.take<bf16_t>((size_t)R * c->Fp);
    s.ssA = cv.take<float>((size_t)c->n_sm * kMaxRows);
    s.ssB = cv.take<float>((size_t)c->n_sm * kMaxRows);
    s.ssC = cv.take<float>((size_t)c->n_sm * kMaxRows);
    s.ssD = cv.take<float>((size_t)c->n_sm * kMaxRows);
    s.att_part = cv.take<float>((size_t)R * sh.n_q_heads * c->max_chunks * (sh.head_dim + 2));
    // control block, cleared by one memset before every launch
    cv.off = align_up(cv.off, 256);
    c->ctrl_off = cv.off;
    int nkeys = (sh.max_K > 1 ? sh.max_K : 1) * kMaxRows;
    s.keys = cv.take<unsigned long long>((size_t)nkeys);
    s.barrier = cv.take<uint32_t>(1);
    s.abort_flag = cv.take<uint32_t>(1);
    s.status = cv.take<uint32_t>(1);
    cv.off = align_up(cv.off, 256);
    c->ctrl_bytes = cv.off - c->ctrl_off;
    float *cosb = cv.take<float>((size_t)sh.max_ctx * (sh.head_dim / 2));
    float *sinb = cv.take<float>((size_t)sh.max_ctx * (sh.head_dim / 2));
    s.rope_cos = cosb;
    s.rope_sin = sinb;
    c->vkeys = cv.take<unsigned long long>(kVerifyMaxRows);
    c->vcounter = cv.take<uint32_t>(1);
    c->st_h = cv.take<bf16_t>((size_t)RB * d);
    c->st_tok = cv.take<int32_t>((size_t)RB);
    c->st_next = cv.take<int32_t>((size_t)RB);
    c->st_out = cv.take<int32_t>((size_t)RB * (sh.max_K > 1 ? sh.max_K : 1) + 2 * kVerifyMaxRows);
    c->st_status = cv.take<uint32_t>(1);
    size_t off = align_up(cv.off, 256);
    off += batched_layout(c->bws, base ? base + off : nullptr, c->bsh);
    return align_up(off, 256);
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int cuda_fail(fmtp_ctx *c, cudaError_t e) {
    c->last_cuda = (int)e;
    return FMTP_ECUDA;
}

int act_stride(int len) { return ((len + 31) & ~31) + 32; }

// Fills geometry / shared-memory configuration for a call with R rows (M rows per sequence).
int configure(fmtp_ctx *c, MegaParams &p, int mode, int B, int M) {
    const fmtp_shape &sh = c->shape;
    std::memset(&p, 0, sizeof(p));
    p.d = sh.d; p.Hq = sh.n_q_heads; p.Hkv = sh.n_kv_heads; p.dh = sh.head_dim; p.F = sh.ffn; p.V = sh.vocab;
    p.qdim = p.Hq * p.dh; p.kvdim = p.Hkv * p.dh; p.page = sh.page_size;
    p.dp = c->dp; p.qp = c->qp; p.Fp = c->Fp;
    p.eps = sh.rms_eps;
    p.KC = c->KC;
    p.stage_bytes = kTileRows * p.KC * 2;
    {   // a stage also has to hold one 64-token K/V chunk of a KV head
        int kvb = 2 * kAttnChunk * p.dh * 2;
        if (kvb > p.stage_bytes) p.stage_bytes = kvb;
        p.stage_bytes = (p.stage_bytes + 127) & ~127;
    }
    p.max_chunks = c->max_chunks;
    p.max_ctx = sh.max_ctx;
    p.wait_limit_ns = kDefaultWaitNs;
    p.mode = mode; p.B = B; p.M = M; p.R = B * M;
    const int R = p.R, Gq = p.Hq / p.Hkv;
    // attention scratch: the rows' query vectors, then one (o, m, l) buffer per working warp group (the rows of a call
    // are dealt to two groups): [4 warps][8 heads][dh + 2] + 64 words
    size_t attn = (size_t)M * Gq * p.dh * 4 + (size_t)(M > 1 ? 2 : 1) * (4 * 8 * (p.dh + 2) + 64) * 4;
    size_t mrg = ((size_t)2 * c->max_chunks + (size_t)kConsumerThreads + 64) * 4;      // chunk-merge scratch
    if (mrg > attn) attn = mrg;
    size_t actd = (size_t)2 * R * act_stride(mode == 0 ? 2 * p.d : (p.d > p.qdim ? p.d : p.qdim)) * 2;
    size_t actq = (size_t)2 * R * act_stride(p.qdim) * 2;
    size_t base = attn > actd ? attn : actd;
    if (actq > base) base = actq;
    base = align_up(base, 128);
    size_t fixed = mega_fixed_smem(R);
    size_t avail = (size_t)c->smem_optin;
    // the ffn-wide input of the down projection is used once per CTA: it is read from global memory (L2), one
    // stage ahead, and the shared memory goes to a deeper ring
    p.scratch_smem = (int)base;
    // tensor memory as a second staging level: full-width stages only (every K a multiple of the stage width), at most
    // four activation rows, the down projection's slice ring inside the staging area
    p.use_tmem = c->tmem_staging && R <= 4 && p.KC == 512 && p.stage_bytes == kTileRows * 512 * 2 && p.d % 512 == 0 &&
                 p.qdim % 512 == 0 && p.F % 512 == 0 && (size_t)16 * R * 512 <= base;
    size_t ring_off = fixed + base;
    if (p.use_tmem) ring_off = align_up(ring_off, 1024) + 1024;        // as mega_smem_bytes lays it out
    int ns = ring_off < avail ? (int)((avail - ring_off) / p.stage_bytes) : 0;
    if (ns > kMaxStages) ns = kMaxStages;
    if (ns < 2) return FMTP_ESHAPE;
    p.n_stages = ns;
    p.s = c->s;
    return FMTP_OK;
}

void set_layer(LayerPtrs &dst, const fmtp_layer_w &w) {
    dst.g_in = w.g_in; dst.wq = w.wq; dst.wk = w.wk; dst.wv = w.wv; dst.wo = w.wo;
    dst.g_post = w.g_post; dst.w_gate = w.w_gate; dst.w_up = w.w_up; dst.w_down = w.w_down;
}
bool layer_ok(const fmtp_layer_w &w) {
    const void *ps[] = {w.g_in, w.wq, w.wk, w.wv, w.wo, w.g_post, w.w_gate, w.w_up, w.w_down};
    for (const void *q : ps) if (!q || !aligned16(q)) return false;
    return true;
}
bool kv_ok(const fmtp_kv &kv) {
    return kv.k_pages && kv.v_pages && kv.block_table && kv.seq_lens && kv.num_pages > 0 && kv.max_pages_per_seq > 0 &&
           aligned16(kv.k_pages) && aligned16(kv.v_pages);
}
void set_kv(KvPtrs &dst, const fmtp_kv &kv) {
    dst.k_pages = kv.k_pages; dst.v_pages = kv.v_pages; dst.block_table = kv.block_table;
    dst.seq_lens = kv.seq_lens; dst.num_pages = kv.num_pages; dst.max_pages = kv.max_pages_per_seq;
}

int launch_mega(fmtp_ctx *c, MegaParams &p, cudaStream_t st) {
    cudaError_t e = cudaMemsetAsync(c->ws + c->ctrl_off, 0, c->ctrl_bytes, st);
    if (e != cudaSuccess) return cuda_fail(c, e);
    int err = 0;
    size_t smem = mega_smem_bytes(p);
    auto &cfg = c->mega_cfg[mega_kernel_index(p)];
    if (cfg.smem != smem || cfg.grid < 1) {       // first call with this footprint: raise the kernel's limit, ask the occupancy
        int grid = mega_max_grid(p, smem, &err);
        if (err) return cuda_fail(c, (cudaError_t)err);
        if (grid < 1) return FMTP_ESHAPE;
        cfg.smem = smem;
        cfg.grid = grid > c->n_sm ? c->n_sm : grid;
    }
    err = mega_launch(p, cfg.grid, st);
    if (err) return cuda_fail(c, (cudaError_t)err);
    c->launches++;
    if (p.use_tmem) c->tmem_launches++;
    return FMTP_OK;
}

// Sequences per launch for a call of B sequences with M rows each: a call with more rows than one
// launch takes runs as several launches over groups of whole sequences. The largest group is the
// one whose input vectors still leave a ring of three stages (two at worst); 0 if even one
// sequence does not fit.
int group_size(fmtp_ctx *c, int mode, int B, int M) {
    for (int i = 0; i < c->n_group_memo; ++i)
        if (c->group_memo[i].mode == mode && c->group_memo[i].B == B && c->group_memo[i].M == M) return c->group_memo[i].G;
    int gmax = kMaxRows / M;
    if (gmax > B) gmax = B;
    int G = 0;
    for (int want = 3; want >= 2 && G == 0; --want)
        for (int g = gmax; g >= 1; --g) {
            MegaParams tmp;
            if (configure(c, tmp, mode, g, M) == FMTP_OK && tmp.n_stages >= want) { G = g; break; }
        }
    if (c->n_group_memo < 16) {
        auto &m = c->group_memo[c->n_group_memo++];
        m.mode = mode; m.B = B; m.M = M; m.G = G;
    }
    return G;
}

int status_to_code(uint32_t st) {
    if (st & FMTP_DEV_TIMEOUT) return FMTP_ETIMEOUT;
    if (st) return FMTP_EBOUNDS;
    return FMTP_OK;
}

}  // namespace

extern "C" {

const char *fmtp_strerror(int status) {
    switch (status) {
        case FMTP_OK: return "ok";
        case FMTP_EINVAL: return "invalid argument (null, misaligned or non-positive)";
        case FMTP_ESHAPE: return "shape not supported by the kernels";
        case FMTP_EUNSUPPORTED: return "not implemented in this build";
        case FMTP_ENOMEM: return "workspace missing or too small";
        case FMTP_ECUDA: return "CUDA runtime error (see fmtp_last_cuda_error)";
        case FMTP_ETIMEOUT: return "a bounded device-side wait gave up";
        case FMTP_EBOUNDS: return "a kernel clamped an out-of-range id, page or position";
        default: return "unknown status";
    }
}

int fmtp_create(const fmtp_shape *sh, fmtp_ctx **out) {
    if (!sh || !out) return FMTP_EINVAL;
    *out = nullptr;
    if (sh->d <= 0 || sh->n_q_heads <= 0 || sh->n_kv_heads <= 0 || sh->ffn <= 0 || sh->vocab <= 0 ||
        sh->page_size <= 0 || sh->max_rows <= 0 || sh->max_ctx <= 0 || sh->max_K < 0 || sh->n_layers < 0)
        return FMTP_EINVAL;
    if (sh->head_dim != 64 && sh->head_dim != 128) return FMTP_ESHAPE;
    if (sh->d % 64 || sh->ffn % 16 || sh->n_q_heads % sh->n_kv_heads || sh->n_q_heads / sh->n_kv_heads > 8 ||
        sh->max_rows > 4096 || sh->n_layers > kMaxLayers)
        return FMTP_ESHAPE;
    int dev = 0, major = 0, sms = 0, optin = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    if (e != cudaSuccess || major < 10) return FMTP_ECUDA;
    fmtp_ctx *c = new (std::nothrow) fmtp_ctx();
    if (!c) return FMTP_ENOMEM;
    std::memset(c, 0, sizeof(*c));
    c->shape = *sh;
    c->n_sm = sms;
    c->smem_optin = optin;
    c->KC = (sh->d % 512 == 0) ? 512 : (sh->d % 256 == 0) ? 256 : (sh->d % 128 == 0) ? 128 : 64;
    c->dp = (sh->d + 31) & ~31;
    c->qp = (sh->n_q_heads * sh->head_dim + 31) & ~31;
    c->Fp = (sh->ffn + 31) & ~31;
    c->max_chunks = (sh->max_ctx + kAttnChunk - 1) / kAttnChunk;
    c->bsh.d = sh->d; c->bsh.Hq = sh->n_q_heads; c->bsh.Hkv = sh->n_kv_heads; c->bsh.dh = sh->head_dim; c->bsh.F = sh->ffn;
    c->bsh.V = sh->vocab; c->bsh.page = sh->page_size; c->bsh.max_ctx = sh->max_ctx; c->bsh.max_K = sh->max_K;
    c->bsh.max_rows = sh->max_rows; c->bsh.eps = sh->rms_eps;
    c->ws_need = layout(c, nullptr);
    const int g1 = group_size(c, 0, kMaxRows, 1);
    if (g1 < 1) { delete c; return FMTP_ESHAPE; }
    // Which path a call takes depends on its number of sequences only (so a sequence scored with 1 or with K+1
    // rows takes the same path and gives the same bits). Small models: the persistent kernel as long as the
    // sequences fit one launch. Models that stream >= 256 MB of layer weights per step: the batched path from
    // three sequences on (measured at the 7B shape: 180 / 182 us per step against 181 / 208 us at 3 / 4 sequences).
    c->batched_min = g1 + 1;
    {
        const double qd = (double)sh->n_q_heads * sh->head_dim, kvd = (double)sh->n_kv_heads * sh->head_dim;
        const double layer_bytes = 2.0 * (2.0 * sh->d * sh->d + sh->d * (qd + 2 * kvd) + qd * sh->d + 3.0 * sh->d * sh->ffn);
        if (layer_bytes >= 256e6 && c->batched_min > 3) c->batched_min = 3;
    }
    if (const char *v = std::getenv("FMTP_BATCHED_MIN")) { int n = std::atoi(v); if (n >= 1) c->batched_min = n; }
    c->tmem_staging = 0;       // measured slower than the plain ring so far: opt-in
    if (const char *v = std::getenv("FMTP_TMEM")) c->tmem_staging = std::atoi(v) != 0;
    c->pinned_bytes = (size_t)sh->max_rows * sh->d * 2 + (size_t)sh->max_rows * 4 * (3 + (sh->max_K > 1 ? sh->max_K : 1)) +
                      2 * kVerifyMaxRows * 4 + 256;
    e = cudaMallocHost(&c->pinned, c->pinned_bytes);
    if (e != cudaSuccess) { delete c; return FMTP_ECUDA; }
    *out = c;
    return FMTP_OK;
}

int fmtp_selftest_inject_wait_timeout(fmtp_ctx *c, int limit_ms, int which) {
    if (!c || (which != 1 && which != 2)) return FMTP_EINVAL;
    if (limit_ms < 1 || limit_ms > 1000) return FMTP_EINVAL;      // bounded on purpose
    c->inject_limit_ns = (unsigned long long)limit_ms * 1000000ull;
    c->inject_which = which;
    return FMTP_OK;
}

int fmtp_destroy(fmtp_ctx *c) {
    if (!c) return FMTP_EINVAL;
    if (c->pinned) cudaFreeHost(c->pinned);
    if (c->vstage) cudaFree(c->vstage);
    delete c;
    return FMTP_OK;
}

size_t fmtp_workspace_bytes(const fmtp_ctx *c) { return c ? c->ws_need : 0; }
int fmtp_last_cuda_error(const fmtp_ctx *c) { return c ? c->last_cuda : 0; }
long long fmtp_launch_count(const fmtp_ctx *c) { return c ? c->launches : 0; }
long long fmtp_tmem_launch_count(const fmtp_ctx *c) { return c ? c->tmem_launches : 0; }

int fmtp_set_workspace(fmtp_ctx *c, void *dev, size_t bytes) {
    if (!c || !dev) return FMTP_EINVAL;
    if ((reinterpret_cast<uintptr_t>(dev) & 255u) != 0) return FMTP_EINVAL;
    if (bytes < c->ws_need) return FMTP_ENOMEM;
    c->ws = static_cast<unsigned char *>(dev);
    c->ws_bytes = bytes;
    layout(c, c->ws);
    cudaError_t e = cudaMemset(dev, 0, c->ws_need);
    if (e != cudaSuccess) return cuda_fail(c, e);
    // rotary table: angle(pos, i) = pos * theta^(-2i/dh), evaluated in double, stored as fp32
    const fmtp_shape &sh = c->shape;
    const int half = sh.head_dim / 2;
    std::vector<float> cs((size_t)sh.max_ctx * half), sn((size_t)sh.max_ctx * half);
    for (int i = 0; i < half; ++i) {
        double inv = std::pow((double)sh.rope_theta, -2.0 * i / sh.head_dim);
        for (int pos = 0; pos < sh.max_ctx; ++pos) {
            double a = (double)pos * inv;
            cs[(size_t)pos * half + i] = (float)std::cos(a);
            sn[(size_t)pos * half + i] = (float)std::sin(a);
        }
    }
    e = cudaMemcpy(const_cast<float *>(c->s.rope_cos), cs.data(), cs.size() * 4, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(const_cast<float *>(c->s.rope_sin), sn.data(), sn.size() * 4, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) return cuda_fail(c, e);
    return FMTP_OK;
}

}  // extern "C"

namespace {

// Everything fastmtp_draft can check on the host, before anything is enqueued.
int check_draft_args(const fmtp_ctx *c, const fmtp_mtp_w *w, const void *h_last, const void *tok_last, int max_ext,
                     const fmtp_kv *kv, int B, int K, const int32_t *subset, int N, const void *out_drafts, const void *out_h) {
    if (!c || !w || !h_last || !tok_last || !kv || !out_drafts) return FMTP_EINVAL;
    if (!c->ws) return FMTP_ENOMEM;
    if (B <= 0 || K <= 0 || max_ext <= 0) return FMTP_EINVAL;
    if ((long long)B * max_ext > c->shape.max_rows || K > c->shape.max_K || max_ext > kBatchRows) return FMTP_ESHAPE;
    if (subset && (N <= 0 || N > c->shape.vocab)) return FMTP_EINVAL;
    if (!w->embed || !w->lm_head || !w->g_hnorm || !w->g_enorm || !w->w_proj || !w->g_final) return FMTP_EINVAL;
    if (!aligned16(w->embed) || !aligned16(w->lm_head) || !aligned16(w->g_hnorm) || !aligned16(w->g_enorm) ||
        !aligned16(w->w_proj) || !aligned16(w->g_final) || !aligned16(h_last) || !layer_ok(w->layer) || !kv_ok(*kv))
        return FMTP_EINVAL;
    if (out_h && !aligned16(out_h)) return FMTP_EINVAL;
    return FMTP_OK;
}

}  // namespace

extern "C" {

int fastmtp_draft(fmtp_ctx *c, const fmtp_mtp_w *w, const fmtp_bf16 *h_last, const int32_t *tok_last,
                  const int32_t *n_ext, int max_ext, const fmtp_kv *kv, int B, int K, const int32_t *subset, int N,
                  int32_t *out_drafts, fmtp_bf16 *out_h, float *out_logits, uint32_t *dev_status, void *stream) {
    int rc = check_draft_args(c, w, h_last, tok_last, max_ext, kv, B, K, subset, N, out_drafts, out_h);
    if (rc) return rc;
    const int Neff = subset ? N : c->shape.vocab;
    const int d = c->shape.d;
    // the persistent kernel takes the call if its sequences are few and the extend rows of a group fit one launch
    const int G = B < c->batched_min ? group_size(c, 0, B, max_ext) : 0;
    if (G < 1) {
        // groups of up to 64 sequences, every weight streamed once per step and group by the tensor-core GEMM path
        for (int b0 = 0; b0 < B; b0 += kBatchRows) {
            BatchedCall bc;
            std::memset(&bc, 0, sizeof(bc));
            bc.sh = c->bsh; bc.ws = c->bws;
            bc.rope_cos = c->s.rope_cos; bc.rope_sin = c->s.rope_sin;
            bc.n_sm = c->n_sm; bc.smem_optin = c->smem_optin; bc.cache = &c->tmaps;
            bc.wait_limit_ns = kDefaultWaitNs;
            if (c->inject_which == 2) { bc.wait_limit_ns = c->inject_limit_ns; bc.inject_gemm_timeout = 1; c->inject_which = 0; }
            bc.B = (B - b0 < kBatchRows) ? B - b0 : kBatchRows;
            bc.K = K; bc.N = Neff; bc.ids = subset;
            bc.M0 = max_ext; bc.n_ext = n_ext ? n_ext + b0 : nullptr;
            bc.h_last = h_last + (size_t)b0 * max_ext * d;
            bc.tok_last = tok_last + (size_t)b0 * max_ext;
            bc.out_drafts = out_drafts + (size_t)b0 * K;
            bc.out_h = out_h ? out_h + (size_t)b0 * K * d : nullptr;
            bc.out_logits = out_logits ? out_logits + (size_t)b0 * K * Neff : nullptr;
            bc.user_status = dev_status;
            bc.embed = w->embed; bc.lm_head = w->lm_head; bc.g_hnorm = w->g_hnorm; bc.g_enorm = w->g_enorm;
            bc.w_proj = w->w_proj; bc.g_final = w->g_final;
            set_layer(bc.layer, w->layer);
            set_kv(bc.kv, *kv);
            bc.kv.block_table += (size_t)b0 * kv->max_pages_per_seq;
            bc.kv.seq_lens += b0;
            int err = batched_draft(bc, static_cast<cudaStream_t>(stream), &c->launches);
            if (err) return cuda_fail(c, (cudaError_t)err);
        }
        return FMTP_OK;
    }
    for (int b0 = 0; b0 < B; b0 += G) {
        const int Bg = (B - b0 < G) ? B - b0 : G;
        MegaParams p;
        rc = configure(c, p, 0, Bg, max_ext);
        if (rc) return rc;
        p.K = K;
        p.N = Neff;
        p.ids = subset;
        if (c->inject_which == 1) { p.wait_limit_ns = c->inject_limit_ns; p.extra_arrivals = 1; c->inject_which = 0; }
        p.h_last = h_last + (size_t)b0 * max_ext * d;
        p.tokens = tok_last + (size_t)b0 * max_ext;
        p.n_ext = n_ext ? n_ext + b0 : nullptr;
        p.out_tokens = out_drafts + (size_t)b0 * K;
        p.out_h = out_h ? out_h + (size_t)b0 * K * d : nullptr;
        p.out_logits_f32 = out_logits ? out_logits + (size_t)b0 * K * Neff : nullptr;
        p.user_status = dev_status;
        p.embed = w->embed; p.lm_head = w->lm_head; p.g_hnorm = w->g_hnorm; p.g_enorm = w->g_enorm;
        p.w_proj = w->w_proj; p.g_final = w->g_final;
        set_layer(p.layers[0], w->layer);
        set_kv(p.kvs[0], *kv);
        p.kvs[0].block_table += (size_t)b0 * kv->max_pages_per_seq;
        p.kvs[0].seq_lens += b0;
        rc = launch_mega(c, p, static_cast<cudaStream_t>(stream));
        if (rc) return rc;
    }
    return FMTP_OK;
}

int fastmtp_draft_host(fmtp_ctx *c, const fmtp_mtp_w *w, const fmtp_bf16 *h_host, const int32_t *tok_host,
                       const int32_t *n_ext_host, int max_ext, const fmtp_kv *kv, int B, int K, const int32_t *subset, int N,
                       int32_t *out_host, void *stream) {
    if (!c || !out_host) return FMTP_EINVAL;
    // every check of the device call first: on a negative return nothing has been enqueued
    int rc = check_draft_args(c, w, c->st_h, tok_host, max_ext, kv, B, K, subset, N, out_host, nullptr);
    if (rc) return rc;
    if (!h_host) return FMTP_EINVAL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t rows = (size_t)B * max_ext;
    const size_t hb = rows * c->shape.d * 2, tb = rows * 4, nb = n_ext_host ? (size_t)B * 4 : 0, ob = (size_t)B * K * 4;
    unsigned char *pin = static_cast<unsigned char *>(c->pinned);
    std::memcpy(pin, h_host, hb);
    std::memcpy(pin + hb, tok_host, tb);
    if (nb) std::memcpy(pin + hb + tb, n_ext_host, nb);
    cudaError_t e = cudaMemcpyAsync(c->st_h, pin, hb, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(c->st_tok, pin + hb, tb, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess && nb) e = cudaMemcpyAsync(c->st_next, pin + hb + tb, nb, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemsetAsync(c->st_status, 0, 4, st);
    if (e != cudaSuccess) return cuda_fail(c, e);
    rc = fastmtp_draft(c, w, c->st_h, c->st_tok, nb ? c->st_next : nullptr, max_ext, kv, B, K, subset, N, c->st_out, nullptr,
                       nullptr, c->st_status, st);
    if (rc) return rc;
    unsigned char *po = pin + align_up(hb + tb + nb, 16);
    e = cudaMemcpyAsync(po, c->st_out, ob, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(po + ob, c->st_status, 4, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(c, e);
    std::memcpy(out_host, po, ob);
    uint32_t stw;
    std::memcpy(&stw, po + ob, 4);
    return status_to_code(stw);
}

int fastmtp_verify_accept(fmtp_ctx *c, const fmtp_bf16 *logits, const int32_t *drafts, int B, int K, int V,
                          int32_t *out_accept, int32_t *out_bonus, int32_t *out_argmax, uint32_t *dev_status,
                          void *stream) {
    if (!c || !logits || !out_accept || !out_bonus || (K > 0 && !drafts)) return FMTP_EINVAL;
    if (!c->ws) return FMTP_ENOMEM;
    if (B <= 0 || K < 0 || V <= 0) return FMTP_EINVAL;
    if ((long long)B * (K + 1) > kVerifyMaxRows) return FMTP_ESHAPE;
    int err = verify_launch(logits, drafts, B, K, V, out_accept, out_bonus, out_argmax, c->vkeys, c->vcounter,
                            c->s.status, dev_status, c->n_sm, static_cast<cudaStream_t>(stream));
    if (err) return cuda_fail(c, (cudaError_t)err);
    c->launches++;
    return FMTP_OK;
}

int fastmtp_accept_ids(fmtp_ctx *c, const int32_t *target_argmax, const int32_t *drafts, int B, int K,
                       int32_t *out_accept, int32_t *out_bonus, void *stream) {
    if (!c || !target_argmax || !out_accept || !out_bonus || (K > 0 && !drafts)) return FMTP_EINVAL;
    if (B <= 0 || K < 0) return FMTP_EINVAL;
    int err = accept_ids_launch(target_argmax, drafts, B, K, out_accept, out_bonus, static_cast<cudaStream_t>(stream));
    if (err) return cuda_fail(c, (cudaError_t)err);
    c->launches++;
    return FMTP_OK;
}

int fastmtp_verify_accept_host(fmtp_ctx *c, const fmtp_bf16 *logits_host, const int32_t *drafts_host, int B, int K,
                               int V, int32_t *accept_host, int32_t *bonus_host, void *stream) {
    if (!c || !logits_host || !accept_host || !bonus_host || (K > 0 && !drafts_host)) return FMTP_EINVAL;
    if (!c->ws) return FMTP_ENOMEM;
    if (B <= 0 || K < 0 || V <= 0) return FMTP_EINVAL;
    if ((long long)B * (K + 1) > kVerifyMaxRows) return FMTP_ESHAPE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    size_t lb = (size_t)B * (K + 1) * V * 2, db = (size_t)B * K * 4;
    size_t need = align_up(lb, 256) + align_up(db + 16, 256);
    cudaError_t e = cudaSuccess;
    if (need > c->vstage_bytes) {   // the one device allocation this library makes (grow-only, freed in destroy)
        if (c->vstage) cudaFree(c->vstage);
        c->vstage = nullptr;
        c->vstage_bytes = 0;
        e = cudaMalloc(&c->vstage, need);
        if (e != cudaSuccess) return cuda_fail(c, e);
        c->vstage_bytes = need;
    }
    unsigned char *dv = static_cast<unsigned char *>(c->vstage);
    int32_t *ddr = reinterpret_cast<int32_t *>(dv + align_up(lb, 256));
    e = cudaMemcpyAsync(dv, logits_host, lb, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess && db) e = cudaMemcpyAsync(ddr, drafts_host, db, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemsetAsync(c->st_status, 0, 4, st);
    if (e != cudaSuccess) return cuda_fail(c, e);
    int32_t *dacc = c->st_out, *dbon = c->st_out + kVerifyMaxRows;
    int rc = fastmtp_verify_accept(c, reinterpret_cast<const fmtp_bf16 *>(dv), ddr, B, K, V, dacc, dbon, nullptr,
                                   c->st_status, st);
    if (rc) return rc;
    unsigned char *pin = static_cast<unsigned char *>(c->pinned);
    e = cudaMemcpyAsync(pin, dacc, (size_t)B * 4, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(pin + (size_t)B * 4, dbon, (size_t)B * 4, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(pin + (size_t)B * 8, c->st_status, 4, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(c, e);
    std::memcpy(accept_host, pin, (size_t)B * 4);
    std::memcpy(bonus_host, pin + (size_t)B * 4, (size_t)B * 4);
    uint32_t stw;
    std::memcpy(&stw, pin + (size_t)B * 8, 4);
    return status_to_code(stw);
}

int fastmtp_target_step(fmtp_ctx *c, const fmtp_target_w *w, const int32_t *tokens, const fmtp_kv *kvs, int B, int M,
                        fmtp_bf16 *out_h, fmtp_bf16 *out_logits, int32_t *out_argmax, uint32_t *dev_status,
                        void *stream) {
    if (!c || !w || !tokens || !kvs) return FMTP_EINVAL;
    if (!c->ws) return FMTP_ENOMEM;
    if (B <= 0 || M <= 0) return FMTP_EINVAL;
    const int nl = c->shape.n_layers;
    if (nl <= 0 || (long long)B * M > c->shape.max_rows) return FMTP_ESHAPE;
    if (!w->embed || !w->lm_head || !w->g_final || !w->layers) return FMTP_EINVAL;
    if (!aligned16(w->embed) || !aligned16(w->lm_head) || !aligned16(w->g_final)) return FMTP_EINVAL;
    for (int l = 0; l < nl; ++l) if (!layer_ok(w->layers[l]) || !kv_ok(kvs[l])) return FMTP_EINVAL;
    const int V = c->shape.vocab, d = c->shape.d;
    if (B >= c->batched_min && M <= kBatchRows) {
        // more rows than one launch of the persistent kernel takes: groups of whole sequences, up to 64 rows each,
        // every layer's weights streamed once per group by the tensor-core GEMM path
        if ((out_h && !aligned16(out_h))) return FMTP_EINVAL;
        const int Gs = kBatchRows / M;
        std::vector<LayerPtrs> layers(nl);
        std::vector<KvPtrs> lkv(nl);
        for (int b0 = 0; b0 < B; b0 += Gs) {
            const int Bg = (B - b0 < Gs) ? B - b0 : Gs;
            BatchedTargetCall tc;
            std::memset(&tc, 0, sizeof(tc));
            tc.sh = c->bsh; tc.ws = c->bws;
            tc.rope_cos = c->s.rope_cos; tc.rope_sin = c->s.rope_sin;
            tc.n_sm = c->n_sm; tc.smem_optin = c->smem_optin; tc.cache = &c->tmaps; tc.wait_limit_ns = kDefaultWaitNs;
            tc.B = Bg; tc.M = M; tc.n_layers = nl;
            tc.tokens = tokens + (size_t)b0 * M;
            tc.out_h = out_h ? out_h + (size_t)b0 * M * d : nullptr;
            tc.out_logits = out_logits ? out_logits + (size_t)b0 * M * V : nullptr;
            tc.out_argmax = out_argmax ? out_argmax + (size_t)b0 * M : nullptr;
            tc.user_status = dev_status;
            tc.embed = w->embed; tc.lm_head = w->lm_head; tc.g_final = w->g_final;
            for (int l = 0; l < nl; ++l) {
                set_layer(layers[l], w->layers[l]);
                set_kv(lkv[l], kvs[l]);
                lkv[l].block_table += (size_t)b0 * kvs[l].max_pages_per_seq;
                lkv[l].seq_lens += b0;
            }
            tc.layers = layers.data();
            tc.kvs = lkv.data();
            int err = batched_target(tc, static_cast<cudaStream_t>(stream), &c->launches);
            if (err) return cuda_fail(c, (cudaError_t)err);
        }
        return FMTP_OK;
    }
    if (M > kMaxRows) return FMTP_ESHAPE;                // the rows of one sequence share a launch
    const int G = group_size(c, 1, B, M);
    if (G < 1) return FMTP_ESHAPE;
    for (int b0 = 0; b0 < B; b0 += G) {
        const int Bg = (B - b0 < G) ? B - b0 : G;
        MegaParams p;
        int rc = configure(c, p, 1, Bg, M);
        if (rc) return rc;
        p.K = 1;
        p.n_layers = nl;
        p.N = V;
        p.ids = nullptr;
        p.tokens = tokens + (size_t)b0 * M;
        p.out_tokens = out_argmax ? out_argmax + (size_t)b0 * M : nullptr;
        p.out_h = out_h ? out_h + (size_t)b0 * M * d : nullptr;
        p.out_logits_bf16 = out_logits ? out_logits + (size_t)b0 * M * V : nullptr;
        p.user_status = dev_status;
        p.embed = w->embed; p.lm_head = w->lm_head; p.g_final = w->g_final;
        for (int l = 0; l < nl; ++l) {
            set_layer(p.layers[l], w->layers[l]);
            set_kv(p.kvs[l], kvs[l]);
            p.kvs[l].block_table += (size_t)b0 * kvs[l].max_pages_per_seq;
            p.kvs[l].seq_lens += b0;
        }
        rc = launch_mega(c, p, static_cast<cudaStream_t>(stream));
        if (rc) return rc;
    }
    return FMTP_OK;
}

}  // extern "C"
