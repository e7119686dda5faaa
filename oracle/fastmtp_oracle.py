"""CPU oracle for the FastMTP draft / verify hot path.  TEST INFRASTRUCTURE ONLY.

A plain, slow, float64 numpy statement of what the path computes, written from the paper:
the recursive K-step draft of one position-shared MTP head (Sec. 2.1 "Architecture Design",
Sec. 2.3 "Drafting phase"), the compressed-vocabulary output head (Sec. 2.2, Eq. 3), greedy
verification with strict acceptance (Sec. 2.3 "Verification phase"; greedy decoding per
Sec. 3.1 "Evaluation Method"), the target decoder stack those steps reuse, and the plain /
speculative decoding loops used to check losslessness (Sec. 3.1 "Hardware Settings" note:
outputs identical to vanilla autoregressive decoding).

Only tests, the smoke check and the benchmark's cpu-baseline leg may import this file. It
shares no code with the CUDA path and imports nothing from the product package; inputs are
plain numpy arrays (bf16 tensors as uint16 bit patterns) and duck-typed shape objects with
attributes d, n_q_heads, n_kv_heads, head_dim, ffn, vocab, rms_eps, rope_theta, page_size.

Precision: every value is float64. Tensors that are bf16 by definition are rounded (nearest
even) exactly where they are stored: weights (given), KV-cache entries, hidden states
crossing the library boundary. The argmax decision is taken on logits rounded to float32,
the precision the kernels decide in. There is no blocking, fusion or reordering.

Readings of points the paper leaves open (the paper only says the head has the DeepSeek-V3
MTP architecture): input to the projection is [RMSNorm_h(h) ; RMSNorm_e(Emb(t))] with a
bias-free d x 2d matrix; the block is a pre-norm decoder layer (RMSNorm, rotary GQA
attention without biases scaled by 1/sqrt(dh), SwiGLU MLP); rotary pairs are (i, i+dh/2)
with inverse frequency theta^(-2i/dh); keys are cached after rotation; the hidden state that
is recursed is the post-final-norm vector that also feeds the output head; ties in an argmax
go to the lowest token id and NaN never wins.

Pins (tests/test_oracle_pins.py): closed forms for RMSNorm / rotary / attention / SwiGLU,
torch CPU library ops, Eq. 3 invariants (compressed argmax == full argmax when it lies in
the subset; full subset == uncompressed head), brute-force acceptance on tiny cases,
prefix property of the recursion, speculative == greedy on tiny models, and the parameter
count of the head. The paper prints no worked numeric example, so beyond those pins the
numeric values are "parity unpinned".
"""
from __future__ import annotations

import math

import numpy as np

# --------------------------------------------------------------------------------------
# bf16 storage format
# --------------------------------------------------------------------------------------

def bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns."""
    b = np.asarray(bits, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def f64_to_bf16(x) -> np.ndarray:
    """Round float64 to bf16 (8 significant bits, nearest even), returned as bit patterns.
    Done directly from float64 so there is a single rounding."""
    x = np.asarray(x, dtype=np.float64)
    m, e = np.frexp(x)                         # x = m * 2^e, 0.5 <= |m| < 1
    e = np.maximum(e, -125)                    # bf16 subnormal range shares one quantum
    quantum = np.ldexp(1.0, e - 8)
    r = np.rint(x / quantum) * quantum         # rint rounds halves to even
    r32 = r.astype(np.float32)                 # exact: r has <= 8 significant bits
    return (r32.view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def round_bf16(x) -> np.ndarray:
    """Value of x after storage as bf16."""
    return bf16_to_f64(f64_to_bf16(x))


class _Widened:
    """Memo of bf16 -> float64 conversions of weight matrices (a speed aid: the converted
    values are identical with or without it; arrays must not be modified in place after
    first use). Bounded so a 28-layer target does not exhaust host memory."""

    def __init__(self, limit_bytes: int = 12 << 30):
        self.limit = limit_bytes
        self.used = 0
        self.memo = {}

    def get(self, bits: np.ndarray) -> np.ndarray:
        hit = self.memo.get(id(bits))
        if hit is not None and hit[0] is bits:
            return hit[1]
        w = bf16_to_f64(bits)
        if self.used + w.nbytes <= self.limit:
            self.memo[id(bits)] = (bits, w)      # keeps `bits` alive, so its id stays unique
            self.used += w.nbytes
        return w


_W = _Widened()


def clear_weight_memo():
    _W.memo.clear()
    _W.used = 0


# --------------------------------------------------------------------------------------
# Building blocks of the MTP module / decoder layer (Sec. 2.1, "Architecture Design")
# --------------------------------------------------------------------------------------

def rmsnorm(x: np.ndarray, gain_bits: np.ndarray, eps: float) -> np.ndarray:
    """x / sqrt(mean(x^2) + eps) * g over the last axis."""
    g = bf16_to_f64(gain_bits)
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * g


def rope(x: np.ndarray, pos: int, theta: float) -> np.ndarray:
    """Rotary embedding of x[..., dh] at position pos; element i pairs with i + dh/2 and the
    pair rotates by angle pos * theta^(-2i/dh)."""
    dh = x.shape[-1]
    half = dh // 2
    i = np.arange(half, dtype=np.float64)
    ang = float(pos) * theta ** (-2.0 * i / dh)
    c, s = np.cos(ang), np.sin(ang)
    a, b = x[..., :half], x[..., half:]
    return np.concatenate([a * c - b * s, b * c + a * s], axis=-1)


def silu(z: np.ndarray) -> np.ndarray:
    return z / (1.0 + np.exp(-z))


def _kv_slot(kv: dict, b: int, pos: int, page_size: int):
    page = int(kv["block_table"][b, pos // page_size])
    return page, pos % page_size


def kv_write(kv: dict, b: int, pos: int, k: np.ndarray, v: np.ndarray, page_size: int):
    """Store k, v ([Hkv, dh]) for sequence b at logical position pos, rounded to bf16."""
    page, off = _kv_slot(kv, b, pos, page_size)
    kv["k_pages"][page, :, off, :] = f64_to_bf16(k)
    kv["v_pages"][page, :, off, :] = f64_to_bf16(v)


def kv_read(kv: dict, b: int, n: int, page_size: int):
    """K, V of positions 0..n-1 of sequence b as float64 [n, Hkv, dh]."""
    Hkv, dh = kv["k_pages"].shape[1], kv["k_pages"].shape[3]
    K = np.empty((n, Hkv, dh))
    V = np.empty((n, Hkv, dh))
    for p0 in range(0, n, page_size):
        page = int(kv["block_table"][b, p0 // page_size])
        m = min(page_size, n - p0)
        K[p0:p0 + m] = bf16_to_f64(kv["k_pages"][page, :, :m, :]).transpose(1, 0, 2)
        V[p0:p0 + m] = bf16_to_f64(kv["v_pages"][page, :, :m, :]).transpose(1, 0, 2)
    return K, V


def gqa_attention(q: np.ndarray, K: np.ndarray, V: np.ndarray) -> np.ndarray:
    """softmax(q K^T / sqrt(dh)) V per query head; q [Hq, dh], K/V [n, Hkv, dh]; query head
    j reads KV head floor(j / (Hq/Hkv))."""
    Hq, dh = q.shape
    Hkv = K.shape[1]
    group = Hq // Hkv
    out = np.empty((Hq, dh))
    for j in range(Hq):
        kh = j // group
        s = K[:, kh, :] @ q[j] / math.sqrt(dh)
        s = s - np.max(s)
        p = np.exp(s)
        p = p / np.sum(p)
        out[j] = p @ V[:, kh, :]
    return out


def decoder_layer(x: np.ndarray, pos: int, lw: dict, kv: dict, b: int, shp) -> np.ndarray:
    """One pre-norm decoder layer on one row x[d] at position pos of sequence b; appends this
    position's K/V to the cache and attends over positions 0..pos (self included)."""
    Hq, Hkv, dh = shp.n_q_heads, shp.n_kv_heads, shp.head_dim
    n = rmsnorm(x, lw["g_in"], shp.rms_eps)
    q = (_W.get(lw["wq"]) @ n).reshape(Hq, dh)
    k = (_W.get(lw["wk"]) @ n).reshape(Hkv, dh)
    v = (_W.get(lw["wv"]) @ n).reshape(Hkv, dh)
    q = rope(q, pos, shp.rope_theta)
    k = rope(k, pos, shp.rope_theta)
    kv_write(kv, b, pos, k, v, shp.page_size)
    K, V = kv_read(kv, b, pos + 1, shp.page_size)
    o = gqa_attention(q, K, V).reshape(Hq * dh)
    x = x + _W.get(lw["wo"]) @ o
    n = rmsnorm(x, lw["g_post"], shp.rms_eps)
    act = silu(_W.get(lw["w_gate"]) @ n) * (_W.get(lw["w_up"]) @ n)
    x = x + _W.get(lw["w_down"]) @ act
    return x


# --------------------------------------------------------------------------------------
# Output heads and the argmax rule (Sec. 2.2, Eq. 3)
# --------------------------------------------------------------------------------------

def head_logits(h: np.ndarray, lm_head_bits: np.ndarray, ids=None, rows_per_block: int = 4096) -> np.ndarray:
    """Logits of the sub-matrix W~[i,:] = W[ids[i],:] (Eq. 3); ids=None is the full head.
    Each logit is the plain sum over the row, l_i = sum_c W[ids[i], c] * h[c], evaluated row by
    row so that a row's value does not depend on which other rows are in the subset (rows are
    only visited in blocks to bound memory)."""
    sel = np.arange(lm_head_bits.shape[0]) if ids is None else np.asarray(ids, dtype=np.int64)
    out = np.empty(sel.shape[0])
    for lo in range(0, sel.shape[0], rows_per_block):
        rows = bf16_to_f64(lm_head_bits[sel[lo:lo + rows_per_block]])
        out[lo:lo + rows_per_block] = np.sum(rows * h, axis=-1)
    return out


def argmax_token(logits: np.ndarray, ids=None):
    """Greedy choice among logits rounded to float32: highest value, ties to the lowest
    token id, NaN never wins (an all-NaN row gives the lowest id). Returns (token, gap)
    where gap is the float64 distance between the two highest distinct candidates' values
    (inf for a single candidate) -- used by parity tests to exempt near ties."""
    l32 = np.asarray(logits, dtype=np.float64).astype(np.float32)
    n = l32.shape[0]
    tok = np.arange(n, dtype=np.int64) if ids is None else np.asarray(ids, dtype=np.int64)
    valid = ~np.isnan(l32)
    if not valid.any():
        return int(tok.min()), 0.0
    best = l32[valid].max()
    winners = tok[valid & (l32 == best)]
    t = int(winners.min())
    lv = np.asarray(logits, dtype=np.float64)[valid]
    if lv.shape[0] < 2:
        return t, math.inf
    top2 = np.partition(lv, lv.shape[0] - 2)[-2:]
    return t, float(top2[1] - top2[0])


# --------------------------------------------------------------------------------------
# MTP step and the recursive draft (Sec. 2.1 step k=1 / k>1; Sec. 2.3 "Drafting phase")
# --------------------------------------------------------------------------------------

def mtp_forward(h_prev: np.ndarray, tok: int, pos: int, W: dict, kv: dict, b: int, shp) -> np.ndarray:
    """One pass of the MTP module on the pair (h_prev, Emb(tok)) at cache position pos:
    normalise both inputs, project their concatenation 2d -> d, run the decoder layer, apply
    the final norm. The result feeds the output head and is the h_prev of the next step."""
    e = bf16_to_f64(W["embed"][tok])
    u = np.concatenate([rmsnorm(h_prev, W["g_hnorm"], shp.rms_eps),
                        rmsnorm(e, W["g_enorm"], shp.rms_eps)])
    x = _W.get(W["w_proj"]) @ u
    x = decoder_layer(x, pos, W["layer"], kv, b, shp)
    return rmsnorm(x, W["g_final"], shp.rms_eps)


def draft(shp, W: dict, h_last_bits: np.ndarray, tok_last: np.ndarray, kv: dict, K: int,
          ids=None, forced=None):
    """K recursive draft steps for every sequence of the batch.

    h_last_bits [B, n_ext, d] (bf16 bits) and tok_last [B, n_ext] are pairs (h_j, t_{j+1})
    for the n_ext newest committed positions j = L .. L+n_ext-1 (L = kv['seq_lens'][b]); they
    extend the MTP cache and the last of them is draft step 1. Step k >= 2 feeds the head's
    own output hidden state and the previous draft at the next cache position. ``kv`` is
    written in place; ``seq_lens`` is not changed. ``forced[b, k]`` >= 0 overrides the token
    recursed after step k (teacher forcing for parity tests).

    Returns dict: drafts [B,K] int32, h_out [B,K,d] float64, gap [B,K] (top-2 logit gap).
    """
    h_last_bits = np.asarray(h_last_bits)
    if h_last_bits.ndim == 2:
        h_last_bits = h_last_bits[:, None, :]
        tok_last = np.asarray(tok_last).reshape(-1, 1)
    B, n_ext, d = h_last_bits.shape
    drafts = np.zeros((B, K), dtype=np.int32)
    h_out = np.zeros((B, K, d))
    gap = np.zeros((B, K))
    for b in range(B):
        L = int(kv["seq_lens"][b])
        h = None
        for m in range(n_ext):
            h = mtp_forward(bf16_to_f64(h_last_bits[b, m]), int(tok_last[b, m]), L + m, W, kv, b, shp)
        pos = L + n_ext - 1
        for k in range(K):
            if k > 0:
                pos += 1
                h = mtp_forward(h, tok, pos, W, kv, b, shp)
            t, g = argmax_token(head_logits(h, W["lm_head"], ids), ids)
            drafts[b, k], gap[b, k], h_out[b, k] = t, g, h
            tok = t if forced is None or forced[b, k] < 0 else int(forced[b, k])
    return {"drafts": drafts, "h_out": h_out, "gap": gap}


# --------------------------------------------------------------------------------------
# Verification (Sec. 2.3 "Verification phase")
# --------------------------------------------------------------------------------------

def verify_accept(logits_bits: np.ndarray, drafts: np.ndarray):
    """Greedy verification: g[b,j] = full-vocabulary argmax of target logits row j; drafts
    are accepted in order until the first one that differs from g; the token emitted after
    the accepted prefix ("bonus") is g at the first unaccepted row. Emitted tokens per round
    = accept_len + 1 (the paper's acceptance length tau averages this)."""
    logits_bits = np.asarray(logits_bits)
    B, M, V = logits_bits.shape
    K = M - 1
    g = np.zeros((B, M), dtype=np.int32)
    for b in range(B):
        for j in range(M):
            g[b, j], _ = argmax_token(bf16_to_f64(logits_bits[b, j]))
    accept = np.zeros(B, dtype=np.int32)
    bonus = np.zeros(B, dtype=np.int32)
    for b in range(B):
        a = 0
        while a < K and int(drafts[b, a]) == int(g[b, a]):
            a += 1
        accept[b] = a
        bonus[b] = g[b, a]
    return accept, bonus, g


# --------------------------------------------------------------------------------------
# Target decoder (Sec. 2.1: embedding + transformer layers F + output head W)
# --------------------------------------------------------------------------------------

def target_forward(shp, W: dict, tokens: np.ndarray, kvs: list, want_logits: bool = True):
    """Run M new tokens per sequence through the target stack, causal among themselves, at
    cache positions L_b .. L_b+M-1 (L_b = kvs[l]['seq_lens'][b]); caches are written in place,
    seq_lens unchanged. Returns h [B,M,d] (post final norm, float64) and full-vocabulary
    logits [B,M,V] (float64) or None."""
    tokens = np.asarray(tokens)
    B, M = tokens.shape
    h = np.zeros((B, M, shp.d))
    logits = np.zeros((B, M, shp.vocab)) if want_logits else None
    for b in range(B):
        L = int(kvs[0]["seq_lens"][b])
        for m in range(M):
            x = bf16_to_f64(W["embed"][int(tokens[b, m])])
            for l, lw in enumerate(W["layers"]):
                x = decoder_layer(x, L + m, lw, kvs[l], b, shp)
            h[b, m] = rmsnorm(x, W["g_final"], shp.rms_eps)
            if want_logits:
                logits[b, m] = head_logits(h[b, m], W["lm_head"])
    return h, logits


def target_forward_block(shp, W: dict, tokens, kvs: list, logit_rows=()):
    """target_forward for ONE sequence (batch index 0) with the work grouped by layer instead of by row.

    Same definition, same order of operations per row: the M new tokens sit at cache positions
    L .. L+M-1, each layer normalises, projects (q, k, v), rotates, appends K/V (rounded to bf16)
    and attends causally, adds the output projection, then the SwiGLU MLP. The only difference is
    that a layer's projections are evaluated for all M rows at once -- one matrix product (a
    library matmul) per weight matrix -- so that a layer's weights are widened once per call and
    not once per row; a long prompt through a deep target is otherwise out of reach. Attention,
    rotary embedding and cache writes run row by row exactly as in decoder_layer. Pinned against
    target_forward on the small shape.

    Returns h [M, d] (post final norm, float64) and {row: full-vocabulary logits} for logit_rows."""
    tokens = [int(t) for t in np.asarray(tokens).ravel()]
    M = len(tokens)
    Hq, Hkv, dh = shp.n_q_heads, shp.n_kv_heads, shp.head_dim
    L = int(kvs[0]["seq_lens"][0])
    x = bf16_to_f64(W["embed"][tokens])                                   # [M, d]
    for l, lw in enumerate(W["layers"]):
        n = rmsnorm(x, lw["g_in"], shp.rms_eps)
        q = (n @ bf16_to_f64(lw["wq"]).T).reshape(M, Hq, dh)
        k = (n @ bf16_to_f64(lw["wk"]).T).reshape(M, Hkv, dh)
        v = (n @ bf16_to_f64(lw["wv"]).T).reshape(M, Hkv, dh)
        o = np.empty((M, Hq * dh))
        for m in range(M):
            pos = L + m
            qm = rope(q[m], pos, shp.rope_theta)
            km = rope(k[m], pos, shp.rope_theta)
            kv_write(kvs[l], 0, pos, km, v[m], shp.page_size)
            Kc, Vc = kv_read(kvs[l], 0, pos + 1, shp.page_size)
            o[m] = gqa_attention(qm, Kc, Vc).reshape(Hq * dh)
        x = x + o @ bf16_to_f64(lw["wo"]).T
        n = rmsnorm(x, lw["g_post"], shp.rms_eps)
        act = silu(n @ bf16_to_f64(lw["w_gate"]).T) * (n @ bf16_to_f64(lw["w_up"]).T)
        x = x + act @ bf16_to_f64(lw["w_down"]).T
    h = rmsnorm(x, W["g_final"], shp.rms_eps)
    logits = {int(r): head_logits(h[int(r)], W["lm_head"]) for r in logit_rows}
    return h, logits


def _boundary_logits(row: np.ndarray) -> np.ndarray:
    """Target logits cross the library boundary as bf16 before any argmax reads them."""
    return bf16_to_f64(f64_to_bf16(row))


def greedy_decode(shp, Wt: dict, prompt: np.ndarray, n_new: int, kvs: list):
    """Vanilla autoregressive greedy decoding of one sequence (batch index 0): the sequence
    speculative decoding must reproduce exactly. kvs must be empty caches (seq_lens == 0)
    with room for len(prompt) + n_new tokens."""
    prompt = [int(t) for t in prompt]
    h, logits = target_forward(shp, Wt, np.array([prompt]), kvs)
    for kv in kvs:
        kv["seq_lens"][0] = len(prompt)
    out = []
    tok, _ = argmax_token(_boundary_logits(logits[0, -1]))
    while True:
        out.append(tok)
        if len(out) >= n_new:
            return out
        h, logits = target_forward(shp, Wt, np.array([[tok]]), kvs)
        for kv in kvs:
            kv["seq_lens"][0] += 1
        tok, _ = argmax_token(_boundary_logits(logits[0, 0]))


def speculative_decode(shp, Wt: dict, Wm: dict, prompt: np.ndarray, n_new: int, K: int, ids,
                       kvs: list, mtp_kv: dict, inject=None):
    """EAGLE-style speculative greedy decoding with the MTP head (Sec. 2.3), batch index 0.

    Round: the target has committed L tokens and produced the next token t_L (the first
    verified token) together with hidden states of its newest positions. The MTP cache is
    extended with the pairs (h_j, t_{j+1}) of the positions committed since the last round
    (the whole shifted prompt on the first round), the last pair being draft step 1; K drafts
    are produced; the target scores [t_L, drafts] in one pass; drafts are accepted up to the
    first mismatch and the target's token at that row is emitted as well.

    ``inject(round_index, K)`` may return a list of K tokens replacing the MTP drafts (tests
    use it to exercise every accepted length). Returns (tokens, stats) with
    stats['accepted'] = accepted length per round.
    """
    prompt = [int(t) for t in prompt]
    P = len(prompt)
    hP, logitsP = target_forward(shp, Wt, np.array([prompt]), kvs)
    for kv in kvs:
        kv["seq_lens"][0] = P
    first, _ = argmax_token(_boundary_logits(logitsP[0, -1]))
    out = [first]
    # pairs not yet in the MTP cache: (h_j, t_{j+1}) for j = 0..P-1, with t_P = first
    pend_h = f64_to_bf16(hP[0])                      # hidden states cross the boundary as bf16
    pend_t = prompt[1:] + [first]
    accepted = []
    rnd = 0
    while len(out) < n_new:
        res = draft(shp, Wm, pend_h[None], np.array([pend_t]), mtp_kv, K, ids)
        mtp_kv["seq_lens"][0] += len(pend_t)
        drafts = [int(t) for t in res["drafts"][0]]
        if inject is not None:
            forced = inject(rnd, K)
            if forced is not None:
                drafts = [int(t) for t in forced]
        row_tokens = [out[-1]] + drafts
        hV, logitsV = target_forward(shp, Wt, np.array([row_tokens]), kvs)
        a, bonus, _ = verify_accept(f64_to_bf16(logitsV), np.array([drafts], dtype=np.int32))
        a, bonus = int(a[0]), int(bonus[0])
        for kv in kvs:
            kv["seq_lens"][0] += a + 1
        new_tokens = drafts[:a] + [bonus]
        out.extend(new_tokens)
        accepted.append(a)
        pend_h = f64_to_bf16(hV[0, :a + 1])
        pend_t = new_tokens
        rnd += 1
    return out[:n_new], {"accepted": accepted}


def mtp_param_count(shp) -> int:
    """Parameters owned by the MTP head (projection, one decoder layer, five norm gains);
    the embedding table and output head are the main model's (Sec. 2.2, Sec. 3.1)."""
    d, F = shp.d, shp.ffn
    qd, kvd = shp.n_q_heads * shp.head_dim, shp.n_kv_heads * shp.head_dim
    return 2 * d * d + d * (qd + 2 * kvd) + qd * d + 3 * d * F + 5 * d
