"""Seeded synthetic inputs for the FastMTP draft / verify hot path.

This module only *draws numbers*: shapes, weight tensors, KV pages, block tables,
token ids, vocabulary subsets and verification cases. It contains none of the
method's arithmetic (no norms, projections, attention, argmax or acceptance), so
that both the CPU oracle's tests and the CUDA path's tests can feed on the very
same bytes without sharing any computational code.

All floating-point tensors are returned as numpy ``uint16`` arrays holding bf16 bit
patterns (round-to-nearest-even from a float32 draw), because bf16 is the storage
type of weights, KV entries and hidden states at the library boundary. Integer
tensors are ``int32``.

Randomness is counter based: every tensor gets its own Philox stream keyed by
``(seed, tag)``, so a tensor's contents do not depend on which other tensors were
generated before it.
"""
from __future__ import annotations

import zlib
from dataclasses import dataclass, replace

import numpy as np

__all__ = [
    "Shape", "TINY", "QWEN7B", "rng", "f32_to_bf16_bits", "bf16_bits_to_f32",
    "normal_bf16", "mtp_weights", "layer_weights", "target_weights", "target_weights_cuda",
    "subset_uniform", "subset_zipf", "context_lengths", "paged_kv",
    "hidden_bf16", "token_ids", "verify_case", "verify_logits_natural",
]


@dataclass(frozen=True)
class Shape:
    """Model geometry (names follow the usual decoder notation)."""
    d: int            # hidden width
    n_q_heads: int    # Hq
    n_kv_heads: int   # Hkv
    head_dim: int     # dh
    ffn: int          # F, SwiGLU inner width
    vocab: int        # V
    n_layers: int     # target decoder depth (the MTP head always has one layer)
    rms_eps: float = 1e-6
    rope_theta: float = 1e4
    page_size: int = 16

    @property
    def q_dim(self) -> int:
        return self.n_q_heads * self.head_dim

    @property
    def kv_dim(self) -> int:
        return self.n_kv_heads * self.head_dim

    def with_layers(self, n: int) -> "Shape":
        return replace(self, n_layers=n)


# Tiny configuration the CPU oracle finishes in well under a second.
TINY = Shape(d=256, n_q_heads=4, n_kv_heads=2, head_dim=64, ffn=688, vocab=4096,
             n_layers=2, rms_eps=1e-6, rope_theta=1e4, page_size=16)
# 7B-class configuration (the headline workload).
QWEN7B = Shape(d=3584, n_q_heads=28, n_kv_heads=4, head_dim=128, ffn=18944,
               vocab=152064, n_layers=28, rms_eps=1e-6, rope_theta=1e6, page_size=16)


def rng(seed: int, tag: str) -> np.random.Generator:
    """Independent Philox stream for ``(seed, tag)``."""
    key = np.array([np.uint64(seed & 0xFFFFFFFFFFFFFFFF),
                    np.uint64(zlib.crc32(tag.encode()) | (len(tag) << 32))], dtype=np.uint64)
    return np.random.Generator(np.random.Philox(key=key))


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit pattern, round to nearest even (finite inputs)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """bf16 bit pattern -> float32 (exact)."""
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def normal_bf16(seed: int, tag: str, shape, std: float, mean: float = 0.0,
                chunk: int = 1 << 24) -> np.ndarray:
    """bf16 bits of ``mean + std * N(0,1)``; drawn in float32, chunked to bound memory."""
    n = int(np.prod(shape))
    out = np.empty(n, dtype=np.uint16)
    g = rng(seed, tag)
    for lo in range(0, n, chunk):
        hi = min(n, lo + chunk)
        x = g.standard_normal(hi - lo, dtype=np.float32)
        x *= np.float32(std)
        if mean != 0.0:
            x += np.float32(mean)
        out[lo:hi] = f32_to_bf16_bits(x)
    return out.reshape(shape)


def _gain(seed: int, tag: str, d: int) -> np.ndarray:
    # RMSNorm gains are 1 + N(0, 0.02) so the gain multiply is exercised
    # without collapsing the activations.
    return normal_bf16(seed, tag, (d,), 0.02, mean=1.0)


def layer_weights(s: Shape, seed: int, prefix: str) -> dict:
    """One decoder layer: all matrices row-major [out, in], ~N(0, 0.02)."""
    w = {
        "g_in": _gain(seed, prefix + ".g_in", s.d),
        "wq": normal_bf16(seed, prefix + ".wq", (s.q_dim, s.d), 0.02),
        "wk": normal_bf16(seed, prefix + ".wk", (s.kv_dim, s.d), 0.02),
        "wv": normal_bf16(seed, prefix + ".wv", (s.kv_dim, s.d), 0.02),
        "wo": normal_bf16(seed, prefix + ".wo", (s.d, s.q_dim), 0.02),
        "g_post": _gain(seed, prefix + ".g_post", s.d),
        "w_gate": normal_bf16(seed, prefix + ".w_gate", (s.ffn, s.d), 0.02),
        "w_up": normal_bf16(seed, prefix + ".w_up", (s.ffn, s.d), 0.02),
        "w_down": normal_bf16(seed, prefix + ".w_down", (s.d, s.ffn), 0.02),
    }
    return w


def mtp_weights(s: Shape, seed: int, embed=None, lm_head=None) -> dict:
    """The position-shared MTP head: two input norms, the 2d->d projection, one decoder
    layer, the final norm, plus the (shared) embedding table and output head."""
    return {
        "embed": embed if embed is not None else normal_bf16(seed, "embed", (s.vocab, s.d), 0.02),
        "lm_head": lm_head if lm_head is not None else normal_bf16(seed, "lm_head", (s.vocab, s.d), 0.02),
        "g_hnorm": _gain(seed, "mtp.g_hnorm", s.d),
        "g_enorm": _gain(seed, "mtp.g_enorm", s.d),
        "w_proj": normal_bf16(seed, "mtp.w_proj", (s.d, 2 * s.d), 0.02),
        "g_final": _gain(seed, "mtp.g_final", s.d),
        "layer": layer_weights(s, seed, "mtp.layer"),
    }


def target_weights(s: Shape, seed: int, embed=None, lm_head=None) -> dict:
    """Random-init target decoder of ``s.n_layers`` layers."""
    return {
        "embed": embed if embed is not None else normal_bf16(seed, "embed", (s.vocab, s.d), 0.02),
        "lm_head": lm_head if lm_head is not None else normal_bf16(seed, "lm_head", (s.vocab, s.d), 0.02),
        "g_final": _gain(seed, "tgt.g_final", s.d),
        "layers": [layer_weights(s, seed, f"tgt.layer{i}") for i in range(s.n_layers)],
    }


def target_weights_cuda(s: Shape, seed: int, device: str = "cuda"):
    """A random-init target decoder drawn on the GPU, for depths at which the host generators take minutes
    (28 layers of the 7B-class shape are 7.6e9 values): every tensor ~N(0, 0.02) in bf16 (gains 1 + N(0, 0.02)) from
    a torch CUDA generator seeded by (seed, tensor name). Returns (device, host): the same bits as a nested dict of
    torch bf16 tensors on the device and as numpy uint16 bit patterns on the host, laid out like target_weights().
    The values differ from target_weights(s, seed): another generator, the same distribution."""
    import torch

    def draw(tag, shape, std, mean=0.0):
        g = torch.Generator(device=device)
        g.manual_seed((seed * 1000003 + zlib.crc32(tag.encode())) & 0x7FFFFFFFFFFFFFFF)
        t = torch.empty(shape, dtype=torch.float32, device=device).normal_(mean, std, generator=g).to(torch.bfloat16)
        return t

    def layer(prefix):
        return {
            "g_in": draw(prefix + ".g_in", (s.d,), 0.02, 1.0),
            "wq": draw(prefix + ".wq", (s.q_dim, s.d), 0.02),
            "wk": draw(prefix + ".wk", (s.kv_dim, s.d), 0.02),
            "wv": draw(prefix + ".wv", (s.kv_dim, s.d), 0.02),
            "wo": draw(prefix + ".wo", (s.d, s.q_dim), 0.02),
            "g_post": draw(prefix + ".g_post", (s.d,), 0.02, 1.0),
            "w_gate": draw(prefix + ".w_gate", (s.ffn, s.d), 0.02),
            "w_up": draw(prefix + ".w_up", (s.ffn, s.d), 0.02),
            "w_down": draw(prefix + ".w_down", (s.d, s.ffn), 0.02),
        }

    dev = {
        "embed": draw("embed", (s.vocab, s.d), 0.02),
        "lm_head": draw("lm_head", (s.vocab, s.d), 0.02),
        "g_final": draw("tgt.g_final", (s.d,), 0.02, 1.0),
        "layers": [layer(f"tgt.layer{i}") for i in range(s.n_layers)],
    }

    def to_host(t):
        return t.cpu().contiguous().view(torch.int16).numpy().view(np.uint16)

    host = {k: to_host(v) for k, v in dev.items() if k != "layers"}
    host["layers"] = [{k: to_host(v) for k, v in l.items()} for l in dev["layers"]]
    return dev, host


def subset_uniform(vocab: int, n: int, seed: int) -> np.ndarray:
    """``n`` distinct token ids drawn uniformly without replacement (unsorted)."""
    g = rng(seed, f"subset_uniform.{vocab}.{n}")
    return g.permutation(vocab)[:n].astype(np.int32)


def subset_zipf(vocab: int, n: int, seed: int, s: float = 1.1) -> np.ndarray:
    """``n`` distinct ids sampled without replacement with weight (id+1)^-s (token id
    stands for frequency rank), by exponential-key top-n; returned sorted ascending.
    ``n == vocab`` yields the identity."""
    if n >= vocab:
        return np.arange(vocab, dtype=np.int32)
    g = rng(seed, f"subset_zipf.{vocab}.{n}")
    w = (np.arange(vocab, dtype=np.float64) + 1.0) ** (-s)
    keys = g.exponential(size=vocab) / w          # smaller key = earlier arrival
    ids = np.argpartition(keys, n)[:n]
    return np.sort(ids).astype(np.int32)


def context_lengths(batch: int, lo: int, hi: int, seed: int) -> np.ndarray:
    """Per-sequence committed context lengths, uniform integers in [lo, hi] inclusive."""
    g = rng(seed, f"ctx.{batch}.{lo}.{hi}")
    return g.integers(lo, hi + 1, size=batch).astype(np.int32)


def paged_kv(s: Shape, seq_lens, extra_tokens: int, seed: int, tag: str = "kv",
             spare_pages: int = 3) -> dict:
    """A paged bf16 KV cache for one layer.

    Pools are ``[num_pages, Hkv, page_size, dh]`` with every entry ~N(0,1) (so the
    committed ``seq_lens[b]`` tokens of each sequence are random, and so is the not yet
    written remainder). Each sequence owns enough pages for ``seq_lens[b] + extra_tokens``
    tokens; the block table is a seeded permutation of the pool so that logical and
    physical page order differ.
    """
    seq_lens = np.asarray(seq_lens, dtype=np.int32)
    B = len(seq_lens)
    pages_per_seq = [(int(L) + extra_tokens + s.page_size - 1) // s.page_size for L in seq_lens]
    max_pages = max(pages_per_seq)
    num_pages = sum(pages_per_seq) + spare_pages
    g = rng(seed, tag + ".table")
    perm = g.permutation(num_pages).astype(np.int32)
    table = np.full((B, max_pages), -1, dtype=np.int32)
    o = 0
    for b, n in enumerate(pages_per_seq):
        table[b, :n] = perm[o:o + n]
        o += n
    shp = (num_pages, s.n_kv_heads, s.page_size, s.head_dim)
    return {
        "k_pages": normal_bf16(seed, tag + ".k", shp, 1.0),
        "v_pages": normal_bf16(seed, tag + ".v", shp, 1.0),
        "block_table": table,
        "seq_lens": seq_lens.copy(),
        "num_pages": num_pages,
        "max_pages_per_seq": max_pages,
    }


def empty_paged_kv(s: Shape, batch: int, max_tokens: int, seed: int, tag: str = "kv0") -> dict:
    """An all-zero paged cache with a shuffled block table and ``seq_lens == 0``."""
    n = (max_tokens + s.page_size - 1) // s.page_size
    num_pages = batch * n + 1
    g = rng(seed, tag + ".table")
    perm = g.permutation(num_pages).astype(np.int32)
    table = perm[:batch * n].reshape(batch, n).copy()
    shp = (num_pages, s.n_kv_heads, s.page_size, s.head_dim)
    return {
        "k_pages": np.zeros(shp, dtype=np.uint16),
        "v_pages": np.zeros(shp, dtype=np.uint16),
        "block_table": table,
        "seq_lens": np.zeros(batch, dtype=np.int32),
        "num_pages": num_pages,
        "max_pages_per_seq": n,
    }


def hidden_bf16(seed: int, shape, tag: str = "h_last") -> np.ndarray:
    """Hidden states ~N(0,1), bf16 bits."""
    return normal_bf16(seed, tag, shape, 1.0)


def token_ids(seed: int, shape, vocab: int, tag: str = "tok") -> np.ndarray:
    return rng(seed, tag).integers(0, vocab, size=shape).astype(np.int32)


def verify_logits_natural(batch: int, rows: int, vocab: int, seed: int, std: float = 2.0) -> np.ndarray:
    """Target logits ``[batch, rows, vocab]`` ~N(0, std) in bf16 with nothing planted:
    the top of a row frequently holds exact bf16 ties."""
    return normal_bf16(seed, f"vlogits.{batch}.{rows}.{vocab}", (batch, rows, vocab), std)


def verify_case(batch: int, K: int, vocab: int, seed: int, p_stop: float = 0.3,
                std: float = 2.0, peak: float = 24.0) -> dict:
    """Verification inputs with a planted answer.

    Logits ``[batch, K+1, vocab]`` are ~N(0, std) in bf16; in every row one seeded token
    ``winner[b, j]`` is overwritten with ``peak`` (far above any N(0, std) draw), which fixes
    the row's maximum without computing one. Planted accepted-prefix lengths follow
    ``P(len = l) = (1 - p_stop)^l * p_stop`` clipped to K. Drafts equal the winners for
    ``j < len``, differ from the winner at ``j == len`` (when ``len < K``) and are random
    after it. Expected result: ``accept_len == length``, ``bonus == winner[b, length]``.
    """
    logits = normal_bf16(seed, f"vcase.logits.{batch}.{K}.{vocab}", (batch, K + 1, vocab), std)
    g = rng(seed, f"vcase.plan.{batch}.{K}.{vocab}")
    winner = g.integers(0, vocab, size=(batch, K + 1)).astype(np.int32)
    peak_bits = f32_to_bf16_bits(np.array([peak], dtype=np.float32))[0]
    bi, ji = np.meshgrid(np.arange(batch), np.arange(K + 1), indexing="ij")
    logits[bi, ji, winner] = peak_bits
    length = np.minimum(g.geometric(p_stop, size=batch) - 1, K).astype(np.int32)
    drafts = g.integers(0, vocab, size=(batch, K)).astype(np.int32) if K > 0 else np.zeros((batch, 0), np.int32)
    for b in range(batch):
        L = int(length[b])
        drafts[b, :L] = winner[b, :L]
        if L < K:
            off = 1 + int(g.integers(0, vocab - 1))
            drafts[b, L] = (int(winner[b, L]) + off) % vocab
    return {"logits": logits, "drafts": drafts, "winner": winner, "length": length}
