"""Decoding loops over the C ABI: plain greedy decoding with the target, and the speculative loop of
FastMTP Sec. 2.3 (draft with the MTP head, score [last token, drafts] with the target in one pass,
accept until the first mismatch).

Host orchestration only: every tensor operation is a library call (fastmtp_target_step,
fastmtp_draft, fastmtp_accept_ids); this module moves token ids between the calls and advances
sequence lengths. It serves the end-to-end tests and `bench.py --e2e-loop`; batch 1.
"""
from __future__ import annotations

import numpy as np
import torch

from . import binding as Bd


class Target:
    """Device copies of a target model's weights and per-layer paged caches (dicts of torch tensors as
    produced by binding.to_device), stepped through fastmtp_target_step.

    All layers hold the same sequence lengths, so they share layer 0's seq_lens tensor: advancing the
    sequence is one device-side add, whose amount may itself be a device tensor (no host round trip)."""

    def __init__(self, ctx, shape, dev_weights, dev_kvs):
        self.ctx, self.shape = ctx, shape
        self.dW = dev_weights
        self.w, self._keep = Bd.target_w(dev_weights)
        self.dkvs = dev_kvs
        self.seq_lens = dev_kvs[0]["seq_lens"]
        for k in dev_kvs[1:]:
            k["seq_lens"] = self.seq_lens
        self._kvs = [Bd.kv(k) for k in dev_kvs]          # the structs hold addresses only: built once
        self.status = torch.zeros(1, dtype=torch.int32, device="cuda")
        self.calls = 0

    def step(self, tokens, want_logits=False):
        """tokens: [B, M] ids (host list / array, or an int32 device tensor, which is used as it is).
        Returns (hidden states [B, M, d] bf16, logits [B, M, V] bf16 or None, greedy token per row
        [B, M] int32), all on the device."""
        s = self.shape
        if isinstance(tokens, torch.Tensor) and tokens.is_cuda:
            t = tokens.contiguous()
        else:
            t = torch.as_tensor(np.asarray(tokens, dtype=np.int32)).cuda()
        B, M = t.shape
        out_h = torch.empty((B, M, s.d), dtype=torch.bfloat16, device="cuda")
        out_l = torch.empty((B, M, s.vocab), dtype=torch.bfloat16, device="cuda") if want_logits else None
        out_a = torch.full((B, M), -1, dtype=torch.int32, device="cuda")
        self.ctx.fastmtp_target_step(self.w, t, self._kvs, B, M, out_h, out_l, out_a, self.status)
        self.calls += 1
        return out_h, out_l, out_a

    def advance(self, n):
        """n: a host integer or an int32 device tensor broadcastable to [B]."""
        self.seq_lens += n


def prefill(tgt: Target, prompt, chunk=8):
    """Runs the prompt through the target in row chunks. Returns (hidden states [P, d] bf16 on the
    device, the first generated token)."""
    hs, last = [], None
    for lo in range(0, len(prompt), chunk):
        part = prompt[lo:lo + chunk]
        h, _, a = tgt.step([part])
        tgt.advance(len(part))
        hs.append(h[0])
        last = a
    return torch.cat(hs, dim=0), int(last[0, -1].item())


def greedy_decode(tgt: Target, prompt, n_new, chunk=8):
    """Vanilla autoregressive greedy decoding: the sequence the speculative loop must reproduce. The greedy token
    of a step is fed to the next step on the device; the host reads all of them once at the end."""
    _, first = prefill(tgt, prompt, chunk)
    toks = [torch.tensor([[first]], dtype=torch.int32, device="cuda")]
    while len(toks) < n_new:
        _, _, a = tgt.step(toks[-1])
        tgt.advance(1)
        toks.append(a)
    return [int(t) for t in torch.cat(toks, dim=1)[0].tolist()]


def speculative_decode(tgt: Target, mtp_w, mtp_kv, subset, prompt, n_new, K, inject=None, chunk=8, ext_chunk=64,
                       max_ext=None):
    """Speculative greedy decoding of one sequence.

    Round: the MTP cache is extended with the pairs (target hidden state, next token) of the positions
    committed since the last round -- all of them in one fastmtp_draft call, which also produces the K
    drafts (a long prompt goes in first, in calls of ext_chunk pairs with K = 1 whose draft is dropped);
    the target scores [last token, drafts] in one fastmtp_target_step that returns only its greedy
    token per row; fastmtp_accept_ids turns those into the accepted length and the bonus token.

    mtp_w: binding.fmtp_mtp_w; mtp_kv: dict of device tensors (its seq_lens is advanced here);
    subset: device int32 tensor or None; inject(round, K, emitted) may return K tokens that replace the
    MTP drafts of that round (tests use it to reach every accepted length with random weights).
    max_ext: rows per sequence of the per-round draft call (default K + 1).
    Returns (tokens, stats) with stats['accepted'] (per round), stats['tau'], stats['target_calls'].
    """
    ctx, s = tgt.ctx, tgt.shape
    max_ext = max_ext or (K + 1)
    pend_h, first = prefill(tgt, prompt, chunk)
    pend_t = list(prompt[1:]) + [first]
    out = [first]
    drafts_d = torch.zeros((1, K), dtype=torch.int32, device="cuda")
    scratch_d = torch.zeros((1, 1), dtype=torch.int32, device="cuda")
    last_d = torch.zeros((1, 1), dtype=torch.int32, device="cuda")
    acc = torch.zeros(1, dtype=torch.int32, device="cuda")
    bon = torch.zeros(1, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    accepted, rnd = [], 0
    calls0 = tgt.calls
    mkv_c = Bd.kv(mtp_kv)                                  # addresses only; seq_lens is advanced in place
    while len(out) < n_new:
        n, pos = len(pend_t), 0
        tok_all = torch.tensor(pend_t, dtype=torch.int32, device="cuda")
        while n - pos > max_ext:                           # a backlog (the prompt): whole chunks first, their draft dropped
            m = min(ext_chunk, n - pos - 1)
            ctx.fastmtp_draft(mtp_w, pend_h[pos:pos + m].contiguous(), tok_all[pos:pos + m].contiguous(), mkv_c, 1, 1,
                              subset, scratch_d, None, None, status, max_ext=m)
            mtp_kv["seq_lens"] += m
            pos += m
        m = n - pos
        ctx.fastmtp_draft(mtp_w, pend_h[pos:].contiguous(), tok_all[pos:].contiguous(), mkv_c, 1, K, subset, drafts_d,
                          None, None, status, max_ext=m)
        mtp_kv["seq_lens"] += m
        if inject is not None:
            forced = inject(rnd, K, len(out))
            if forced is not None:
                drafts_d.copy_(torch.tensor([[int(t) for t in forced]], dtype=torch.int32), non_blocking=True)
        # the target scores [last token, drafts]; both stay on the device, and the round's one read-back brings the
        # drafts, the accepted length and the bonus token together
        last_d[0, 0] = out[-1]
        h, _, a = tgt.step(torch.cat([last_d, drafts_d], dim=1))
        ctx.fastmtp_accept_ids(a, drafts_d, 1, K, acc, bon)
        rec = torch.cat([drafts_d[0], acc, bon]).tolist()
        drafts, na, bonus = [int(t) for t in rec[:K]], int(rec[K]), int(rec[K + 1])
        tgt.advance(na + 1)
        new = drafts[:na] + [bonus]
        out.extend(new)
        accepted.append(na)
        pend_h, pend_t = h[0, :na + 1], new
        rnd += 1
    assert int(status.item()) == 0 and int(tgt.status.item()) == 0, "a kernel flagged an out-of-range id, page or position"
    emitted = sum(a + 1 for a in accepted)
    stats = {"accepted": accepted, "tau": emitted / max(1, len(accepted)), "target_calls": tgt.calls - calls0,
             "pending_pairs": len(pend_t),      # committed by the target, not yet in the MTP cache (the next round's extend rows)
             "accept_rate_by_position": [float(np.mean([a > k for a in accepted])) for k in range(K)] if accepted else []}
    return out[:n_new], stats
