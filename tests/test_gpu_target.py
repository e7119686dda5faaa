"""GPU parity of fastmtp_target_step and of the speculative loop built from the three calls."""
import numpy as np
import pytest
import torch

from oracle import fastmtp_oracle as O
from paper_2509_18362_b200 import inputs as I
from tests.gpu_util import GAP_TOL, close, copy_kv, ids_match

pytestmark = pytest.mark.gpu


def _binding():
    from paper_2509_18362_b200 import binding
    return binding


class GpuTarget:
    """Device copies of a target model and its per-layer caches, stepped through the C ABI."""

    def __init__(self, shape, Wt, kvs, max_ctx):
        Bd = _binding()
        self.Bd, self.shape = Bd, shape
        self.ctx = Bd.Context(shape, max_rows=8, max_K=8, max_ctx=max_ctx)
        self.dW = Bd.to_device(Wt)
        self.w, self._keep = Bd.target_w(self.dW)
        self.dkvs = [Bd.to_device(copy_kv(kv)) for kv in kvs]

    def step(self, tokens, want_logits=True):
        Bd, s = self.Bd, self.shape
        tokens = np.asarray(tokens, dtype=np.int32)
        B, M = tokens.shape
        out_h = torch.zeros((B, M, s.d), dtype=torch.bfloat16, device="cuda")
        out_l = torch.zeros((B, M, s.vocab), dtype=torch.bfloat16, device="cuda") if want_logits else None
        out_a = torch.full((B, M), -1, dtype=torch.int32, device="cuda")
        st = torch.zeros(1, dtype=torch.int32, device="cuda")
        self.ctx.fastmtp_target_step(self.w, torch.from_numpy(tokens).cuda(), [Bd.kv(k) for k in self.dkvs], B, M,
                                     out_h, out_l, out_a, st)
        torch.cuda.synchronize()
        assert int(st.item()) == 0
        return out_h, out_l, out_a.cpu().numpy()

    def advance(self, n):
        for k in self.dkvs:
            k["seq_lens"] += torch.as_tensor(n, dtype=torch.int32, device="cuda")

    def close(self):
        self.ctx.close()


def _bf16_gap(row):
    """Top-2 gap of an oracle logit row, less one bf16 spacing at the winner's magnitude: the
    greedy choice is made on bf16-rounded logits, so two candidates closer than the tolerance
    plus one spacing can legitimately round to a tie (lowest id) on one side only."""
    top2 = np.partition(row, row.shape[0] - 2)[-2:]
    ulp = 2.0 ** (np.floor(np.log2(max(abs(top2[1]), 1e-30))) - 7)
    return float(top2[1] - top2[0] - ulp)


def _gaps(logits64):
    """Top-2 gap of every row of oracle logits after bf16 rounding (the precision the greedy
    choice is made in at the boundary)."""
    flat = logits64.reshape(-1, logits64.shape[-1])
    toks, gaps = [], []
    for row in flat:
        t, _ = O.argmax_token(O.round_bf16(row))
        toks.append(t)
        gaps.append(_bf16_gap(row))
    return np.array(toks), np.array(gaps)


@pytest.mark.parametrize("n_layers", [1, 3])
def test_target_step_prefill_decode_verify(n_layers):
    shape = I.TINY.with_layers(n_layers)
    Wt = I.target_weights(shape, 300 + n_layers)
    B = 2
    kvs = [I.empty_paged_kv(shape, B, 48, 310 + l) for l in range(n_layers)]
    okvs = [copy_kv(kv) for kv in kvs]
    gpu = GpuTarget(shape, Wt, kvs, 64)
    toks = I.token_ids(320, (B, 11), shape.vocab)
    # rows per call: 4 + 4 + 3 (prefill chunks), then 1 (decode), then 4 (verify-shaped)
    for lo, hi in [(0, 4), (4, 8), (8, 11)]:
        h, l, a = gpu.step(toks[:, lo:hi])
        rh, rl = O.target_forward(shape, Wt, toks[:, lo:hi], okvs)
        close(h.float().cpu().numpy(), rh, f"target h rows {lo}:{hi}")
        close(l.float().cpu().numpy(), rl, f"target logits rows {lo}:{hi}")
        rt, gap = _gaps(rl)
        ids_match(a, rt, gap, "target argmax")
        gpu.advance(hi - lo)
        for kv in okvs:
            kv["seq_lens"] += hi - lo
    for M in (1, 4):
        t = I.token_ids(330 + M, (B, M), shape.vocab)
        h, l, a = gpu.step(t)
        rh, rl = O.target_forward(shape, Wt, t, okvs)
        close(h.float().cpu().numpy(), rh, f"target h M={M}")
        close(l.float().cpu().numpy(), rl, f"target logits M={M}")
        # the kernel's own argmax equals the argmax of the logits it wrote (decided on bf16 values)
        own = [O.argmax_token(O.bf16_to_f64(row))[0] for row in
               _binding().bf16_bits(l).reshape(-1, shape.vocab)]
        assert np.array_equal(a.ravel(), np.array(own))
        gpu.advance(M)
        for kv in okvs:
            kv["seq_lens"] += M
    for l in range(n_layers):
        close(O.bf16_to_f64(_binding().bf16_bits(gpu.dkvs[l]["k_pages"])), O.bf16_to_f64(okvs[l]["k_pages"]),
              f"layer {l} K cache")
    gpu.close()


def test_target_step_more_rows_than_one_launch():
    """10 sequences x 3 rows = 30 rows, more sequences than one persistent launch takes: the batched tensor-core path (every
    layer's weights streamed once for all rows). Hidden states, logits, the kernel's own argmax and the K/V appended
    by both layers against the oracle, over two consecutive calls."""
    shape = I.TINY.with_layers(2)
    Wt = I.target_weights(shape, 611)
    B, M = 10, 3
    kvs = [I.empty_paged_kv(shape, B, 32, 620 + l) for l in range(2)]
    okvs = [copy_kv(kv) for kv in kvs]
    Bd = _binding()
    gpu = GpuTarget(shape, Wt, kvs, 64)
    gpu.ctx.close()
    gpu.ctx = Bd.Context(shape, max_rows=32, max_K=8, max_ctx=64)
    for it in range(2):
        t = I.token_ids(630 + it, (B, M), shape.vocab)
        h, l, a = gpu.step(t)
        rh, rl = O.target_forward(shape, Wt, t, okvs)
        close(h.float().cpu().numpy(), rh, "target h 30 rows")
        close(l.float().cpu().numpy(), rl, "target logits 30 rows")
        rt, gap = _gaps(rl)
        ids_match(a, rt, gap, "target argmax 30 rows")
        own = [O.argmax_token(O.bf16_to_f64(row))[0] for row in Bd.bf16_bits(l).reshape(-1, shape.vocab)]
        assert np.array_equal(a.ravel(), np.array(own))      # decided on the bf16 logits it wrote
        gpu.advance(M)
        for kv in okvs:
            kv["seq_lens"] += M
    assert gpu.ctx.launch_count > 6                            # a sequence of kernels per layer, not grouped launches
    for l in range(2):
        close(O.bf16_to_f64(Bd.bf16_bits(gpu.dkvs[l]["k_pages"])), O.bf16_to_f64(okvs[l]["k_pages"]), f"layer {l} K cache")
        close(O.bf16_to_f64(Bd.bf16_bits(gpu.dkvs[l]["v_pages"])), O.bf16_to_f64(okvs[l]["v_pages"]), f"layer {l} V cache")
    gpu.close()


def test_batched_target_rows_do_not_depend_on_the_batch():
    """On the batched path too, a row's hidden state and logits are the same bits whether its sequence is scored
    with 8 or with 11 other sequences, and with or without the logits being written."""
    shape = I.TINY.with_layers(2)
    Wt = I.target_weights(shape, 711)
    B, M = 12, 3
    Bd = _binding()
    L = [int(x) for x in I.context_lengths(B, 0, 300, 712)]
    kvs = [I.paged_kv(shape, L, M + 1, 720 + l, tag="t%d" % l) for l in range(2)]
    t = I.token_ids(730, (B, M), shape.vocab)
    big = GpuTarget(shape, Wt, kvs, max(L) + M + 2)
    big.ctx.close()
    big.ctx = Bd.Context(shape, max_rows=64, max_K=8, max_ctx=max(L) + M + 2)
    h12, l12, a12 = big.step(t)
    big.close()
    sub = [dict(kv) for kv in kvs]
    for kv in sub:
        kv["block_table"] = kv["block_table"][:9].copy()
        kv["seq_lens"] = kv["seq_lens"][:9].copy()
    small = GpuTarget(shape, Wt, sub, max(L) + M + 2)
    small.ctx.close()
    small.ctx = Bd.Context(shape, max_rows=64, max_K=8, max_ctx=max(L) + M + 2)
    h3, l3, a3 = small.step(t[:9])
    h3b, _, a3b = small.step(t[:9], want_logits=False)       # K/V slots are rewritten with the same values
    small.close()
    assert torch.equal(h3, h12[:9]) and torch.equal(l3, l12[:9]) and np.array_equal(a3, a12[:9])
    assert torch.equal(h3b, h3) and np.array_equal(a3b, a3)


def test_rows_do_not_depend_on_rows_per_call():
    """A position's hidden state and logits are bit-identical whether it is scored alone (M=1)
    or as one of several rows (M=4): the property that makes verification lossless."""
    shape = I.TINY.with_layers(2)
    Wt = I.target_weights(shape, 401)
    kvs = [I.empty_paged_kv(shape, 1, 48, 410 + l) for l in range(2)]
    toks = I.token_ids(420, (1, 8), shape.vocab)
    a = GpuTarget(shape, Wt, kvs, 64)
    hs, ls = [], []
    for j in range(8):
        h, l, _ = a.step(toks[:, j:j + 1])
        a.advance(1)
        hs.append(h)
        ls.append(l)
    a.close()
    b = GpuTarget(shape, Wt, kvs, 64)
    h4a, l4a, _ = b.step(toks[:, 0:4])
    b.advance(4)
    h4b, l4b, _ = b.step(toks[:, 4:8])
    b.close()
    one_h = torch.cat(hs, dim=1)
    one_l = torch.cat(ls, dim=1)
    assert torch.equal(one_h, torch.cat([h4a, h4b], dim=1))
    assert torch.equal(one_l, torch.cat([l4a, l4b], dim=1))


def oracle_checks_greedy_tokens(shape, Wt, prompt, tokens, mk_kvs):
    """The oracle's target on [prompt ; tokens[:-1]] in one teacher-forced pass: at every generated position its greedy
    choice (on bf16-rounded logits) equals the library's token, except at near ties. Returns the number of exemptions."""
    n = len(tokens)
    seq = np.array([list(prompt) + [int(t) for t in tokens[:-1]]])
    okvs = mk_kvs()
    hh, _ = O.target_forward(shape, Wt, seq, okvs, want_logits=False)
    exempt = 0
    for i in range(n):
        row = O.head_logits(hh[0, len(prompt) - 1 + i], Wt["lm_head"])
        t, _ = O.argmax_token(O.round_bf16(row))
        if t != int(tokens[i]):
            assert _bf16_gap(row) < GAP_TOL, f"token {i}: oracle {t}, gpu {int(tokens[i])}"
            exempt += 1
    return exempt


def speculative_vs_greedy(shape, seed, K, n_new, prompt_len, N, max_ctx, n_oracle):
    """Greedy decoding and speculative decoding (MTP drafts; every other round drafts that are right for a planted
    number of positions) by the library on the same random model, through the loops of paper_2509_18362_b200.loop
    (extend rows in one draft call, target argmax only, acceptance on token ids). Returns both token lists and the
    accepted lengths, after checking the first n_oracle greedy tokens against the oracle."""
    Bd = _binding()
    from paper_2509_18362_b200 import loop
    L = shape.n_layers
    Wt = I.target_weights(shape, seed)
    Wm = I.mtp_weights(shape, seed + 1, embed=Wt["embed"], lm_head=Wt["lm_head"])
    prompt = [int(t) for t in I.token_ids(seed + 2, (prompt_len,), shape.vocab)]
    ids = I.subset_uniform(shape.vocab, N, seed + 3)
    mk = lambda: [I.empty_paged_kv(shape, 1, max_ctx, seed + 10 + l) for l in range(L)]
    ctx = Bd.Context(shape, max_rows=64, max_K=8, max_ctx=max_ctx)
    dW = Bd.to_device(Wt)

    ref = loop.greedy_decode(loop.Target(ctx, shape, dW, [Bd.to_device(kv) for kv in mk()]), prompt, n_new + K + 1)

    tgt = loop.Target(ctx, shape, dW, [Bd.to_device(kv) for kv in mk()])
    dWm = dict(Bd.to_device({k: v for k, v in Wm.items() if k not in ("embed", "lm_head")}),
               embed=dW["embed"], lm_head=dW["lm_head"])                   # shared with the target, one copy
    mkv = Bd.to_device(I.empty_paged_kv(shape, 1, max_ctx, seed + 20))

    def inject(rnd, K, emitted):
        if rnd % 2 == 0:
            return None
        n_ok = (rnd // 2) % (K + 1)                                          # drafts right for a planted number of positions
        good = ref[emitted:emitted + K]
        return list(good[:n_ok]) + [(t + 1) % shape.vocab for t in good[n_ok:]]

    out, stats = loop.speculative_decode(tgt, Bd.mtp_w(dWm), mkv, torch.from_numpy(ids).cuda(), prompt, n_new, K, inject)
    # the MTP cache trails the target's by exactly the pairs the next round would extend it with
    assert int(mkv["seq_lens"].item()) + stats["pending_pairs"] == int(tgt.dkvs[0]["seq_lens"].item())
    ctx.close()
    exempt = oracle_checks_greedy_tokens(shape, Wt, prompt, ref[:n_oracle], mk)
    O.clear_weight_memo()
    print(f"loop: tau {stats['tau']:.2f}, accepted {stats['accepted']}, oracle exemptions {exempt}/{n_oracle}")
    return ref, out, stats["accepted"]


def test_speculative_loop_is_token_identical_to_greedy_on_gpu():
    """Draft with the MTP head, score [last, drafts] with the target in one call, accept with
    fastmtp_verify_accept: the emitted sequence equals plain greedy decoding by the same
    library; and the first tokens agree with the oracle's greedy run up to near ties."""
    K, n_new = 3, 40
    ref, out, accepted = speculative_vs_greedy(I.TINY.with_layers(2), 501, K, n_new, 19, 1024, 128, 12)
    assert out[:n_new] == ref[:n_new]
    assert {0, 1, 2, 3} <= set(accepted)
