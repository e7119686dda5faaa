"""Parity at the benchmark's full size: the 7B-class MTP head (d=3584, 28/4 heads of 128, ffn 18944,
V=152064, subset 32768, 2048 cached tokens, K=3) in the launch configuration bench.py times, checked
against the oracle on every draft, every hidden state and sampled subset logits."""
import os

import numpy as np
import pytest
import torch

from oracle import fastmtp_oracle as O
from paper_2509_18362_b200 import inputs as I
from tests.gpu_util import GAP_TOL as GAP, close, copy_kv, ids_match

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def seven_b():
    shape = I.QWEN7B
    W = I.mtp_weights(shape, 1234)
    from paper_2509_18362_b200 import binding as Bd
    return shape, W, Bd.to_device(W)


def _subset(shape, N, kind, seed):
    if N is None:
        return None
    return I.subset_uniform(shape.vocab, N, seed) if kind == "uniform" else I.subset_zipf(shape.vocab, N, seed)


@pytest.mark.parametrize("seed,B,ctx_lens,N,subset_kind,K", [
    (1234, 1, [2048], 32768, "uniform", 3),          # the benchmark's configuration
    (1234, 3, [2048, 777, 1], 32768, "zipf", 3),     # three sequences: the batched path at this width
    (1300, 1, [2048], None, "-", 3),                 # full vocabulary: the ungathered 1.09 GB head, 1188 tiles of rows
    (1400, 1, [1500], 8192, "zipf", 3),              # smallest subset of the paper's sweep
    (1500, 1, [2048], 65536, "zipf", 2),             # largest compressed subset of the sweep
    (1600, 1, [3000], 32768, "uniform", 5),          # five draft steps
    (1700, 2, [2048, 8000], 32768, "zipf", 3),       # two activation rows in the persistent kernel, 126 attention chunks
])
def test_7b_draft_matches_oracle(seven_b, seed, B, ctx_lens, N, subset_kind, K):
    from paper_2509_18362_b200 import binding as Bd
    shape, W, dW = seven_b
    kv = I.paged_kv(shape, ctx_lens, K + 1, seed + 1)
    h = I.hidden_bf16(seed + 2, (B, shape.d))
    tok = I.token_ids(seed + 3, (B,), shape.vocab)
    ids = _subset(shape, N, subset_kind, seed + 4)
    n_head = shape.vocab if ids is None else N
    dids = None if ids is None else torch.from_numpy(ids).cuda()
    ctx = Bd.Context(shape, max_rows=8, max_K=8, max_ctx=max(ctx_lens) + K + 1)
    dkv = Bd.to_device(copy_kv(kv))
    out_d = torch.full((B, K), -1, dtype=torch.int32, device="cuda")
    out_h = torch.zeros((B, K, shape.d), dtype=torch.bfloat16, device="cuda")
    out_l = torch.zeros((B, K, n_head), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ctx.fastmtp_draft(Bd.mtp_w(dW), Bd.bf16_tensor(h), torch.from_numpy(tok).cuda(), Bd.kv(dkv), B, K,
                      dids, out_d, out_h, out_l, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    drafts = out_d.cpu().numpy()
    # the production call (no debug logits) gives the same drafts
    out_d2 = torch.full((B, K), -1, dtype=torch.int32, device="cuda")
    dkv2 = Bd.to_device(copy_kv(kv))
    ctx.fastmtp_draft(Bd.mtp_w(dW), Bd.bf16_tensor(h), torch.from_numpy(tok).cuda(), Bd.kv(dkv2), B, K, dids, out_d2)
    torch.cuda.synchronize()
    assert np.array_equal(out_d2.cpu().numpy(), drafts)

    okv = copy_kv(kv)
    ref = O.draft(shape, W, h, tok, okv, K, ids, forced=drafts)
    exempt = ids_match(drafts, ref["drafts"], ref["gap"], "7B drafts")
    close(out_h.float().cpu().numpy(), ref["h_out"], "7B h_out")
    # sampled logits: 512 head rows per (sequence, step), computed one by one by the oracle
    g = I.rng(7, "logit-sample")
    lg = out_l.cpu().numpy()
    for b in range(B):
        for k in range(K):
            rows = g.choice(n_head, size=512, replace=False)
            want = O.head_logits(ref["h_out"][b, k], W["lm_head"], rows if ids is None else ids[rows])
            close(lg[b, k, rows], want, f"7B logits b={b} k={k}")
    # K/V appended for the K new positions of every sequence
    gk, gv = Bd.bf16_bits(dkv["k_pages"]), Bd.bf16_bits(dkv["v_pages"])
    for b in range(B):
        for k in range(K):
            pos = ctx_lens[b] + k
            page = int(kv["block_table"][b, pos // shape.page_size])
            close(O.bf16_to_f64(gk[page, :, pos % shape.page_size]), O.bf16_to_f64(okv["k_pages"][page, :, pos % shape.page_size]), "7B K append")
            close(O.bf16_to_f64(gv[page, :, pos % shape.page_size]), O.bf16_to_f64(okv["v_pages"][page, :, pos % shape.page_size]), "7B V append")
    ctx.close()
    O.clear_weight_memo()
    print(f"7B B={B} N={N} K={K} ctx={ctx_lens}: drafts {drafts.tolist()} near-tie exemptions {exempt} of {B * K}")


@pytest.mark.parametrize("B,lo,hi", [(16, 512, 3000), (64, 512, 8192)])
def test_7b_batched_draft_matches_oracle_on_sampled_sequences(seven_b, B, lo, hi):
    """Ragged batches (contexts uniform in [lo, hi]; 64 sequences in [512, 8192] is the ragged serving configuration)
    through the batched tensor-core path at the 7B shape; three sequences (first, last, the longest context) are
    recomputed by the oracle."""
    from paper_2509_18362_b200 import binding as Bd
    shape, W, dW = seven_b
    K, N, seed = 3, 32768, 77 + B
    ctx_lens = [int(x) for x in I.context_lengths(B, lo, hi, seed)]
    kv = I.paged_kv(shape, ctx_lens, K + 1, seed + 1)
    h = I.hidden_bf16(seed + 2, (B, shape.d))
    tok = I.token_ids(seed + 3, (B,), shape.vocab)
    ids = I.subset_zipf(shape.vocab, N, seed + 4)
    ctx = Bd.Context(shape, max_rows=B, max_K=8, max_ctx=max(ctx_lens) + K + 1)
    dkv = Bd.to_device(copy_kv(kv))
    out_d = torch.full((B, K), -1, dtype=torch.int32, device="cuda")
    out_h = torch.zeros((B, K, shape.d), dtype=torch.bfloat16, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ctx.fastmtp_draft(Bd.mtp_w(dW), Bd.bf16_tensor(h), torch.from_numpy(tok).cuda(), Bd.kv(dkv), B, K,
                      torch.from_numpy(ids).cuda(), out_d, out_h, None, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    drafts, hout = out_d.cpu().numpy(), out_h.float().cpu().numpy()
    gk = Bd.bf16_bits(dkv["k_pages"])
    sel = sorted({0, B - 1, int(np.argmax(ctx_lens))})
    okv = copy_kv(kv)
    okv["block_table"], okv["seq_lens"] = okv["block_table"][sel], okv["seq_lens"][sel]
    ref = O.draft(shape, W, h[sel], tok[sel], okv, K, ids, forced=drafts[sel])
    exempt = ids_match(drafts[sel], ref["drafts"], ref["gap"], "7B batched drafts")
    close(hout[sel], ref["h_out"], "7B batched h_out")
    for i, b in enumerate(sel):
        for k in range(K):
            pos = ctx_lens[b] + k
            page = int(kv["block_table"][b, pos // shape.page_size])
            close(O.bf16_to_f64(gk[page, :, pos % shape.page_size]),
                  O.bf16_to_f64(okv["k_pages"][page, :, pos % shape.page_size]), "7B batched K append")
    ctx.close()
    O.clear_weight_memo()
    print(f"7B batched B={B} ctx in [{min(ctx_lens)}, {max(ctx_lens)}]: near-tie exemptions {exempt} of {len(sel) * K}")


def test_verify_accept_full_size():
    """[64, 4, 152064] bf16 logits with planted prefix lengths: exact recovery, equal to the oracle."""
    from paper_2509_18362_b200 import binding as Bd
    ctx = Bd.Context(I.TINY, max_rows=8, max_K=8, max_ctx=64)
    case = I.verify_case(64, 3, 152064, 4321)
    acc = torch.zeros(64, dtype=torch.int32, device="cuda")
    bon = torch.zeros(64, dtype=torch.int32, device="cuda")
    ctx.fastmtp_verify_accept(Bd.bf16_tensor(case["logits"]), torch.from_numpy(case["drafts"]).cuda(), 64, 3, 152064, acc, bon)
    torch.cuda.synchronize()
    assert np.array_equal(acc.cpu().numpy(), case["length"])
    ra, rb, _ = O.verify_accept(case["logits"][:8], case["drafts"][:8])        # oracle on a sample of the batch
    assert np.array_equal(acc.cpu().numpy()[:8], ra) and np.array_equal(bon.cpu().numpy()[:8], rb)
    ctx.close()


def test_speculative_loop_at_7b_width_is_lossless():
    """The end-to-end greedy speculative loop at the 7B-class width (d=3584, GQA 28/4, ffn 18944,
    V=152064, subset 32768, K=3) with a 2-layer random target and a short prompt: token-identical to plain greedy
    decoding by the same library, first tokens checked against the oracle. (The full depth, prompt and length run
    in test_full_depth_speculative_loop_is_lossless_and_matches_the_oracle.)"""
    from tests.test_gpu_target import speculative_vs_greedy
    K, n_new = 3, 20
    ref, out, accepted = speculative_vs_greedy(I.QWEN7B.with_layers(2), 7001, K, n_new, 24, 32768, 128, 4)
    assert out[:n_new] == ref[:n_new]
    assert max(accepted) >= 2 and min(accepted) == 0


def test_7b_width_batched_target_step_matches_oracle_on_sampled_sequences():
    """8 sequences x 4 rows (verification-shaped, 32 rows) through a 2-layer target at the 7B width on the batched
    path; two of the sequences are recomputed by the oracle: hidden states, sampled logits, argmax."""
    from paper_2509_18362_b200 import binding as Bd
    from tests.test_gpu_target import GpuTarget, _bf16_gap
    shape = I.QWEN7B.with_layers(2)
    Wt = I.target_weights(shape, 9001)
    B, M = 8, 4
    L = [int(x) for x in I.context_lengths(B, 100, 700, 9002)]
    kvs = [I.paged_kv(shape, L, M + 1, 9010 + l, tag="t7b%d" % l) for l in range(2)]
    t = I.token_ids(9020, (B, M), shape.vocab)
    gpu = GpuTarget(shape, Wt, kvs, max(L) + M + 2)
    gpu.ctx.close()
    gpu.ctx = Bd.Context(shape, max_rows=B * M, max_K=8, max_ctx=max(L) + M + 2)
    h, l, a = gpu.step(t)
    assert gpu.ctx.launch_count > 10
    sel = [0, B - 1]
    okvs = [copy_kv(kv) for kv in kvs]
    for kv in okvs:
        kv["block_table"], kv["seq_lens"] = kv["block_table"][sel], kv["seq_lens"][sel]
    rh, rl = O.target_forward(shape, Wt, t[sel], okvs)
    close(h.float().cpu().numpy()[sel], rh, "7B-width batched target h")
    lg = l.float().cpu().numpy()[sel]
    g = I.rng(11, "tlogit-sample")
    cols = g.choice(shape.vocab, size=4096, replace=False)
    close(lg[:, :, cols], rl[:, :, cols], "7B-width batched target logits (sampled columns)")
    for i, b in enumerate(sel):
        for m in range(M):
            tok, _ = O.argmax_token(O.round_bf16(rl[i, m]))
            if a[b, m] != tok:
                assert _bf16_gap(rl[i, m]) < GAP, f"argmax mismatch outside a near tie at b={b} m={m}"
    own = [O.argmax_token(O.bf16_to_f64(row))[0] for row in Bd.bf16_bits(l)[sel].reshape(-1, shape.vocab)]
    assert np.array_equal(a[sel].ravel(), np.array(own))
    gpu.close()
    O.clear_weight_memo()


def test_full_depth_speculative_loop_is_lossless_and_matches_the_oracle():
    """The end-to-end configuration at full depth: a random 28-layer target of the 7B-class shape (d=3584, GQA 28/4,
    ffn 18944, V=152064) plus the position-shared MTP layer (shared embedding and output head, subset 32768), batch 1,
    a 512-token prompt, 256 generated tokens, K=3. The speculative loop (extend rows in one draft call, target argmax
    only, acceptance on ids; every other round drafts that are right for a planted number of positions, since random
    weights accept almost nothing) emits exactly the tokens of plain greedy decoding by the same library; the first
    16 of them and the hidden state of the last prompt position agree with the oracle, which runs prompt + 15 tokens
    teacher-forced in one layer-grouped pass (about two minutes of host time)."""
    import time
    from paper_2509_18362_b200 import binding as Bd, loop
    from tests.test_gpu_target import _bf16_gap
    shape, seed, P, n_new, K, N, n_oracle = I.QWEN7B, 5005, 512, 256, 3, 32768, 16
    max_ctx = P + n_new + K + 3
    t0 = time.time()
    dWt, Wt = I.target_weights_cuda(shape, seed)
    Wm = I.mtp_weights(shape, seed + 1, embed=Wt["embed"], lm_head=Wt["lm_head"])
    prompt = [int(t) for t in I.token_ids(seed + 2, (P,), shape.vocab)]
    ids = I.subset_uniform(shape.vocab, N, seed + 3)
    mk = lambda: [I.empty_paged_kv(shape, 1, max_ctx, seed + 10 + l) for l in range(shape.n_layers)]
    ctx = Bd.Context(shape, max_rows=64, max_K=8, max_ctx=max_ctx)
    t_gen = time.time() - t0

    probe = loop.Target(ctx, shape, dWt, [Bd.to_device(kv) for kv in mk()])
    h_prompt, _ = loop.prefill(probe, prompt)
    torch.cuda.synchronize()
    t0 = time.time()
    ref = loop.greedy_decode(loop.Target(ctx, shape, dWt, [Bd.to_device(kv) for kv in mk()]), prompt, n_new + K + 1)
    torch.cuda.synchronize()
    t_greedy = time.time() - t0

    tgt = loop.Target(ctx, shape, dWt, [Bd.to_device(kv) for kv in mk()])
    dWm = dict(Bd.to_device({k: v for k, v in Wm.items() if k not in ("embed", "lm_head")}),
               embed=dWt["embed"], lm_head=dWt["lm_head"])
    mkv = Bd.to_device(I.empty_paged_kv(shape, 1, max_ctx, seed + 20))

    def inject(rnd, K, emitted):
        if rnd % 2 == 0:
            return None
        n_ok = (rnd // 2) % (K + 1)
        good = ref[emitted:emitted + K]
        return list(good[:n_ok]) + [(t + 1) % shape.vocab for t in good[n_ok:]]

    t0 = time.time()
    out, stats = loop.speculative_decode(tgt, Bd.mtp_w(dWm), mkv, torch.from_numpy(ids).cuda(), prompt, n_new, K, inject)
    torch.cuda.synchronize()
    t_spec = time.time() - t0
    assert out == ref[:n_new]                                          # all 256 tokens
    assert {0, 1, 2, 3} <= set(stats["accepted"])
    assert int(mkv["seq_lens"].item()) + stats["pending_pairs"] == int(tgt.dkvs[0]["seq_lens"].item())
    ctx.close()

    t0 = time.time()
    seq = prompt + [int(t) for t in ref[:n_oracle - 1]]
    rows = list(range(P - 1, P - 1 + n_oracle))
    hh, logits = O.target_forward_block(shape, Wt, seq, mk(), logit_rows=rows)
    t_oracle = time.time() - t0
    exempt = 0
    for i, r in enumerate(rows):
        t, _ = O.argmax_token(O.round_bf16(logits[r]))
        if t != ref[i]:
            assert _bf16_gap(logits[r]) < GAP, f"token {i}: oracle {t}, gpu {ref[i]}"
            exempt += 1
    close(h_prompt[P - 1].float().cpu().numpy(), hh[P - 1], "hidden state of the last prompt position, 28 layers deep")
    close(h_prompt[::37].float().cpu().numpy(), hh[:P:37], "sampled prompt hidden states, 28 layers deep")
    print(f"full depth: weights {t_gen:.0f} s, greedy {n_new + K + 1} tokens {t_greedy:.2f} s "
          f"({(n_new + K + 1) / t_greedy:.0f} tok/s incl. 512-token prefill), speculative {n_new} tokens {t_spec:.2f} s, "
          f"tau {stats['tau']:.2f} (half the rounds injected), acceptance by position {stats['accept_rate_by_position']}, "
          f"oracle {t_oracle:.0f} s on {os.cpu_count()} host cores, near-tie exemptions {exempt} of {n_oracle}")
