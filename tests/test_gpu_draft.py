"""GPU parity of fastmtp_draft against the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import fastmtp_oracle as O
from paper_2509_18362_b200 import inputs as I
from tests.gpu_util import close, copy_kv, ids_match

pytestmark = pytest.mark.gpu


def _binding():
    from paper_2509_18362_b200 import binding
    return binding


def run_draft_case(shape, seed, B, L, K, N, subset="uniform", want_logits=True, max_ctx=None):
    """Runs the same seeded case through the oracle and the CUDA path; returns both results."""
    Bd = _binding()
    W = I.mtp_weights(shape, seed)
    kv = I.paged_kv(shape, list(L), K + 1, seed + 1)
    h = I.hidden_bf16(seed + 2, (B, shape.d))
    tok = I.token_ids(seed + 3, (B,), shape.vocab)
    if N is None:
        ids = None
    elif subset == "uniform":
        ids = I.subset_uniform(shape.vocab, N, seed + 4)
    else:
        ids = I.subset_zipf(shape.vocab, N, seed + 4)
    n_head = shape.vocab if ids is None else len(ids)

    ctx = Bd.Context(shape, max_rows=max(8, B), max_K=8, max_ctx=max_ctx or (max(L) + K + 1))
    dW = Bd.to_device(W)
    dkv = Bd.to_device(copy_kv(kv))
    dh = Bd.bf16_tensor(h)
    dtok = torch.from_numpy(tok).cuda()
    dids = None if ids is None else torch.from_numpy(ids).cuda()
    out_d = torch.full((B, K), -1, dtype=torch.int32, device="cuda")
    out_h = torch.zeros((B, K, shape.d), dtype=torch.bfloat16, device="cuda")
    out_l = torch.zeros((B, K, n_head), dtype=torch.float32, device="cuda") if want_logits else None
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ctx.fastmtp_draft(Bd.mtp_w(dW), dh, dtok, Bd.kv(dkv), B, K, dids, out_d, out_h, out_l, status)
    torch.cuda.synchronize()
    got = {
        "drafts": out_d.cpu().numpy(),
        "h_out": out_h.float().cpu().numpy(),
        "logits": None if out_l is None else out_l.cpu().numpy(),
        "status": int(status.item()),
        "k_pages": Bd.bf16_bits(dkv["k_pages"]),
        "v_pages": Bd.bf16_bits(dkv["v_pages"]),
        "launches": ctx.launch_count,
        "tmem_launches": ctx.tmem_launch_count,
    }
    ctx.close()

    okv = copy_kv(kv)
    ref = O.draft(shape, W, h, tok, okv, K, ids, forced=got["drafts"])
    ref["kv"] = okv
    ref["ids"] = ids
    ref["W"] = W
    return got, ref


def check_draft(got, ref, what):
    assert got["status"] == 0, f"{what}: device status {got['status']:#x}"
    exempt = ids_match(got["drafts"], ref["drafts"], ref["gap"], what + " drafts")
    close(got["h_out"], ref["h_out"], what + " h_out")
    close(O.bf16_to_f64(got["k_pages"]), O.bf16_to_f64(ref["kv"]["k_pages"]), what + " K cache")
    close(O.bf16_to_f64(got["v_pages"]), O.bf16_to_f64(ref["kv"]["v_pages"]), what + " V cache")
    return exempt


def test_tiny_config_batch1():
    """d=256, 4/2 heads of 64, ffn 688, V=4096, subset 1024, 64 cached tokens, K=3."""
    got, ref = run_draft_case(I.TINY, 1234, 1, [64], 3, 1024)
    check_draft(got, ref, "tiny")
    assert got["launches"] == 1           # all K steps inside one launch
    # debug logits against the oracle's, row by row of the subset
    for k in range(3):
        lg = O.head_logits(ref["h_out"][0, k], ref["W"]["lm_head"], ref["ids"])
        close(got["logits"][0, k], lg, f"tiny logits step {k}")


@pytest.mark.parametrize("B,L,K,N", [
    (1, [70], 3, 1500),           # ragged last head tile
    (2, [5, 130], 2, None),       # full vocabulary, context crossing an attention chunk
    (4, [0, 63, 64, 200], 2, 640),
])
def test_tensor_memory_staging_matches_oracle(B, L, K, N, monkeypatch):
    """The persistent kernel's optional second staging level (FMTP_TMEM=1, read when the context is created): a shape
    whose contraction lengths are all multiples of the 512-wide stage (d=2048, 8/2 heads of 128, ffn 1536), so that
    every phase runs its first eight stages through tensor memory and the rest from the shared-memory stages in the
    slot layout; also against the same call without it."""
    shape = I.Shape(d=2048, n_q_heads=8, n_kv_heads=2, head_dim=128, ffn=1536, vocab=4096, n_layers=1, rms_eps=1e-6,
                    rope_theta=1e4, page_size=16)
    monkeypatch.setenv("FMTP_TMEM", "1")
    got, ref = run_draft_case(shape, 4100 + B, B, L, K, N)
    check_draft(got, ref, f"tmem B={B} K={K} N={N}")
    assert got["launches"] == 1 and got["tmem_launches"] == 1
    monkeypatch.setenv("FMTP_TMEM", "0")
    plain, _ = run_draft_case(shape, 4100 + B, B, L, K, N)
    assert plain["tmem_launches"] == 0
    assert np.array_equal(plain["drafts"], got["drafts"])
    close(plain["logits"], got["logits"], "tmem vs plain logits")


@pytest.mark.parametrize("B,L,K,N", [
    (2, [5, 130], 2, 1000),       # ragged subset size, context crossing an attention chunk
    (3, [1, 15, 16], 4, 37),      # page-boundary contexts, tiny subset
    (8, [0, 3, 17, 31, 64, 127, 128, 200], 1, 4096),   # empty context, full-size subset, 8 rows
    (1, [257], 5, None),          # NULL subset = full vocabulary
])
def test_tiny_shapes_ragged(B, L, K, N):
    got, ref = run_draft_case(I.TINY, 77 + B, B, L, K, N)
    check_draft(got, ref, f"tiny B={B} K={K} N={N}")


@pytest.mark.parametrize("B,lo,hi,K,N,subset", [
    (20, 0, 200, 3, 1024, "zipf"),        # 20 sequences, ragged contexts below one attention chunk
    (64, 0, 700, 2, 1000, "uniform"),     # a full group; contexts up to three 256-token attention chunks; ragged subset
    (9, 250, 260, 4, None, "uniform"),    # contexts crossing the chunk boundary during the K steps; full vocabulary
    (70, 0, 90, 1, 37, "uniform"),        # two groups (64 + 6); fewer head rows than one 128-row tile
])
def test_batched_path_matches_oracle(B, lo, hi, K, N, subset):
    """More sequences than one persistent-kernel launch takes: the tensor-core GEMM path (every weight
    streamed once per step for the whole group)."""
    L = [int(x) for x in I.context_lengths(B, lo, hi, 9 + B)]
    got, ref = run_draft_case(I.TINY, 800 + B, B, L, K, N, subset=subset, max_ctx=hi + K + 2)
    check_draft(got, ref, f"tiny batched B={B}")
    assert got["launches"] > 3            # a sequence of kernels per step, not one persistent launch per group
    for b in (0, B - 1):
        for k in range(K):
            lg = O.head_logits(ref["h_out"][b, k], ref["W"]["lm_head"], ref["ids"])
            close(got["logits"][b, k], lg, f"tiny batched logits b={b} step {k}")
    # the production call (no debug logits) gathers the head rows in ascending id order: same results
    prod, _ = run_draft_case(I.TINY, 800 + B, B, L, K, N, subset=subset, max_ctx=hi + K + 2, want_logits=False)
    assert np.array_equal(prod["drafts"], got["drafts"]) and np.array_equal(prod["h_out"], got["h_out"])


def test_batched_path_subset_with_repeated_ids():
    """A subset array that repeats ids (outside the contract, but harmless): same drafts as the distinct subset."""
    Bd = _binding()
    shape = I.TINY
    W = I.mtp_weights(shape, 31)
    L = [int(x) for x in I.context_lengths(10, 0, 50, 32)]
    kv = I.paged_kv(shape, L, 3, 33)
    h = I.hidden_bf16(34, (10, shape.d))
    tok = I.token_ids(35, (10,), shape.vocab)
    ids = I.subset_uniform(shape.vocab, 300, 36)
    rep = np.concatenate([ids, ids[:77], ids[5:6]]).astype(np.int32)
    dW = Bd.to_device(W)
    outs = []
    for arr in (ids, rep):
        ctx = Bd.Context(shape, max_rows=16, max_K=8, max_ctx=64)
        dkv = Bd.to_device(copy_kv(kv))
        out_d = torch.zeros((10, 2), dtype=torch.int32, device="cuda")
        st = torch.zeros(1, dtype=torch.int32, device="cuda")
        ctx.fastmtp_draft(Bd.mtp_w(dW), Bd.bf16_tensor(h), torch.from_numpy(tok).cuda(), Bd.kv(dkv), 10, 2,
                          torch.from_numpy(arr).cuda(), out_d, None, None, st)
        torch.cuda.synchronize()
        assert int(st.item()) == 0
        outs.append(out_d.cpu().numpy())
        ctx.close()
    assert np.array_equal(outs[0], outs[1])


def test_batched_path_odd_geometry():
    """head_dim 128, 7 query heads per KV head, ffn and d not multiples of the GEMM's 64-wide K block
    or 128-row tile, 12 sequences."""
    shape = I.Shape(d=448, n_q_heads=7, n_kv_heads=1, head_dim=128, ffn=1200, vocab=3001, n_layers=1,
                    rms_eps=1e-6, rope_theta=1e6, page_size=16)
    L = [int(x) for x in I.context_lengths(12, 0, 400, 3)]
    got, ref = run_draft_case(shape, 6, 12, L, 3, 777, subset="zipf")
    check_draft(got, ref, "odd geometry batched")


@pytest.mark.parametrize("B,L,K", [
    (1, [191], 3),                # last chunk one token short of full: the rows written in this call cross into a new chunk
    (3, [0, 64, 130], 2),         # empty context, chunk-aligned context
    (12, [0, 5, 63, 64, 65, 127, 128, 129, 200, 255, 256, 300], 2),   # the batched path's attention at the same geometry
])
def test_eight_query_heads_per_kv_head(B, L, K):
    """The widest group the library takes (8 query heads on one KV head, head_dim 64): every row of the attention
    operand carries a head, in the persistent kernel (1 and 3 sequences) and on the batched path (12)."""
    shape = I.Shape(d=512, n_q_heads=8, n_kv_heads=1, head_dim=64, ffn=1024, vocab=2048, n_layers=1,
                    rms_eps=1e-6, rope_theta=1e4, page_size=16)
    got, ref = run_draft_case(shape, 8800 + B, B, L, K, 500)
    check_draft(got, ref, f"8 heads per KV head B={B}")


def test_batched_path_bit_reproducible_and_batch_invariant():
    """Two runs agree bit for bit, and a sequence's result is the same in a group of 12 and of 40."""
    L = [int(x) for x in I.context_lengths(40, 0, 300, 5)]
    a, _ = run_draft_case(I.TINY, 4711, 40, L, 3, 1024)
    b, _ = run_draft_case(I.TINY, 4711, 40, L, 3, 1024)
    assert np.array_equal(a["drafts"], b["drafts"]) and np.array_equal(a["h_out"], b["h_out"])
    assert np.array_equal(a["logits"], b["logits"]) and np.array_equal(a["k_pages"], b["k_pages"])
    # the first 12 sequences alone (same seeds => same weights and inputs for those rows)
    Bd = _binding()
    shape = I.TINY
    W = I.mtp_weights(shape, 4711)
    kv = I.paged_kv(shape, L, 4, 4712)
    h = I.hidden_bf16(4713, (40, shape.d))
    tok = I.token_ids(4714, (40,), shape.vocab)
    ids = I.subset_uniform(shape.vocab, 1024, 4715)
    ctx = Bd.Context(shape, max_rows=64, max_K=8, max_ctx=max(L) + 4)
    dW, dkv = Bd.to_device(W), Bd.to_device(copy_kv(kv))
    sub = dict(dkv)
    sub["block_table"] = dkv["block_table"][:12].contiguous()
    sub["seq_lens"] = dkv["seq_lens"][:12].contiguous()
    out_d = torch.zeros((12, 3), dtype=torch.int32, device="cuda")
    out_h = torch.zeros((12, 3, shape.d), dtype=torch.bfloat16, device="cuda")
    ctx.fastmtp_draft(Bd.mtp_w(dW), Bd.bf16_tensor(h[:12]), torch.from_numpy(tok[:12]).cuda(), Bd.kv(sub), 12, 3,
                      torch.from_numpy(ids).cuda(), out_d, out_h)
    torch.cuda.synchronize()
    assert np.array_equal(out_d.cpu().numpy(), a["drafts"][:12])
    assert np.array_equal(out_h.float().cpu().numpy(), a["h_out"][:12])
    ctx.close()


def test_odd_geometry():
    """head_dim 128, 7 query heads per KV head, ffn not a multiple of the tile, V odd-sized."""
    shape = I.Shape(d=448, n_q_heads=7, n_kv_heads=1, head_dim=128, ffn=1200, vocab=3001, n_layers=1,
                    rms_eps=1e-6, rope_theta=1e6, page_size=16)
    got, ref = run_draft_case(shape, 5, 2, [40, 300], 3, 777, subset="zipf")
    check_draft(got, ref, "odd geometry")


def test_full_subset_equals_uncompressed_head():
    """Eq. 3 with the subset covering the vocabulary reproduces the full head."""
    got_full, _ = run_draft_case(I.TINY, 99, 2, [20, 33], 3, None)
    Bd = _binding()
    shape = I.TINY
    # same case, subset = a permutation of the whole vocabulary
    W = I.mtp_weights(shape, 99)
    kv = I.paged_kv(shape, [20, 33], 4, 100)
    h = I.hidden_bf16(101, (2, shape.d))
    tok = I.token_ids(102, (2,), shape.vocab)
    perm = I.subset_uniform(shape.vocab, shape.vocab, 7)
    ctx = Bd.Context(shape, max_rows=8, max_K=8, max_ctx=64)
    dW, dkv = Bd.to_device(W), Bd.to_device(kv)
    out_d = torch.zeros((2, 3), dtype=torch.int32, device="cuda")
    ctx.fastmtp_draft(Bd.mtp_w(dW), Bd.bf16_tensor(h), torch.from_numpy(tok).cuda(), Bd.kv(dkv), 2, 3,
                      torch.from_numpy(perm).cuda(), out_d)
    torch.cuda.synchronize()
    assert np.array_equal(out_d.cpu().numpy(), got_full["drafts"])
    ctx.close()


def test_run_to_run_bit_reproducible():
    a, _ = run_draft_case(I.TINY, 5150, 4, [64, 100, 7, 129], 3, 1024)
    b, _ = run_draft_case(I.TINY, 5150, 4, [64, 100, 7, 129], 3, 1024)
    assert np.array_equal(a["drafts"], b["drafts"])
    assert np.array_equal(a["h_out"], b["h_out"])
    assert np.array_equal(a["logits"], b["logits"])
    assert np.array_equal(a["k_pages"], b["k_pages"])


def test_row_results_do_not_depend_on_batch():
    """A sequence's drafts and hidden states are the same alone and inside a batch."""
    Ls = [64, 100, 7]
    full, _ = run_draft_case(I.TINY, 4242, 3, Ls, 3, 1024)
    Bd = _binding()
    shape = I.TINY
    W = I.mtp_weights(shape, 4242)
    kv = I.paged_kv(shape, Ls, 4, 4243)
    h = I.hidden_bf16(4244, (3, shape.d))
    tok = I.token_ids(4245, (3,), shape.vocab)
    ids = I.subset_uniform(shape.vocab, 1024, 4246)
    dW = Bd.to_device(W)
    for b in range(3):
        ctx = Bd.Context(shape, max_rows=8, max_K=8, max_ctx=128)
        dkv = Bd.to_device(copy_kv(kv))
        one = dict(dkv)
        one["block_table"] = dkv["block_table"][b:b + 1].contiguous()
        one["seq_lens"] = dkv["seq_lens"][b:b + 1].contiguous()
        out_d = torch.zeros((1, 3), dtype=torch.int32, device="cuda")
        out_h = torch.zeros((1, 3, shape.d), dtype=torch.bfloat16, device="cuda")
        ctx.fastmtp_draft(Bd.mtp_w(dW), Bd.bf16_tensor(h[b:b + 1]), torch.from_numpy(tok[b:b + 1]).cuda(),
                          Bd.kv(one), 1, 3, torch.from_numpy(ids).cuda(), out_d, out_h)
        torch.cuda.synchronize()
        assert np.array_equal(out_d.cpu().numpy()[0], full["drafts"][b])
        assert np.array_equal(out_h.float().cpu().numpy()[0], full["h_out"][b])
        ctx.close()


def test_bad_inputs_are_flagged_not_faulted():
    """Out-of-range token / subset ids are clamped and reported through the status word."""
    Bd = _binding()
    shape = I.TINY
    W = I.mtp_weights(shape, 3)
    kv = I.paged_kv(shape, [10], 4, 4)
    ctx = Bd.Context(shape, max_rows=8, max_K=8, max_ctx=32)
    dW, dkv = Bd.to_device(W), Bd.to_device(kv)
    h = Bd.bf16_tensor(I.hidden_bf16(5, (1, shape.d)))
    tok = torch.tensor([shape.vocab + 5], dtype=torch.int32, device="cuda")
    ids = torch.tensor([1, 2, shape.vocab, 3, -1, 9, 10, 11], dtype=torch.int32, device="cuda")
    out_d = torch.zeros((1, 2), dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ctx.fastmtp_draft(Bd.mtp_w(dW), h, tok, Bd.kv(dkv), 1, 2, ids, out_d, None, None, status)
    torch.cuda.synchronize()
    assert int(status.item()) & Bd.DEV_BAD_TOKEN
    # host-side validation: too many rows / steps, null pointers
    with pytest.raises(Bd.FastMTPError):
        ctx.fastmtp_draft(Bd.mtp_w(dW), h, tok, Bd.kv(dkv), 9, 2, ids, out_d)
    with pytest.raises(Bd.FastMTPError):
        ctx.fastmtp_draft(Bd.mtp_w(dW), h, tok, Bd.kv(dkv), 1, 9, ids, out_d)
    with pytest.raises(Bd.FastMTPError):
        ctx.fastmtp_draft(Bd.mtp_w(dW), None, tok, Bd.kv(dkv), 1, 2, ids, out_d)
    ctx.close()


def _extend_case(shape, seed, L, n_ext, max_ext, K, N):
    """Seeded inputs of a draft call with extend rows: h_last [B, max_ext, d], tok_last [B, max_ext]; the rows beyond
    n_ext[b] are padding and are filled with NaN patterns and an invalid token so that any use of them shows."""
    B = len(L)
    W = I.mtp_weights(shape, seed)
    kv = I.paged_kv(shape, list(L), max_ext + K, seed + 1)
    h = I.hidden_bf16(seed + 2, (B, max_ext, shape.d))
    tok = I.token_ids(seed + 3, (B, max_ext), shape.vocab)
    for b in range(B):
        h[b, n_ext[b]:] = 0x7FC0
        tok[b, n_ext[b]:] = -7
    ids = None if N is None else I.subset_uniform(shape.vocab, N, seed + 4)
    return W, kv, h, tok, ids


def _run_extend(Bd, shape, W, kv, h, tok, ids, n_ext, max_ext, K, max_ctx, pass_n_ext=True):
    B = h.shape[0]
    ctx = Bd.Context(shape, max_rows=max(8, B * max_ext), max_K=8, max_ctx=max_ctx)
    dW, dkv = Bd.to_device(W), Bd.to_device(copy_kv(kv))
    out_d = torch.full((B, K), -1, dtype=torch.int32, device="cuda")
    out_h = torch.zeros((B, K, shape.d), dtype=torch.bfloat16, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    dn = torch.tensor(list(n_ext), dtype=torch.int32, device="cuda") if pass_n_ext else None
    ctx.fastmtp_draft(Bd.mtp_w(dW), Bd.bf16_tensor(h), torch.from_numpy(tok).cuda(), Bd.kv(dkv), B, K,
                      None if ids is None else torch.from_numpy(ids).cuda(), out_d, out_h, None, st, n_ext=dn, max_ext=max_ext)
    torch.cuda.synchronize()
    res = {"drafts": out_d.cpu().numpy(), "h_out": out_h.float().cpu().numpy(), "h_bits": Bd.bf16_bits(out_h),
           "status": int(st.item()), "k_pages": Bd.bf16_bits(dkv["k_pages"]), "v_pages": Bd.bf16_bits(dkv["v_pages"]),
           "launches": ctx.launch_count}
    ctx.close()
    return res


@pytest.mark.parametrize("L,n_ext,max_ext,K,N", [
    ([64], [3], 4, 3, 1024),                         # one sequence, a padding row, persistent kernel
    ([5, 130], [1, 4], 4, 2, 1000),                  # eight activation rows in one launch, contexts across a chunk edge
    ([0], [8], 8, 3, None),                          # a whole short prompt as extend rows into an empty cache; full vocabulary
    ([3, 17, 64, 127, 200, 9, 31, 250, 77, 140, 15, 1], [1, 4, 2, 3, 4, 1, 2, 3, 4, 1, 2, 3], 4, 3, 1024),   # batched path, one pass
    (list(range(0, 400, 10)), [1 + (7 * b) % 3 for b in range(40)], 3, 2, 777),                             # 120 rows: two passes of 63
])
def test_extend_rows_in_one_call_match_the_oracle(L, n_ext, max_ext, K, N):
    """Sec. 2.3 "Drafting phase", step k = 1: the pairs (target hidden state, next token) of the positions committed
    since the last call run through the MTP module in one pass, causal among themselves; only the last one feeds the
    head. Drafts, hidden states and both caches against the oracle, sequence by sequence (each with its own n_ext)."""
    Bd = _binding()
    shape, seed = I.TINY, 300 + len(L)
    W, kv, h, tok, ids = _extend_case(shape, seed, L, n_ext, max_ext, K, N)
    got = _run_extend(Bd, shape, W, kv, h, tok, ids, n_ext, max_ext, K, max(L) + max_ext + K + 1)
    assert got["status"] == 0, f"device status {got['status']:#x}"
    okv = copy_kv(kv)
    exempt = 0
    for b in range(len(L)):
        one = dict(okv)                               # pools shared (written in place), tables of sequence b
        one["block_table"], one["seq_lens"] = okv["block_table"][b:b + 1], okv["seq_lens"][b:b + 1]
        ref = O.draft(shape, W, h[b:b + 1, :n_ext[b]], tok[b:b + 1, :n_ext[b]], one, K, ids, forced=got["drafts"][b:b + 1])
        exempt += ids_match(got["drafts"][b], ref["drafts"], ref["gap"], f"extend drafts b={b}")
        close(got["h_out"][b:b + 1], ref["h_out"], f"extend h_out b={b}")
    close(O.bf16_to_f64(got["k_pages"]), O.bf16_to_f64(okv["k_pages"]), "extend K cache")
    close(O.bf16_to_f64(got["v_pages"]), O.bf16_to_f64(okv["v_pages"]), "extend V cache")
    if len(L) >= 12:
        assert got["launches"] > 3                    # the batched path ran


def test_extend_in_one_call_equals_one_pair_per_call_bit_for_bit():
    """On the persistent path three extend rows in one call give the bits of three calls with one pair each (the
    first two with K = 1, their drafts discarded): a row's arithmetic does not depend on the rows beside it."""
    Bd = _binding()
    shape, seed, K = I.TINY, 4100, 3
    L, n = [70, 9], 3
    W, kv, h, tok, ids = _extend_case(shape, seed, L, [n, n], n, K, 1024)
    one = _run_extend(Bd, shape, W, kv, h, tok, ids, [n, n], n, K, 128, pass_n_ext=False)
    ctx = Bd.Context(shape, max_rows=8, max_K=8, max_ctx=128)
    dW, dkv = Bd.to_device(W), Bd.to_device(copy_kv(kv))
    out_d = torch.full((2, K), -1, dtype=torch.int32, device="cuda")
    out_h = torch.zeros((2, K, shape.d), dtype=torch.bfloat16, device="cuda")
    dids = torch.from_numpy(ids).cuda()
    for m in range(n):
        steps = K if m == n - 1 else 1
        ctx.fastmtp_draft(Bd.mtp_w(dW), Bd.bf16_tensor(np.ascontiguousarray(h[:, m])), torch.from_numpy(np.ascontiguousarray(tok[:, m])).cuda(),
                          Bd.kv(dkv), 2, steps, dids, out_d[:, :steps].contiguous() if steps < K else out_d,
                          None if steps < K else out_h)
        dkv["seq_lens"] += 1
    torch.cuda.synchronize()
    assert np.array_equal(out_d.cpu().numpy(), one["drafts"])
    assert np.array_equal(Bd.bf16_bits(out_h), one["h_bits"])
    assert np.array_equal(Bd.bf16_bits(dkv["k_pages"]), one["k_pages"]) and np.array_equal(Bd.bf16_bits(dkv["v_pages"]), one["v_pages"])
    ctx.close()


@pytest.mark.parametrize("B", [2, 10])
def test_positions_beyond_the_cache_are_flagged_and_leave_other_sequences_alone(B):
    """Sequence 0 sits two tokens below the end of its block table (and of max_ctx) and is asked for three
    draft steps: the step without a slot is flagged FMTP_DEV_BAD_POS, nothing is written outside the
    workspace or the pages, and every other sequence of the launch gives the bits it gives in a call
    of its own. B = 2 runs in the persistent kernel, B = 10 on the batched path."""
    Bd = _binding()
    shape, K, seed = I.TINY, 3, 900 + B
    L = [62] + [20 + 3 * b for b in range(1, B)]
    W = I.mtp_weights(shape, seed)
    kv = I.paged_kv(shape, L, 2, seed + 1)                 # 64 slots for sequence 0: positions 62, 63 exist, 64 does not
    assert kv["max_pages_per_seq"] * shape.page_size == 64
    h = I.hidden_bf16(seed + 2, (B, shape.d))
    tok = I.token_ids(seed + 3, (B,), shape.vocab)
    ids = torch.from_numpy(I.subset_uniform(shape.vocab, 1024, seed + 4)).cuda()
    dW = Bd.to_device(W)

    def run(rows):
        ctx = Bd.Context(shape, max_rows=16, max_K=8, max_ctx=64)
        dkv = Bd.to_device(copy_kv(kv))
        sub = dict(dkv)
        sub["block_table"] = dkv["block_table"][rows].contiguous()
        sub["seq_lens"] = dkv["seq_lens"][rows].contiguous()
        n = len(rows)
        out_d = torch.full((n, K), -1, dtype=torch.int32, device="cuda")
        out_h = torch.zeros((n, K, shape.d), dtype=torch.bfloat16, device="cuda")
        st = torch.zeros(1, dtype=torch.int32, device="cuda")
        ctx.fastmtp_draft(Bd.mtp_w(dW), Bd.bf16_tensor(h[rows]), torch.from_numpy(tok[rows]).cuda(), Bd.kv(sub), n, K,
                          ids, out_d, out_h, None, st)
        torch.cuda.synchronize()
        res = out_d.cpu().numpy(), out_h.float().cpu().numpy(), int(st.item()), Bd.bf16_bits(dkv["k_pages"])
        ctx.close()
        return res

    d_all, h_all, st_all, k_all = run(list(range(B)))
    assert st_all & Bd.DEV_BAD_POS and not st_all & Bd.DEV_TIMEOUT
    d_rest, h_rest, st_rest, k_rest = run(list(range(1, B)))
    assert st_rest == 0
    assert np.array_equal(d_all[1:], d_rest) and np.array_equal(h_all[1:], h_rest)
    # the pages of the other sequences hold the same bits; sequence 0's first two steps are in range and correct
    own0 = set(int(x) for x in kv["block_table"][0] if x >= 0)
    others = [pg for pg in range(kv["num_pages"]) if pg not in own0]
    assert np.array_equal(k_all[others], k_rest[others])
    okv = copy_kv(kv)
    okv["block_table"], okv["seq_lens"] = okv["block_table"][:1], okv["seq_lens"][:1]
    ref = O.draft(shape, W, h[:1], tok[:1], okv, 2, ids.cpu().numpy(), forced=d_all[:1, :2])
    ids_match(d_all[:1, :2], ref["drafts"], ref["gap"], "in-range steps of the overflowing sequence")
    close(h_all[:1, :2], ref["h_out"], "in-range steps of the overflowing sequence")


@pytest.mark.parametrize("B,K", [(1, 3), (20, 3), (64, 2)])
def test_draft_call_captured_in_a_cuda_graph_replays_on_the_current_state(B, K):
    """One fastmtp_draft call (all K steps; the persistent kernel at B = 1, the batched path's chain of kernels
    otherwise) is captured into a CUDA graph and replayed after the sequences have advanced and the inputs have
    changed: sequence lengths, block tables, tokens and hidden states are read on the device, so the replay gives the
    bits of an eager call on the same state."""
    Bd = _binding()
    shape, seed = I.TINY, 6100 + B
    L = [int(x) for x in I.context_lengths(B, 0, 150, seed)]
    W = I.mtp_weights(shape, seed)
    kv = I.paged_kv(shape, L, K + 2, seed + 1)
    dW, dkv = Bd.to_device(W), Bd.to_device(copy_kv(kv))
    dh = Bd.bf16_tensor(I.hidden_bf16(seed + 2, (B, shape.d)))
    dtok = torch.from_numpy(I.token_ids(seed + 3, (B,), shape.vocab)).cuda()
    dids = torch.from_numpy(I.subset_uniform(shape.vocab, 1024, seed + 4)).cuda()
    ctx = Bd.Context(shape, max_rows=max(8, B), max_K=8, max_ctx=max(L) + K + 3)
    out_d = torch.full((B, K), -1, dtype=torch.int32, device="cuda")
    out_h = torch.zeros((B, K, shape.d), dtype=torch.bfloat16, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    w, ckv = Bd.mtp_w(dW), Bd.kv(dkv)

    def call():
        ctx.fastmtp_draft(w, dh, dtok, ckv, B, K, dids, out_d, out_h, None, st)

    call()                                       # eager warm-up: set-up that belongs outside a capture happens here
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.graph(graph, stream=side):
        call()
    # the state moves on: one more committed token per sequence, new inputs
    dkv["seq_lens"] += 1
    dh.copy_(Bd.bf16_tensor(I.hidden_bf16(seed + 5, (B, shape.d))))
    dtok.copy_(torch.from_numpy(I.token_ids(seed + 6, (B,), shape.vocab)).cuda())
    torch.cuda.synchronize()
    k0, v0 = dkv["k_pages"].clone(), dkv["v_pages"].clone()
    out_d.fill_(-1); out_h.zero_()
    graph.replay()
    torch.cuda.synchronize()
    g_d, g_h, g_k, g_v = out_d.clone(), out_h.clone(), dkv["k_pages"].clone(), dkv["v_pages"].clone()
    assert int(st.item()) == 0
    dkv["k_pages"].copy_(k0); dkv["v_pages"].copy_(v0)
    out_d.fill_(-1); out_h.zero_()
    call()
    torch.cuda.synchronize()
    assert torch.equal(out_d, g_d) and torch.equal(out_h, g_h)
    assert torch.equal(dkv["k_pages"], g_k) and torch.equal(dkv["v_pages"], g_v)
    assert (g_d >= 0).all()
    ctx.close()


@pytest.mark.parametrize("which,B", [(1, 2), (2, 12)])
def test_a_wait_inside_the_draft_kernels_runs_out_and_the_context_stays_usable(which, B):
    """Failure detection without a fault, in the kernels' own code: the next draft call is armed so that the
    persistent kernel's grid barrier (which = 1) or a ring stage of the batched path's first GEMM (which = 2) waits
    for an arrival that never comes, with a 20 ms limit. The wait gives up, FMTP_DEV_TIMEOUT reaches the status word,
    the other CTAs and warp roles stop waiting, the call returns in bounded time, and the same context then gives the
    bits it gave before."""
    import time
    Bd = _binding()
    shape, K, seed = I.TINY, 2, 7300 + which
    L = [int(x) for x in I.context_lengths(B, 0, 100, seed)]
    W = I.mtp_weights(shape, seed)
    kv = I.paged_kv(shape, L, K + 1, seed + 1)
    dW = Bd.to_device(W)
    dh = Bd.bf16_tensor(I.hidden_bf16(seed + 2, (B, shape.d)))
    dtok = torch.from_numpy(I.token_ids(seed + 3, (B,), shape.vocab)).cuda()
    dids = torch.from_numpy(I.subset_uniform(shape.vocab, 1024, seed + 4)).cuda()
    ctx = Bd.Context(shape, max_rows=16, max_K=8, max_ctx=128)

    def run():
        dkv = Bd.to_device(copy_kv(kv))
        out_d = torch.full((B, K), -1, dtype=torch.int32, device="cuda")
        out_h = torch.zeros((B, K, shape.d), dtype=torch.bfloat16, device="cuda")
        st = torch.zeros(1, dtype=torch.int32, device="cuda")
        t0 = time.time()
        ctx.fastmtp_draft(Bd.mtp_w(dW), dh, dtok, Bd.kv(dkv), B, K, dids, out_d, out_h, None, st)
        torch.cuda.synchronize()
        return out_d.cpu().numpy(), Bd.bf16_bits(out_h), int(st.item()), time.time() - t0

    d0, h0, st0, _ = run()
    assert st0 == 0
    ctx.fmtp_selftest_inject_wait_timeout(20, which)
    _, _, st1, dt = run()
    assert st1 & Bd.DEV_TIMEOUT
    assert 0.015 < dt < 2.0                                  # gave up soon after the limit, nothing hung
    d2, h2, st2, _ = run()                                   # the arming was for one call; tensor memory and barriers are clean
    assert st2 == 0 and np.array_equal(d2, d0) and np.array_equal(h2, h0)
    with pytest.raises(Bd.FastMTPError):
        ctx.fmtp_selftest_inject_wait_timeout(5000, which)   # limits above one second are refused on the host
    ctx.close()


def test_host_entry_point_matches_device_entry_point():
    Bd = _binding()
    shape = I.TINY
    W = I.mtp_weights(shape, 11)
    kv = I.paged_kv(shape, [64, 9], 4, 12)
    h = I.hidden_bf16(13, (2, shape.d))
    tok = I.token_ids(14, (2,), shape.vocab)
    ids = torch.from_numpy(I.subset_uniform(shape.vocab, 1024, 15)).cuda()
    dW = Bd.to_device(W)
    ctx = Bd.Context(shape, max_rows=8, max_K=8, max_ctx=128)
    dkv = Bd.to_device(copy_kv(kv))
    out_d = torch.zeros((2, 3), dtype=torch.int32, device="cuda")
    ctx.fastmtp_draft(Bd.mtp_w(dW), Bd.bf16_tensor(h), torch.from_numpy(tok).cuda(), Bd.kv(dkv), 2, 3, ids, out_d)
    torch.cuda.synchronize()
    dkv2 = Bd.to_device(copy_kv(kv))
    out_host = torch.zeros((2, 3), dtype=torch.int32)
    ctx.fastmtp_draft_host(Bd.mtp_w(dW), Bd.bf16_tensor(h, "cpu"), torch.from_numpy(tok), Bd.kv(dkv2), 2, 3, ids,
                           out_host)
    assert np.array_equal(out_host.numpy(), out_d.cpu().numpy())
    ctx.close()
