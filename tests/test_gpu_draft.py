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
