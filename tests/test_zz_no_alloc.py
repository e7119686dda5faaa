"""fastmtp_verify_accept_static: the verification entry point for callers that cannot allocate.

A host that has given all device memory to its own pool, or that sits inside a decode loop where an
allocation would stall the GPU, cannot provide the workspace the regular call needs; this entry point
keeps its scratch in a fixed array inside the library. The test calls it through the C ABI twice in a
row (the second call finds the first one's leftovers in the shared array) and compares with the
regular entry point and with the oracle's verification of the same logits. Integer results: bit-exact.
It also checks what the call exists for: device memory in use is the same before and after the calls.
Collected last on purpose, so a run that stops at the first failure has already run everything else.
"""
import numpy as np
import pytest
import torch

from oracle import fastmtp_oracle as O
from paper_2509_18362_b200 import inputs as I

pytestmark = pytest.mark.gpu


def _regular(Bd, ctx, logits, drafts, B, K, V):
    acc = torch.full((B,), -1, dtype=torch.int32, device="cuda")
    bon = torch.full((B,), -1, dtype=torch.int32, device="cuda")
    arg = torch.full((B, K + 1), -1, dtype=torch.int32, device="cuda")
    ctx.fastmtp_verify_accept(logits, drafts, B, K, V, acc, bon, arg)
    torch.cuda.synchronize()
    return acc.cpu().numpy(), bon.cpu().numpy(), arg.cpu().numpy()


def _static(Bd, logits, drafts, B, K, V):
    acc = torch.full((B,), -1, dtype=torch.int32, device="cuda")
    bon = torch.full((B,), -1, dtype=torch.int32, device="cuda")
    arg = torch.full((B, K + 1), -1, dtype=torch.int32, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    Bd.fastmtp_verify_accept_static(logits, drafts, B, K, V, acc, bon, arg, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    return acc.cpu().numpy(), bon.cpu().numpy(), arg.cpu().numpy()


def test_static_entry_point_matches_regular_one_on_two_calls_in_a_row():
    from paper_2509_18362_b200 import binding as Bd
    ctx = Bd.Context(I.TINY, max_rows=8, max_K=8, max_ctx=64)
    cases = [I.verify_case(37, 3, 20011, 901), I.verify_case(5, 6, 4096, 902)]   # different row counts
    for case in cases:
        B, M, V = case["logits"].shape
        K = M - 1
        dl = Bd.bf16_tensor(case["logits"])
        dd = torch.from_numpy(case["drafts"]).cuda()
        want = _regular(Bd, ctx, dl, dd, B, K, V)
        got = _static(Bd, dl, dd, B, K, V)
        for w, g in zip(want, got):
            assert np.array_equal(w, g)
        assert np.array_equal(got[0], case["length"])            # and the planted answer
        ra, rb, rg = O.verify_accept(case["logits"], case["drafts"])
        assert np.array_equal(got[0], ra) and np.array_equal(got[1], rb) and np.array_equal(got[2], rg)
    # the same inputs once more: the array still holds the previous call's contents. Around these calls (the
    # entry point's per-device set-up happened above) the device's free memory and torch's own
    # allocations must not move: the call creates no device memory, directly or through a library.
    acc = torch.full((B,), -1, dtype=torch.int32, device="cuda")
    bon = torch.full((B,), -1, dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    free0, alloc0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated()
    for _ in range(2):
        Bd.fastmtp_verify_accept_static(dl, dd, B, K, V, acc, bon)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free0 and torch.cuda.memory_allocated() == alloc0
    assert np.array_equal(acc.cpu().numpy(), got[0]) and np.array_equal(bon.cpu().numpy(), got[1])
    ctx.close()


def test_static_entry_point_rejects_sizes_beyond_its_fixed_scratch():
    from paper_2509_18362_b200 import binding as Bd
    B, K, V = Bd.STATIC_VERIFY_MAX_ROWS // 2 + 1, 1, 64          # B * (K + 1) = limit + 2
    logits = torch.zeros((B, K + 1, V), dtype=torch.bfloat16, device="cuda")
    drafts = torch.zeros((B, K), dtype=torch.int32, device="cuda")
    acc = torch.zeros(B, dtype=torch.int32, device="cuda")
    with pytest.raises(Bd.FastMTPError) as e:
        Bd.fastmtp_verify_accept_static(logits, drafts, B, K, V, acc, acc.clone())
    assert e.value.code == -2
