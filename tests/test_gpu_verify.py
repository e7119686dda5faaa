"""GPU parity of fastmtp_verify_accept against the CPU oracle (bit-exact: integer results)."""
import numpy as np
import pytest
import torch

from oracle import fastmtp_oracle as O
from paper_2509_18362_b200 import inputs as I

pytestmark = pytest.mark.gpu


def _ctx():
    from paper_2509_18362_b200 import binding as Bd
    return Bd, Bd.Context(I.TINY, max_rows=8, max_K=8, max_ctx=64)


def _run(Bd, ctx, logits_bits, drafts, host=False):
    B, M, V = logits_bits.shape
    K = M - 1
    if host:
        acc = torch.zeros(B, dtype=torch.int32)
        bon = torch.zeros(B, dtype=torch.int32)
        ctx.fastmtp_verify_accept_host(Bd.bf16_tensor(logits_bits, "cpu"), torch.from_numpy(drafts), B, K, V, acc, bon)
        return acc.numpy(), bon.numpy(), None
    dl = Bd.bf16_tensor(logits_bits)
    dd = torch.from_numpy(np.ascontiguousarray(drafts)).cuda()
    acc = torch.full((B,), -1, dtype=torch.int32, device="cuda")
    bon = torch.full((B,), -1, dtype=torch.int32, device="cuda")
    arg = torch.full((B, M), -1, dtype=torch.int32, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    ctx.fastmtp_verify_accept(dl, dd if K > 0 else None, B, K, V, acc, bon, arg, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    return acc.cpu().numpy(), bon.cpu().numpy(), arg.cpu().numpy()


@pytest.mark.parametrize("B,K,V", [(1, 3, 4096), (5, 0, 1000), (7, 2, 16385), (64, 3, 152064), (3, 7, 33)])
def test_planted_prefix_lengths(B, K, V):
    Bd, ctx = _ctx()
    case = I.verify_case(B, K, V, 1000 + B)
    a, bonus, g = _run(Bd, ctx, case["logits"], case["drafts"])
    ra, rb, rg = O.verify_accept(case["logits"], case["drafts"])
    assert np.array_equal(a, ra) and np.array_equal(bonus, rb) and np.array_equal(g, rg)
    assert np.array_equal(a, case["length"])          # the planted answer
    # second call on the same context: scratch was cleared by the first
    a2, b2, _ = _run(Bd, ctx, case["logits"], case["drafts"])
    assert np.array_equal(a2, ra) and np.array_equal(b2, rb)
    ctx.close()


def test_natural_ties_go_to_lowest_id():
    """bf16 logits ~N(0,2) tie at the top of a row; both sides must pick the lowest id."""
    Bd, ctx = _ctx()
    logits = I.verify_logits_natural(16, 4, 152064, 7)
    _, _, rg = O.verify_accept(logits, np.zeros((16, 3), np.int32))
    drafts = rg[:, :3].copy()
    drafts[::2, 1] += 1                                  # every other sequence: mismatch at j = 1
    a, bonus, g = _run(Bd, ctx, logits, drafts)
    ra, rb, _ = O.verify_accept(logits, drafts)
    assert np.array_equal(g, rg) and np.array_equal(a, ra) and np.array_equal(bonus, rb)
    ctx.close()


def test_special_values_and_unaligned_rows():
    Bd, ctx = _ctx()
    V = 1001                                             # odd V: rows after the first are not 16-byte aligned
    g = I.rng(3, "special")
    x = g.standard_normal((2, 3, V)).astype(np.float32)
    x[0, 0, 5] = np.nan
    x[0, 0, 17] = np.inf
    x[0, 1, :] = -np.inf
    x[0, 1, 900] = -1e30
    x[1, 0, :] = 0.25                                    # all equal: id 0
    x[1, 2, 1000] = 50.0                                 # winner is the very last element
    bits = I.f32_to_bf16_bits(x).reshape(x.shape)
    bits[0, 0, 5] = 0x7FC0
    drafts = np.array([[17, 900], [0, 3]], dtype=np.int32)
    a, bonus, gg = _run(Bd, ctx, bits, drafts)
    ra, rb, rg = O.verify_accept(bits, drafts)
    assert np.array_equal(gg, rg) and np.array_equal(a, ra) and np.array_equal(bonus, rb)
    assert gg[0, 0] == 17 and gg[0, 1] == 900 and gg[1, 0] == 0 and gg[1, 2] == 1000
    ctx.close()


@pytest.mark.parametrize("B,K,V", [(1, 3, 4096), (5, 0, 1000), (64, 3, 152064), (300, 7, 33)])
def test_accept_on_token_ids_equals_the_oracle(B, K, V):
    """fastmtp_accept_ids consumes the target's per-row greedy tokens instead of logits: same accepted lengths and
    bonus tokens as the oracle's verification of the logits those tokens came from (planted prefixes and natural ties)."""
    Bd, ctx = _ctx()
    case = I.verify_case(B, K, V, 2000 + B)
    for logits, drafts in ((case["logits"], case["drafts"]),
                           (I.verify_logits_natural(min(B, 8), K + 1, V, 5), case["drafts"][:min(B, 8)])):
        ra, rb, rg = O.verify_accept(logits, drafts)
        n = logits.shape[0]
        if K > 0 and n > 1:
            drafts = drafts.copy()
            drafts[1, :K] = rg[1, :K]                      # one fully accepted sequence
            ra, rb, rg = O.verify_accept(logits, drafts)
        acc = torch.full((n,), -1, dtype=torch.int32, device="cuda")
        bon = torch.full((n,), -1, dtype=torch.int32, device="cuda")
        ctx.fastmtp_accept_ids(torch.from_numpy(rg).cuda(), torch.from_numpy(np.ascontiguousarray(drafts)).cuda() if K > 0 else None,
                               n, K, acc, bon)
        torch.cuda.synchronize()
        assert np.array_equal(acc.cpu().numpy(), ra) and np.array_equal(bon.cpu().numpy(), rb)
    ctx.close()


def test_host_entry_point():
    Bd, ctx = _ctx()
    case = I.verify_case(9, 3, 5000, 21)
    a, bonus, _ = _run(Bd, ctx, case["logits"], case["drafts"], host=True)
    ra, rb, _ = O.verify_accept(case["logits"], case["drafts"])
    assert np.array_equal(a, ra) and np.array_equal(bonus, rb)
    ctx.close()


def test_a_wait_that_runs_out_sets_the_timeout_flag_and_leaves_the_device_usable():
    """Failure detection without a fault: the library's bounded wait, given an event that never comes and a
    20 ms limit, reports FMTP_DEV_TIMEOUT through the status word and returns; the next call works."""
    Bd, ctx = _ctx()
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    waited = torch.zeros(1, dtype=torch.int64, device="cuda")
    Bd.fmtp_selftest_wait_timeout(st, 20, waited)
    torch.cuda.synchronize()
    assert int(st.item()) & Bd.DEV_TIMEOUT
    assert 20e6 <= int(waited.item()) < 500e6            # gave up soon after the limit
    with pytest.raises(Bd.FastMTPError):
        Bd.fmtp_selftest_wait_timeout(st, 5000)          # limits above one second are refused on the host
    case = I.verify_case(3, 2, 999, 5)
    a, bonus, _ = _run(Bd, ctx, case["logits"], case["drafts"])
    assert np.array_equal(a, case["length"])
    ctx.close()
