"""Pins for the CPU oracle: every check compares the oracle with something other than
itself -- closed forms, invariants the paper states (Eq. 3; Sec. 2.3 losslessness; the
acceptance-length metric of Sec. 3.1), brute force on tiny inputs, or an independent
library implementation (torch CPU ops, the transformers Llama decoder in float64)."""
import itertools
import math
import os
import types

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import fastmtp_oracle as O
from paper_2509_18362_b200 import inputs as I

SMALL = I.Shape(d=64, n_q_heads=4, n_kv_heads=2, head_dim=16, ffn=96, vocab=50, n_layers=2,
                rms_eps=1e-6, rope_theta=1e4, page_size=4)
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _ones_gain(d):
    return I.f32_to_bf16_bits(np.ones(d, dtype=np.float32))


# ------------------------------------------------------------------ bf16 storage format

def test_bf16_roundtrip_matches_torch_library():
    g = np.random.default_rng(0)
    x = np.concatenate([g.standard_normal(20000) * 10.0 ** g.integers(-30, 30, 20000),
                        [0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895313892515355e38, 1e-40, -1e-39]])
    ours = O.f64_to_bf16(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    # torch rounds float64 -> bf16 through float32 (double rounding); exclude the rare inputs
    # whose float32 image sits exactly on a bf16 half-way point
    x32 = x.astype(np.float32)
    halfway = (x32.view(np.uint32) & 0xFFFF) == 0x8000
    assert np.array_equal(ours[~halfway], ref[~halfway])
    assert np.array_equal(O.bf16_to_f64(ref), torch.from_numpy(ref.view(np.int16)).view(torch.bfloat16).double().numpy())


def test_bf16_halfway_goes_to_even():
    # 1 + 2^-8 is half-way between bf16 neighbours 1.0 and 1.0078125 -> even mantissa (1.0)
    assert O.round_bf16(np.array([1.0 + 2.0 ** -8]))[0] == 1.0
    # 1 + 3*2^-8 is half-way between 1.0078125 and 1.015625 -> 1.015625 (even)
    assert O.round_bf16(np.array([1.0 + 3 * 2.0 ** -8]))[0] == 1.015625
    # a hair above half-way must round up even though its float32 image would not
    assert O.round_bf16(np.array([1.0 + 2.0 ** -8 + 2.0 ** -40]))[0] == 1.0078125


def test_generator_bf16_bits_agree_with_torch():
    x = np.random.default_rng(1).standard_normal(10000).astype(np.float32)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(I.f32_to_bf16_bits(x), ref)


# ------------------------------------------------------------------ RMSNorm

def test_rmsnorm_constant_vector_closed_form():
    d, c, eps = 32, 3.0, 1e-6
    out = O.rmsnorm(np.full(d, c), _ones_gain(d), eps)
    assert np.allclose(out, c / math.sqrt(c * c + eps), rtol=0, atol=1e-15)


def test_rmsnorm_matches_torch_library():
    g = np.random.default_rng(2)
    x = g.standard_normal((5, 48))
    gain = I.normal_bf16(3, "g", (48,), 0.02, mean=1.0)
    ref = F.rms_norm(torch.from_numpy(x), (48,), torch.from_numpy(O.bf16_to_f64(gain)), eps=1e-6).numpy()
    assert np.allclose(O.rmsnorm(x, gain, 1e-6), ref, rtol=1e-13, atol=1e-13)


def test_rmsnorm_eps_is_inside_the_root():
    # for x = 0 the output is 0; for tiny x the scale is x / sqrt(eps)
    out = O.rmsnorm(np.full(4, 1e-9), _ones_gain(4), 1e-6)
    assert np.allclose(out, 1e-9 / math.sqrt(1e-18 + 1e-6), rtol=1e-12)


# ------------------------------------------------------------------ rotary embedding

def test_rope_position_zero_is_identity_and_norm_is_kept():
    x = np.random.default_rng(3).standard_normal((3, 16))
    assert np.array_equal(O.rope(x, 0, 1e4), x)
    y = O.rope(x, 37, 1e4)
    assert np.allclose(np.linalg.norm(y, axis=-1), np.linalg.norm(x, axis=-1), rtol=1e-13)


def test_rope_two_dims_is_a_plane_rotation_by_pos():
    # dh = 2: one pair, frequency theta^0 = 1 -> rotation by `pos` radians
    y = O.rope(np.array([1.0, 0.0]), 0.5, 1e4)
    assert np.allclose(y, [math.cos(0.5), math.sin(0.5)], atol=1e-15)


def test_rope_pairing_and_frequency():
    # dh = 4: element 1 pairs with element 3 at frequency theta^(-2/4)
    theta, pos = 1e4, 7
    y = O.rope(np.array([0.0, 1.0, 0.0, 0.0]), pos, theta)
    a = pos * theta ** -0.5
    assert np.allclose(y, [0.0, math.cos(a), 0.0, math.sin(a)], atol=1e-15)


def test_rope_inner_product_depends_on_relative_position_only():
    g = np.random.default_rng(4)
    q, k = g.standard_normal(32), g.standard_normal(32)
    a = O.rope(q, 19, 1e6) @ O.rope(k, 11, 1e6)
    b = O.rope(q, 108, 1e6) @ O.rope(k, 100, 1e6)
    assert abs(a - b) < 1e-11


# ------------------------------------------------------------------ attention, SiLU

def test_attention_single_token_returns_its_value():
    g = np.random.default_rng(5)
    q = g.standard_normal((4, 16))
    K, V = g.standard_normal((1, 2, 16)), g.standard_normal((1, 2, 16))
    out = O.gqa_attention(q, K, V)
    assert np.allclose(out[:2], V[0, 0]) and np.allclose(out[2:], V[0, 1])


def test_attention_identical_keys_gives_mean_value():
    g = np.random.default_rng(6)
    q = g.standard_normal((4, 16))
    K = np.repeat(g.standard_normal((1, 2, 16)), 9, axis=0)
    V = g.standard_normal((9, 2, 16))
    out = O.gqa_attention(q, K, V)
    assert np.allclose(out[0], V[:, 0].mean(0)) and np.allclose(out[3], V[:, 1].mean(0))


def test_attention_matches_torch_sdpa_with_gqa():
    g = np.random.default_rng(7)
    Hq, Hkv, dh, n = 6, 2, 8, 13
    q, K, V = g.standard_normal((Hq, dh)), g.standard_normal((n, Hkv, dh)), g.standard_normal((n, Hkv, dh))
    ref = F.scaled_dot_product_attention(
        torch.from_numpy(q)[None, :, None, :], torch.from_numpy(K).permute(1, 0, 2)[None],
        torch.from_numpy(V).permute(1, 0, 2)[None], enable_gqa=True)[0, :, 0, :].numpy()
    assert np.allclose(O.gqa_attention(q, K, V), ref, rtol=1e-12, atol=1e-12)


def test_silu_matches_torch_and_known_values():
    z = np.linspace(-20, 20, 101)
    assert np.allclose(O.silu(z), F.silu(torch.from_numpy(z)).numpy(), rtol=1e-13, atol=1e-15)
    assert O.silu(np.array([0.0]))[0] == 0.0
    assert abs(O.silu(np.array([1.0]))[0] - 1.0 / (1.0 + math.exp(-1.0))) < 1e-15


# ------------------------------------------------------------------ decoder stack vs an independent library model

def _hf_model(shape, Wt):
    from transformers import LlamaConfig, LlamaForCausalLM
    cfg = LlamaConfig(hidden_size=shape.d, intermediate_size=shape.ffn, num_hidden_layers=shape.n_layers,
                      num_attention_heads=shape.n_q_heads, num_key_value_heads=shape.n_kv_heads,
                      head_dim=shape.head_dim, vocab_size=shape.vocab, rms_norm_eps=shape.rms_eps,
                      rope_theta=shape.rope_theta, attention_bias=False, mlp_bias=False,
                      tie_word_embeddings=False, max_position_embeddings=512)
    m = LlamaForCausalLM(cfg).double().eval()
    t = lambda bits: torch.from_numpy(O.bf16_to_f64(bits))
    sd = {"model.embed_tokens.weight": t(Wt["embed"]), "lm_head.weight": t(Wt["lm_head"]),
          "model.norm.weight": t(Wt["g_final"])}
    for i, lw in enumerate(Wt["layers"]):
        p = f"model.layers.{i}."
        sd.update({p + "self_attn.q_proj.weight": t(lw["wq"]), p + "self_attn.k_proj.weight": t(lw["wk"]),
                   p + "self_attn.v_proj.weight": t(lw["wv"]), p + "self_attn.o_proj.weight": t(lw["wo"]),
                   p + "mlp.gate_proj.weight": t(lw["w_gate"]), p + "mlp.up_proj.weight": t(lw["w_up"]),
                   p + "mlp.down_proj.weight": t(lw["w_down"]), p + "input_layernorm.weight": t(lw["g_in"]),
                   p + "post_attention_layernorm.weight": t(lw["g_post"])})
    missing, unexpected = m.load_state_dict(sd, strict=False)
    assert not unexpected and all("rotary" in k or "inv_freq" in k for k in missing), (missing, unexpected)
    return m


def test_target_stack_matches_transformers_llama_float64():
    """The full target forward (embedding, pre-norm layers with rotary GQA attention over a
    paged cache, SwiGLU, final norm, output head) against the transformers Llama decoder.
    The only modelling difference is that the oracle stores K/V as bf16 (relative 2^-9), so
    agreement is to ~1e-2 of the logit scale: a wrong sign, pairing, head mapping, norm
    placement or transposed operand is off by the scale itself."""
    shape = SMALL
    # weights with std 0.15 so that attention and MLP contribute at the scale of the residual
    Wt = I.target_weights(shape, 11)
    for lw in Wt["layers"]:
        for k in ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down"):
            lw[k] = I.normal_bf16(12, k + str(id(lw) % 7), lw[k].shape, 0.15)
    Wt["embed"] = I.normal_bf16(13, "e", Wt["embed"].shape, 1.0)
    Wt["lm_head"] = I.normal_bf16(13, "h", Wt["lm_head"].shape, 0.15)
    toks = I.token_ids(14, (1, 11), shape.vocab)
    kvs = [I.empty_paged_kv(shape, 1, 16, 15 + l) for l in range(shape.n_layers)]
    h, logits = O.target_forward(shape, Wt, toks, kvs)
    with torch.no_grad():
        out = _hf_model(shape, Wt)(torch.from_numpy(toks.astype(np.int64)), output_hidden_states=True)
    ref_logits = out.logits[0].numpy()
    ref_h = out.hidden_states[-1][0].numpy()
    scale = ref_logits.std()
    assert np.abs(logits[0] - ref_logits).max() < 2e-2 * scale
    assert np.abs(h[0] - ref_h).max() < 2e-2 * ref_h.std()
    # structural sensitivity of this pin: a different rotary pairing would miss by far more
    assert scale > 0.5


def test_incremental_decode_equals_prefill_and_paging_is_transparent():
    shape = SMALL
    Wt = I.target_weights(shape, 21)
    toks = I.token_ids(22, (1, 9), shape.vocab)
    kv_a = [I.empty_paged_kv(shape, 1, 12, 30 + l) for l in range(shape.n_layers)]
    kv_b = [I.empty_paged_kv(shape, 1, 12, 40 + l) for l in range(shape.n_layers)]   # other page order
    _, full = O.target_forward(shape, Wt, toks, kv_a)
    rows = []
    for m in range(toks.shape[1]):
        _, lg = O.target_forward(shape, Wt, toks[:, m:m + 1], kv_b)
        for kv in kv_b:
            kv["seq_lens"][0] += 1
        rows.append(lg[0, 0])
    assert np.array_equal(np.stack(rows), full[0])


def test_layer_with_zero_output_projections_is_identity():
    shape = SMALL
    lw = I.layer_weights(shape, 5, "l")
    lw["wo"] = np.zeros_like(lw["wo"])
    lw["w_down"] = np.zeros_like(lw["w_down"])
    kv = I.empty_paged_kv(shape, 1, 8, 6)
    x = np.random.default_rng(8).standard_normal(shape.d)
    assert np.array_equal(O.decoder_layer(x, 0, lw, kv, 0, shape), x)


# ------------------------------------------------------------------ MTP module (Sec. 2.1)

def _mtp_case(seed=31, shape=SMALL):
    W = I.mtp_weights(shape, seed)
    kv = I.paged_kv(shape, [6], 8, seed + 1)
    h = O.bf16_to_f64(I.hidden_bf16(seed + 2, (shape.d,)))
    return shape, W, kv, h


def test_mtp_projection_reads_hidden_half_then_embedding_half():
    """W_p = [I 0] must give x = RMSNorm_h(h); W_p = [0 I] must give x = RMSNorm_e(Emb(t));
    with the layer's output projections zeroed the module then returns RMSNorm_final(x)."""
    shape, W, kv, h = _mtp_case()
    d = shape.d
    W["layer"]["wo"] = np.zeros_like(W["layer"]["wo"])
    W["layer"]["w_down"] = np.zeros_like(W["layer"]["w_down"])
    eye = I.f32_to_bf16_bits(np.eye(d, dtype=np.float32))
    zero = np.zeros((d, d), dtype=np.uint16)
    tok = 17
    W["w_proj"] = np.concatenate([eye, zero], axis=1)
    got = O.mtp_forward(h, tok, 6, W, kv, 0, shape)
    want = O.rmsnorm(O.rmsnorm(h, W["g_hnorm"], shape.rms_eps), W["g_final"], shape.rms_eps)
    assert np.allclose(got, want, rtol=1e-13, atol=1e-13)
    W["w_proj"] = np.concatenate([zero, eye], axis=1)
    got = O.mtp_forward(h, tok, 6, W, kv, 0, shape)
    e = O.bf16_to_f64(W["embed"][tok])
    want = O.rmsnorm(O.rmsnorm(e, W["g_enorm"], shape.rms_eps), W["g_final"], shape.rms_eps)
    assert np.allclose(got, want, rtol=1e-13, atol=1e-13)


def test_mtp_projection_is_linear_in_the_two_halves():
    shape, W, kv, h = _mtp_case(41)
    d = shape.d
    W["layer"]["wo"] = np.zeros_like(W["layer"]["wo"])
    W["layer"]["w_down"] = np.zeros_like(W["layer"]["w_down"])
    W["g_final"] = _ones_gain(d)
    tok = 3
    # undo the final norm's scale by comparing directions and norms separately is awkward;
    # instead compare un-normalised x through a final norm on both sides (torch library ops)
    Wp = torch.from_numpy(O.bf16_to_f64(W["w_proj"]))
    hh = F.rms_norm(torch.from_numpy(h), (d,), torch.from_numpy(O.bf16_to_f64(W["g_hnorm"])), eps=shape.rms_eps)
    ee = F.rms_norm(torch.from_numpy(O.bf16_to_f64(W["embed"][tok])), (d,),
                    torch.from_numpy(O.bf16_to_f64(W["g_enorm"])), eps=shape.rms_eps)
    x = Wp[:, :d] @ hh + Wp[:, d:] @ ee
    want = F.rms_norm(x, (d,), None, eps=shape.rms_eps).numpy()
    got = O.mtp_forward(h, tok, 6, W, kv, 0, shape)
    assert np.allclose(got, want, rtol=1e-12, atol=1e-12)


def test_mtp_head_parameter_count():
    # closed form vs the element count of independently generated tensors
    for shape in (I.TINY, SMALL):
        W = I.mtp_weights(shape, 1)
        n = sum(v.size for k, v in W.items() if k not in ("embed", "lm_head", "layer"))
        n += sum(v.size for v in W["layer"].values())
        assert O.mtp_param_count(shape) == n
    assert O.mtp_param_count(I.TINY) == 857_344
    assert O.mtp_param_count(I.QWEN7B) == 258_754_048
    # the head is a small fraction of a 7B-class model, no V x d matrix of its own (Sec. 3.1: < 3 %)
    seven_b = 28 * (O.mtp_param_count(I.QWEN7B) - 2 * 3584 * 3584) + 2 * 152064 * 3584
    assert O.mtp_param_count(I.QWEN7B) / seven_b < 0.04


# ------------------------------------------------------------------ compressed head (Eq. 3)

@pytest.mark.parametrize("V,N", [(16, 5), (257, 64), (4096, 1024)])
def test_compressed_head_invariants(V, N):
    d = 32
    lm = I.normal_bf16(51, f"lm{V}", (V, d), 0.5)
    hits = 0
    for trial in range(40):
        h = np.random.default_rng(100 + trial).standard_normal(d)
        full = O.head_logits(h, lm)
        ids = I.subset_uniform(V, N, 200 + trial)
        comp = O.head_logits(h, lm, ids)
        # Eq. 3: row i of the compressed head is row ids[i] of the full head
        assert np.array_equal(comp, full[ids])
        t_full, _ = O.argmax_token(full)
        t_comp, _ = O.argmax_token(comp, ids)
        assert t_comp in set(ids.tolist())
        if t_full in set(ids.tolist()):
            hits += 1
            assert t_comp == t_full                       # I1
        else:
            assert full[t_comp] <= full[t_full]
        # I2: the identity subset reproduces the uncompressed head bit for bit
        ident = np.arange(V, dtype=np.int32)
        assert np.array_equal(O.head_logits(h, lm, ident), full)
        assert O.argmax_token(O.head_logits(h, lm, ident), ident)[0] == t_full
    assert hits > 0


def test_argmax_rule_brute_force():
    g = np.random.default_rng(9)
    for trial in range(300):
        n = int(g.integers(1, 9))
        vals = g.integers(-2, 3, n).astype(np.float64)            # many ties
        if trial % 5 == 0:
            vals[g.integers(0, n)] = np.nan
        ids = g.permutation(50)[:n]
        best_t, best_v = None, None
        for v, t in sorted(zip(vals.tolist(), ids.tolist()), key=lambda p: p[1]):   # ascending token id
            if math.isnan(v):
                continue
            if best_v is None or v > best_v:
                best_t, best_v = t, v
        if best_t is None:
            best_t = int(ids.min())
        assert O.argmax_token(vals, ids)[0] == best_t
    # float32 decision: values closer than float32 resolution tie, lowest id wins
    assert O.argmax_token(np.array([1.0, 1.0 + 1e-12]), np.array([7, 3]))[0] == 3
    assert O.argmax_token(np.array([1.0 + 1e-12, 1.0]), np.array([7, 3]))[0] == 3
    t, gap = O.argmax_token(np.array([0.5, 2.0, 1.25]))
    assert t == 1 and gap == 0.75


# ------------------------------------------------------------------ verification (Sec. 2.3)

def _common_prefix_len(a, b):
    return len(os.path.commonprefix([list(a), list(b)]))


def test_verify_accept_enumerated():
    V, K = 3, 3
    g = np.random.default_rng(10)
    for trial in range(30):
        vals = g.integers(0, 3, (1, K + 1, V)).astype(np.float32)     # small ints: exact bf16, many ties
        bits = I.f32_to_bf16_bits(vals)
        gold = np.argmax(vals[0], axis=-1)                            # numpy: first (= lowest id) maximum
        for drafts in itertools.product(range(V), repeat=K):
            a, bonus, gg = O.verify_accept(bits, np.array([drafts], dtype=np.int32))
            want = _common_prefix_len(drafts, gold[:K])
            assert a[0] == want and bonus[0] == gold[want] and np.array_equal(gg[0], gold)
            assert 1 <= a[0] + 1 <= K + 1


def test_verify_accept_k0_emits_exactly_one_token():
    # K = 0 is vanilla decoding: acceptance length tau = 1.00 (Table 1, baseline row)
    with open(os.path.join(GOLDEN, "paper_tau.txt")) as f:
        rows = [l.split() for l in f if l.strip() and not l.startswith("#")]
    base = [r for r in rows if r[0] == "baseline"][0]
    assert float(base[2]) == 1.00
    bits = I.verify_logits_natural(5, 1, 97, 3)
    a, bonus, g = O.verify_accept(bits, np.zeros((5, 0), dtype=np.int32))
    assert np.all(a == 0) and np.array_equal(bonus, g[:, 0])
    assert np.mean(a + 1) == float(base[2])
    # every tau the paper prints respects 1 <= tau <= K + 1, the range of accept_len + 1
    for name, K, tau in rows:
        assert 1.0 <= float(tau) <= int(K) + 1


def test_verify_accept_planted_cases():
    case = I.verify_case(64, 3, 2048, 77)
    a, bonus, g = O.verify_accept(case["logits"], case["drafts"])
    assert np.array_equal(a, case["length"])
    assert np.array_equal(bonus, case["winner"][np.arange(64), case["length"]])
    assert np.array_equal(g, case["winner"])
    assert len(set(case["length"].tolist())) == 4          # every accepted length 0..K occurs
    # all-matching drafts accept K
    a, bonus, _ = O.verify_accept(case["logits"], case["winner"][:, :3])
    assert np.all(a == 3) and np.array_equal(bonus, case["winner"][:, 3])


# ------------------------------------------------------------------ recursion (Sec. 2.1 / 2.3)

def _draft_case(seed, shape=SMALL, B=2, L=(5, 9), K=3, N=20):
    W = I.mtp_weights(shape, seed)
    kv = I.paged_kv(shape, list(L), K + 2, seed + 1)
    h = I.hidden_bf16(seed + 2, (B, shape.d))
    tok = I.token_ids(seed + 3, (B,), shape.vocab)
    ids = I.subset_uniform(shape.vocab, N, seed + 4)
    return shape, W, kv, h, tok, ids


def _copy_kv(kv):
    return {k: (v.copy() if isinstance(v, np.ndarray) else v) for k, v in kv.items()}


def test_draft_prefix_property_and_restart():
    shape, W, kv, h, tok, ids = _draft_case(61)
    r3 = O.draft(shape, W, h, tok, _copy_kv(kv), 3, ids)
    for k in (1, 2):
        rk = O.draft(shape, W, h, tok, _copy_kv(kv), k, ids)
        assert np.array_equal(rk["drafts"], r3["drafts"][:, :k])
        assert np.array_equal(rk["h_out"], r3["h_out"][:, :k])
    # step k > 1 is a fresh single step on (own hidden state, previous draft) one slot later
    kv1 = _copy_kv(kv)
    r1 = O.draft(shape, W, h, tok, kv1, 1, ids)
    for b in range(2):
        hb = O.mtp_forward(r1["h_out"][b, 0], int(r1["drafts"][b, 0]), int(kv["seq_lens"][b]) + 1,
                           W, kv1, b, shape)
        assert np.allclose(hb, r3["h_out"][b, 1], rtol=1e-13, atol=1e-13)
    assert set(r3["drafts"].ravel().tolist()) <= set(ids.tolist())


def test_draft_extend_rows_equal_sequential_single_row_calls():
    shape, W, kv, _, _, ids = _draft_case(71, B=1, L=(4,))
    h3 = I.hidden_bf16(72, (1, 3, shape.d))
    t3 = I.token_ids(73, (1, 3), shape.vocab)
    ext = O.draft(shape, W, h3, t3, _copy_kv(kv), 2, ids)
    kv2 = _copy_kv(kv)
    for m in range(3):
        r = O.draft(shape, W, h3[:, m], t3[:, m], kv2, 2 if m == 2 else 1, ids)
        kv2["seq_lens"][0] += 1
    assert np.array_equal(r["drafts"], ext["drafts"]) and np.array_equal(r["h_out"], ext["h_out"])


# ------------------------------------------------------------------ losslessness (Sec. 2.3, Sec. 3.1)

def _loop_case(seed, n_layers=2):
    shape = SMALL.with_layers(n_layers)
    Wt = I.target_weights(shape, seed)
    Wm = I.mtp_weights(shape, seed + 1, embed=Wt["embed"], lm_head=Wt["lm_head"])
    prompt = I.token_ids(seed + 2, (7,), shape.vocab)
    ids = I.subset_uniform(shape.vocab, 24, seed + 3)
    mk = lambda s0: [I.empty_paged_kv(shape, 1, 48, s0 + l) for l in range(n_layers)]
    return shape, Wt, Wm, prompt, ids, mk


@pytest.mark.parametrize("K", [1, 3])
def test_speculative_equals_greedy_with_mtp_drafts(K):
    shape, Wt, Wm, prompt, ids, mk = _loop_case(81)
    n_new = 14
    ref = O.greedy_decode(shape, Wt, prompt, n_new, mk(1))
    out, st = O.speculative_decode(shape, Wt, Wm, prompt, n_new, K, ids, mk(5),
                                   I.empty_paged_kv(shape, 1, 48, 9))
    assert out == ref
    assert all(0 <= a <= K for a in st["accepted"])


def test_speculative_equals_greedy_with_injected_drafts_of_every_accept_length():
    shape, Wt, Wm, prompt, ids, mk = _loop_case(91)
    n_new, K = 20, 3
    ref = O.greedy_decode(shape, Wt, prompt, n_new + K + 1, mk(1))
    plan = [3, 0, 2, 1, 3, 3, 0, 1, 2, 3, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0]
    state = {"emitted": 1}

    def inject(rnd, K_):
        # perfect drafts from the greedy run for the first plan[rnd] positions, then a wrong one
        e = state["emitted"]
        good = ref[e:e + K_]
        n_ok = plan[rnd]
        d = list(good[:n_ok]) + [(t + 1) % shape.vocab for t in good[n_ok:]]
        state["emitted"] = e + n_ok + 1
        return d

    out, st = O.speculative_decode(shape, Wt, Wm, prompt, n_new, K, ids, mk(5),
                                   I.empty_paged_kv(shape, 1, 64, 9), inject=inject)
    assert out == ref[:n_new]
    assert st["accepted"] == plan[:len(st["accepted"])]
    assert {0, 1, 2, 3} <= set(st["accepted"])


def test_speculative_with_all_wrong_drafts_is_plain_decoding():
    shape, Wt, Wm, prompt, ids, mk = _loop_case(95)
    ref = O.greedy_decode(shape, Wt, prompt, 8, mk(1))
    pos = {"i": 1}

    def inject(rnd, K_):
        e = pos["i"]
        pos["i"] += 1
        return [(ref[min(e, len(ref) - 1)] + 1) % shape.vocab] * K_

    out, st = O.speculative_decode(shape, Wt, Wm, prompt, 8, 2, ids, mk(5),
                                   I.empty_paged_kv(shape, 1, 48, 9), inject=inject)
    assert out == ref and set(st["accepted"]) == {0}


def test_tiny_config_draft_runs_and_is_deterministic():
    shape = I.TINY
    W = I.mtp_weights(shape, 1234)
    kv = I.paged_kv(shape, [64], 4, 1234)
    h = I.hidden_bf16(1234, (1, shape.d))
    tok = I.token_ids(1234, (1,), shape.vocab)
    ids = I.subset_uniform(shape.vocab, 1024, 1234)
    a = O.draft(shape, W, h, tok, _copy_kv(kv), 3, ids)
    b = O.draft(shape, W, h, tok, _copy_kv(kv), 3, ids)
    assert np.array_equal(a["drafts"], b["drafts"]) and a["drafts"].shape == (1, 3)
    assert np.all(np.abs(np.sqrt((a["h_out"] ** 2).mean(-1)) - 1.0) < 0.1)      # post-norm rms ~ gains ~ 1


def test_layer_grouped_target_forward_equals_the_row_by_row_one():
    """target_forward_block (a layer's projections as one matrix product over all rows) computes what target_forward
    computes row by row: hidden states, logits and both layers' caches, on a prompt that crosses pages and with rows
    appended to a non-empty cache."""
    shp = I.TINY.with_layers(3)
    Wt = I.target_weights(shp, 71)
    toks = I.token_ids(72, (1, 37), shp.vocab)
    a = [I.empty_paged_kv(shp, 1, 64, 80 + l) for l in range(3)]
    b = [{k: (v.copy() if isinstance(v, np.ndarray) else v) for k, v in kv.items()} for kv in a]
    for lo, hi in ((0, 29), (29, 37)):                      # a prefill, then more rows on top of it
        h1, l1 = O.target_forward(shp, Wt, toks[:, lo:hi], a)
        h2, l2 = O.target_forward_block(shp, Wt, toks[0, lo:hi], b, logit_rows=(0, hi - lo - 1))
        assert np.max(np.abs(h1[0] - h2)) <= 1e-12 * max(1.0, np.max(np.abs(h1)))
        for r, lg in l2.items():
            assert np.max(np.abs(l1[0, r] - lg)) <= 1e-12 * max(1.0, np.max(np.abs(lg)))
        for kv in a + b:
            kv["seq_lens"][0] += hi - lo
    for x, y in zip(a, b):
        assert np.array_equal(x["k_pages"], y["k_pages"]) and np.array_equal(x["v_pages"], y["v_pages"])
