"""Pins for the oracle's transformer forward: things fixed by mathematics or by
an independent library, chosen so that a dropped term, wrong sign, wrong index
or transposed operand fails at least one of them."""
import dataclasses
import math

import numpy as np
import pytest
import torch

import oracle
from synth import MODEL_SHAPES, make_weights

TINY = MODEL_SHAPES["tiny"]


def rel(a, b):
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


# ---------------------------------------------------------------- elementwise pins
def test_rmsnorm_hand_values_and_scale_invariance():
    a = oracle.rmsnorm(np.array([[3.0, 4.0]]), np.array([1.0, 2.0]), 0.0)
    # mean square 12.5 -> rms 3.5355339...
    assert np.allclose(a, [[3 / math.sqrt(12.5), 8 / math.sqrt(12.5)]], rtol=1e-15)
    rng = np.random.default_rng(0)
    h, g = rng.standard_normal((5, 64)), rng.standard_normal(64)
    assert rel(oracle.rmsnorm(7.5 * h, g, 1e-12), oracle.rmsnorm(h, g, 1e-12)) < 1e-10
    # eps matters when the row is tiny
    z = oracle.rmsnorm(np.full((1, 4), 1e-4), np.ones(4), 1e-6)
    assert np.allclose(z, 1e-4 / math.sqrt(1e-8 + 1e-6))


def test_silu_hand_values():
    z = oracle.silu(np.array([0.0, 1.0, -1.0]))
    assert np.allclose(z, [0.0, 0.7310585786300049, -0.2689414213699951], atol=1e-15)


def test_rope_hand_values():
    # hd = 4, base 10000: theta = p * [1, 0.01]; pairs are (0,2) and (1,3)
    x = np.array([[[1.0, 2.0, 3.0, 4.0]]])
    y = oracle.apply_rope(x, np.array([1]), 10000.0)[0, 0]
    c1, s1, c2, s2 = math.cos(1.0), math.sin(1.0), math.cos(0.01), math.sin(0.01)
    assert np.allclose(y, [1 * c1 - 3 * s1, 2 * c2 - 4 * s2, 3 * c1 + 1 * s1, 4 * c2 + 2 * s2], rtol=1e-14)
    # hd = 64, pair 1 at position 3: theta = 3 * 10000^(-2/64)
    cos, sin = oracle.rope_cos_sin(np.array([3]), 64, 10000.0)
    assert math.isclose(cos[0, 1], math.cos(3 * 10000 ** (-1 / 32)), rel_tol=1e-14)


def test_rope_identity_norm_and_relative_position():
    rng = np.random.default_rng(1)
    q = rng.standard_normal((1, 3, 64))
    k = rng.standard_normal((1, 3, 64))
    assert np.array_equal(oracle.apply_rope(q, np.array([0]), 10000.0), q)
    r = oracle.apply_rope(np.repeat(q, 5, 0), np.arange(5) * 37, 10000.0)
    assert np.allclose(np.linalg.norm(r, axis=-1), np.linalg.norm(q, axis=-1), rtol=1e-12)

    def dot(m, n):
        a = oracle.apply_rope(q, np.array([m]), 10000.0)
        b = oracle.apply_rope(k, np.array([n]), 10000.0)
        return (a * b).sum(-1)
    assert np.allclose(dot(9, 4), dot(105, 100), rtol=1e-9, atol=1e-11)
    assert not np.allclose(dot(9, 4), dot(4, 9), rtol=1e-3)  # direction of rotation matters


# ---------------------------------------------------------------- attention pins
def test_attention_equals_bruteforce():
    rng = np.random.default_rng(2)
    n, Hq, Hkv, hd = 7, 4, 2, 8
    q, k, v = (rng.standard_normal((n, H, hd)) for H in (Hq, Hkv, Hkv))
    fast = oracle.causal_attention(q, k, v)
    slow = np.array(oracle.attention_bruteforce(q.tolist(), k.tolist(), v.tolist()))
    assert rel(fast, slow) < 1e-13


def test_attention_closed_forms():
    rng = np.random.default_rng(3)
    n, Hq, Hkv, hd = 9, 4, 2, 16
    q, k, v = (rng.standard_normal((n, H, hd)) for H in (Hq, Hkv, Hkv))
    # single token: output is its own value row
    o1 = oracle.causal_attention(q[:1], k[:1], v[:1])
    assert np.allclose(o1[0, 0], v[0, 0]) and np.allclose(o1[0, 3], v[0, 1])
    # zero queries: uniform weights -> running mean of the values
    o0 = oracle.causal_attention(np.zeros_like(q), k, v)
    run = np.cumsum(v, axis=0) / np.arange(1, n + 1)[:, None, None]
    for hq in range(Hq):
        assert np.allclose(o0[:, hq], run[:, hq // 2], rtol=1e-12)
    # grouped-query == multi-head with the KV heads replicated
    mha = oracle.causal_attention(q, np.repeat(k, 2, axis=1), np.repeat(v, 2, axis=1))
    assert np.allclose(oracle.causal_attention(q, k, v), mha, rtol=1e-13)
    # first row never sees later keys
    k2, v2 = k.copy(), v.copy()
    k2[1:] += 5.0
    v2[1:] -= 3.0
    assert np.allclose(oracle.causal_attention(q, k2, v2)[0], oracle.causal_attention(q, k, v)[0])


# ---------------------------------------------------------------- whole-forward pins
@pytest.fixture(scope="module")
def tiny_w():
    return make_weights(TINY, seed=1, dtype=torch.float32)


def test_prefill_equals_incremental_decode(tiny_w):
    toks = np.random.default_rng(4).integers(0, TINY.vocab, 41)
    K1, V1 = oracle.prefill_kv(tiny_w, TINY, toks)
    K2, V2 = oracle.decode_incremental_kv(tiny_w, TINY, toks)
    assert rel(K1, K2) < 1e-12 and rel(V1, V2) < 1e-12


def test_three_layer_prefill_equals_incremental_decode():
    shape = dataclasses.replace(TINY, n_layers=3)
    w = make_weights(shape, seed=7, dtype=torch.float32)
    toks = np.random.default_rng(5).integers(0, shape.vocab, 19)
    K1, V1 = oracle.prefill_kv(w, shape, toks)
    K2, V2 = oracle.decode_incremental_kv(w, shape, toks)
    assert rel(K1, K2) < 1e-12 and rel(V1, V2) < 1e-12


def test_causality_and_layer_prefix(tiny_w):
    rng = np.random.default_rng(6)
    toks = rng.integers(0, TINY.vocab, 50)
    K, V = oracle.prefill_kv(tiny_w, TINY, toks)
    other = toks.copy()
    other[30:] = rng.integers(0, TINY.vocab, 20)
    K2, V2 = oracle.prefill_kv(tiny_w, TINY, other)
    assert rel(K2[:, :30], K[:, :30]) < 1e-13 and rel(V2[:, :30], V[:, :30]) < 1e-13
    assert rel(K2[1, 30:], K[1, 30:]) > 1e-3
    # a truncated prefix gives the same rows; fewer layers give the same leading layers
    K3, V3 = oracle.prefill_kv(tiny_w, TINY, toks[:23])
    assert rel(K3, K[:, :23]) < 1e-13 and rel(V3, V[:, :23]) < 1e-13
    K4, V4 = oracle.prefill_kv(tiny_w, TINY, toks, n_layers=1)
    assert np.array_equal(K4[0], K[0]) and np.array_equal(V4[0], V[0])


def test_layer0_dependencies(tiny_w):
    toks = np.array([5, 9, 5, 5, 9])
    K, V = oracle.prefill_kv(tiny_w, TINY, toks)
    # layer-0 V depends on the token id only; layer-0 K on (id, position)
    assert np.array_equal(V[0, 0], V[0, 2]) and np.array_equal(V[0, 1], V[0, 4])
    assert not np.allclose(K[0, 0], K[0, 2])
    assert not np.allclose(V[1, 0], V[1, 2])  # deeper layers see context


def test_zeroed_output_projections_closed_form():
    shape = dataclasses.replace(TINY, n_layers=3)
    w = make_weights(shape, seed=3, dtype=torch.float32)
    for l in range(3):
        w["wo"][l].zero_()
        w["wd"][l].zero_()
    toks = np.random.default_rng(8).integers(0, shape.vocab, 12)
    K, V = oracle.prefill_kv(w, shape, toks)
    E = w["embed"].double().numpy()[toks]
    for l in range(3):
        g = w["ln1"][l].double().numpy()
        a = E / np.sqrt((E * E).mean(-1, keepdims=True) + shape.rms_eps) * g
        v = (a @ w["wv"][l].double().numpy().T).reshape(12, shape.n_kv_heads, shape.head_dim)
        k = (a @ w["wk"][l].double().numpy().T).reshape(12, shape.n_kv_heads, shape.head_dim)
        assert rel(V[l], v) < 1e-13
        assert rel(K[l, 0], k[0]) < 1e-13          # position 0: no rotation
        assert np.allclose(np.linalg.norm(K[l], axis=-1), np.linalg.norm(k, axis=-1), rtol=1e-12)


def test_library_model_pin():
    """The special case that reduces to a library routine: transformers' Llama
    decoder (fp64, eager attention) built with the same weights returns the
    post-RoPE K and raw V of every layer in its cache."""
    transformers = pytest.importorskip("transformers")
    shape = dataclasses.replace(TINY, n_layers=3)
    w = make_weights(shape, seed=11, dtype=torch.float32)
    cfg = transformers.LlamaConfig(
        vocab_size=shape.vocab, hidden_size=shape.d_model, intermediate_size=shape.ffn,
        num_hidden_layers=shape.n_layers, num_attention_heads=shape.n_q_heads,
        num_key_value_heads=shape.n_kv_heads, head_dim=shape.head_dim, rms_norm_eps=shape.rms_eps,
        rope_theta=shape.rope_base, attention_bias=False, mlp_bias=False,
        max_position_embeddings=512, attn_implementation="eager")
    m = transformers.LlamaModel(cfg).to(torch.float64).eval()
    sd = {"embed_tokens.weight": w["embed"], "norm.weight": torch.ones(shape.d_model)}
    names = {"ln1": "input_layernorm", "ln2": "post_attention_layernorm", "wq": "self_attn.q_proj",
             "wk": "self_attn.k_proj", "wv": "self_attn.v_proj", "wo": "self_attn.o_proj",
             "wg": "mlp.gate_proj", "wu": "mlp.up_proj", "wd": "mlp.down_proj"}
    for l in range(shape.n_layers):
        for s, nm in names.items():
            sd[f"layers.{l}.{nm}.weight"] = w[s][l]
    m.load_state_dict({k: v.double() for k, v in sd.items()}, strict=True)
    toks = np.random.default_rng(12).integers(0, shape.vocab, 77)
    with torch.no_grad():
        out = m(input_ids=torch.as_tensor(toks)[None], use_cache=True)
    K, V = oracle.prefill_kv(w, shape, toks)
    for l in range(shape.n_layers):
        lk = out.past_key_values.layers[l].keys[0].permute(1, 0, 2).numpy()
        lv = out.past_key_values.layers[l].values[0].permute(1, 0, 2).numpy()
        # the library evaluates its rotary angles in fp32: agreement to ~1e-6
        assert rel(K[l], lk) < 2e-5, (l, rel(K[l], lk))
        assert rel(V[l], lv) < 2e-5, (l, rel(V[l], lv))


def test_bf16_activation_reading(tiny_w):
    """The bf16-storage reading of the forward: its rounding is the arena's
    rounding, it changes nothing when there is nothing to round, and it stays
    within a few bf16 roundings of the definition."""
    x = np.random.default_rng(9).standard_normal(5000) * 7
    assert np.array_equal(oracle.round_bf16(x), oracle.bf16_bits_to_f64(oracle.to_bf16_bits(x)))
    lib = torch.from_numpy(x).float().to(torch.bfloat16).double().numpy()
    assert np.array_equal(oracle.round_bf16(x), lib)
    toks = np.random.default_rng(10).integers(0, TINY.vocab, 33)
    K, V = oracle.prefill_kv(tiny_w, TINY, toks)
    Kb, Vb = oracle.prefill_kv(tiny_w, TINY, toks, act_bf16=True)
    # layer 0: only the norm output was rounded on the way to K/V -> about one bf16 rounding (2^-9 / sqrt 3)
    assert 3e-4 < rel(Kb[0], K[0]) < 3e-3 and 3e-4 < rel(Vb[0], V[0]) < 3e-3
    assert rel(Kb[1], K[1]) < 1e-2
    # rounding the attention weights of a single-key row changes nothing: exp(0) = 1 is exact
    q, k, v = (np.random.default_rng(11).standard_normal((1, H, 8)) for H in (4, 2, 2))
    assert np.array_equal(oracle.causal_attention(q, k, v, round_p=oracle.round_bf16), oracle.causal_attention(q, k, v))


def test_resume_logits_library_pin():
    """Next-token logits against transformers' LlamaForCausalLM (fp64) with the same weights."""
    transformers = pytest.importorskip("transformers")
    shape = dataclasses.replace(TINY, n_layers=2)
    w = make_weights(shape, seed=13, dtype=torch.float32)
    g = torch.Generator().manual_seed(5)
    final_gain = 1.0 + 0.02 * torch.randn(shape.d_model, generator=g)
    lm_head = 0.02 * torch.randn(shape.vocab, shape.d_model, generator=g)
    cfg = transformers.LlamaConfig(
        vocab_size=shape.vocab, hidden_size=shape.d_model, intermediate_size=shape.ffn,
        num_hidden_layers=shape.n_layers, num_attention_heads=shape.n_q_heads,
        num_key_value_heads=shape.n_kv_heads, head_dim=shape.head_dim, rms_norm_eps=shape.rms_eps,
        rope_theta=shape.rope_base, attention_bias=False, mlp_bias=False,
        max_position_embeddings=512, attn_implementation="eager", tie_word_embeddings=False)
    m = transformers.LlamaForCausalLM(cfg).to(torch.float64).eval()
    sd = {"model.embed_tokens.weight": w["embed"], "model.norm.weight": final_gain, "lm_head.weight": lm_head}
    names = {"ln1": "input_layernorm", "ln2": "post_attention_layernorm", "wq": "self_attn.q_proj",
             "wk": "self_attn.k_proj", "wv": "self_attn.v_proj", "wo": "self_attn.o_proj",
             "wg": "mlp.gate_proj", "wu": "mlp.up_proj", "wd": "mlp.down_proj"}
    for l in range(shape.n_layers):
        for s_, nm in names.items():
            sd[f"model.layers.{l}.{nm}.weight"] = w[s_][l]
    m.load_state_dict({k: v.double() for k, v in sd.items()}, strict=True)
    toks = np.random.default_rng(14).integers(0, shape.vocab, 45)
    with torch.no_grad():
        want = m(input_ids=torch.as_tensor(toks)[None]).logits[0, -1].numpy()
    got = oracle.resume_logits(w, shape, toks, final_gain, lm_head)
    assert got.shape == (shape.vocab,)
    assert rel(got, want) < 2e-5
    # a one-token prefix: attention is the identity on v, closed form available through prefill pieces
    one = oracle.resume_logits(w, shape, toks[:1], final_gain, lm_head)
    assert np.isfinite(one).all() and rel(one, got) > 1e-3


# ---------------------------------------------------------------- projection variants
def _variant_library_kv(family, shape, w, toks):
    transformers = pytest.importorskip("transformers")
    common = dict(vocab_size=shape.vocab, hidden_size=shape.d_model, intermediate_size=shape.ffn,
                  num_hidden_layers=shape.n_layers, num_attention_heads=shape.n_q_heads,
                  num_key_value_heads=shape.n_kv_heads, rms_norm_eps=shape.rms_eps, rope_theta=shape.rope_base,
                  max_position_embeddings=512, attn_implementation="eager")
    if family == "qwen2":
        m = transformers.Qwen2Model(transformers.Qwen2Config(use_sliding_window=False, **common))
    else:
        m = transformers.Qwen3Model(transformers.Qwen3Config(
            head_dim=shape.head_dim, attention_bias="bq" in w, use_sliding_window=False, **common))
    m = m.to(torch.float64).eval()
    sd = {"embed_tokens.weight": w["embed"], "norm.weight": torch.ones(shape.d_model)}
    names = {"ln1": "input_layernorm.weight", "ln2": "post_attention_layernorm.weight",
             "wq": "self_attn.q_proj.weight", "wk": "self_attn.k_proj.weight", "wv": "self_attn.v_proj.weight",
             "wo": "self_attn.o_proj.weight", "wg": "mlp.gate_proj.weight", "wu": "mlp.up_proj.weight",
             "wd": "mlp.down_proj.weight", "bq": "self_attn.q_proj.bias", "bk": "self_attn.k_proj.bias",
             "bv": "self_attn.v_proj.bias", "qn": "self_attn.q_norm.weight", "kn": "self_attn.k_norm.weight"}
    for l in range(shape.n_layers):
        for s, nm in names.items():
            if s in w:
                sd[f"layers.{l}.{nm}"] = w[s][l]
        if family == "qwen3" and "bq" in w:   # this family's bias switch also gives the output projection one
            sd[f"layers.{l}.self_attn.o_proj.bias"] = torch.zeros(shape.d_model)
    m.load_state_dict({k: v.double() for k, v in sd.items()}, strict=True)
    with torch.no_grad():
        out = m(input_ids=torch.as_tensor(toks)[None], use_cache=True)
    lk = [out.past_key_values.layers[l].keys[0].permute(1, 0, 2).numpy() for l in range(shape.n_layers)]
    lv = [out.past_key_values.layers[l].values[0].permute(1, 0, 2).numpy() for l in range(shape.n_layers)]
    return lk, lv


@pytest.mark.parametrize("family,bias,norm", [("qwen2", True, False), ("qwen3", False, True), ("qwen3", True, True)])
def test_variant_library_pins(family, bias, norm):
    """Library decoders of the two model families (q/k/v biases; per-head q/k
    RMSNorm before RoPE) with the same weights hold the same K/V in their cache."""
    shape = dataclasses.replace(TINY, n_layers=3)
    w = make_weights(shape, seed=21, dtype=torch.float32, qkv_bias=bias, qk_norm=norm)
    assert ("bq" in w) == bias and ("qn" in w) == norm
    toks = np.random.default_rng(22).integers(0, shape.vocab, 53)
    lk, lv = _variant_library_kv(family, shape, w, toks)
    K, V = oracle.prefill_kv(w, shape, toks)
    plain = {k: v for k, v in w.items() if k not in ("bq", "bk", "bv", "qn", "kn")}
    K0, _ = oracle.prefill_kv(plain, shape, toks)
    for l in range(shape.n_layers):
        assert rel(K[l], lk[l]) < 2e-5, (l, rel(K[l], lk[l]))
        assert rel(V[l], lv[l]) < 2e-5, (l, rel(V[l], lv[l]))
    assert rel(K[0], K0[0]) > 1e-2          # the variant terms are not a no-op
    # and the token-at-a-time decode agrees with the one-shot prefill
    K2, V2 = oracle.decode_incremental_kv(w, shape, toks[:17])
    assert rel(K[:, :17], K2) < 1e-12 and rel(V[:, :17], V2) < 1e-12


def test_variant_invariants():
    """What mathematics fixes about the two variant terms at layer 0: the V bias
    is added once and unrotated; the K bias is rotated with the row; with QK-norm
    the K rows no longer depend on the scale of wk, and each rotate-half pair keeps
    the squared length gain and normalisation give it (so the gain acts before RoPE)."""
    shape = dataclasses.replace(TINY, n_layers=1)
    toks = np.random.default_rng(23).integers(0, shape.vocab, 29)
    wb = make_weights(shape, seed=24, dtype=torch.float32, qkv_bias=True)
    plain = {k: v for k, v in wb.items() if k not in ("bq", "bk", "bv")}
    K, V = oracle.prefill_kv(wb, shape, toks)
    K0, V0 = oracle.prefill_kv(plain, shape, toks)
    bk = wb["bk"][0].double().numpy().reshape(shape.n_kv_heads, shape.head_dim)
    bv = wb["bv"][0].double().numpy().reshape(shape.n_kv_heads, shape.head_dim)
    assert np.allclose(V[0] - V0[0], bv[None], atol=1e-13)
    dK = K[0] - K0[0]
    assert np.allclose(dK[0], bk, atol=1e-13)                       # position 0: no rotation
    half = shape.head_dim // 2
    pair = lambda x: x[..., :half] ** 2 + x[..., half:] ** 2
    assert np.allclose(pair(dK), pair(bk)[None], rtol=1e-10)         # a rotation of the bias at every position
    assert not np.allclose(dK[5], bk, atol=1e-3)

    wn = make_weights(shape, seed=25, dtype=torch.float32, qk_norm=True)
    Kn, _ = oracle.prefill_kv(wn, shape, toks)
    scaled = dict(wn)
    scaled["wk"] = [wn["wk"][0] * 3.0]
    Ks, _ = oracle.prefill_kv(scaled, shape, toks)
    assert rel(Ks, Kn) < 1e-4                                        # only eps sees the scale
    g = wn["kn"][0].double().numpy()
    a = oracle.rmsnorm(wn["embed"].double().numpy()[toks], wn["ln1"][0].double().numpy(), shape.rms_eps)
    x = (a @ wn["wk"][0].double().numpy().T).reshape(len(toks), shape.n_kv_heads, shape.head_dim)
    xhat = x / np.sqrt((x * x).mean(-1, keepdims=True) + shape.rms_eps)
    assert np.allclose(pair(Kn[0]), pair(xhat * g), rtol=1e-10)
    assert not np.allclose(pair(Kn[0]), pair(xhat) * pair(g[None, None]) / 2, rtol=1e-3)


def test_sampled_rows_equal_the_full_prefill():
    """prefill_kv_rows (what the long-prefix GPU tests compare against) restates rows of
    prefill_kv, which the library pins above hold in place; with and without the variant terms."""
    for bias, norm in ((False, False), (True, True)):
        shape = dataclasses.replace(TINY, n_layers=2)
        w = make_weights(shape, seed=31, dtype=torch.float32, qkv_bias=bias, qk_norm=norm)
        toks = np.random.default_rng(32).integers(0, shape.vocab, 97)
        rows = [0, 1, 15, 16, 63, 96]
        K, V = oracle.prefill_kv(w, shape, toks, n_layers=2)
        K0, V0, K1, V1 = oracle.prefill_kv_rows(w, shape, toks, rows)
        assert rel(K0, K[0]) < 1e-13 and rel(V0, V[0]) < 1e-13
        assert rel(K1, K[1][rows]) < 1e-12 and rel(V1, V[1][rows]) < 1e-12
        assert rel(K1, K[1][[r + 1 for r in rows[:-1]] + [0]]) > 1e-2      # the rows are not interchangeable
        # the bf16 storage reading, row by row, is the full prefill's
        Kf, Vf = oracle.prefill_kv(w, shape, toks, n_layers=2, act_bf16=True)
        K0f, V0f, K1f, V1f = oracle.prefill_kv_rows(w, shape, toks, rows, act_bf16=True)
        assert rel(K0f, Kf[0]) < 1e-13 and rel(V0f, Vf[0]) < 1e-13
        assert rel(K1f, Kf[1][rows]) < 1e-12 and rel(V1f, Vf[1][rows]) < 1e-12
        assert 1e-4 < rel(K1f, K1) < 3e-2                                  # and it does differ from the definition
