"""Pins for the oracle's layer arithmetic: brute force, closed forms, library routines."""
import math

import numpy as np
import pytest
import torch

from oracle import tidar_oracle as O
from tidar_synth import CONFIGS, gen_model_weights, gen_token_ids, tensor_id


def _cfg(sh, beta=1.0):
    return O.OracleConfig(sh.n_layers, sh.d_model, sh.n_q_heads, sh.n_kv_heads, sh.head_dim, sh.d_ffn,
                          sh.vocab, sh.rope_theta, sh.rms_eps, sh.mask_token_id, beta)


# ---------------------------------------------------------------- attention
def _brute_row(q_row, K, V, allowed, hd):
    """One query row, python loops and math.exp only."""
    cols = [c for c in range(len(K)) if allowed[c]]
    scores = [sum(q_row[d] * K[c][d] for d in range(hd)) / math.sqrt(hd) for c in cols]
    mx = max(scores)
    e = [math.exp(s - mx) for s in scores]
    z = sum(e)
    return [sum(e[i] / z * V[c][d] for i, c in enumerate(cols)) for d in range(hd)]


def test_attention_matches_brute_force_on_decode_mask():
    rng = np.random.default_rng(0)
    n, k, Hq, Hkv, hd = 5, 3, 4, 2, 8
    T = O.n_slots(k)
    mask = O.build_decode_mask(n, k)
    q = rng.standard_normal((T, Hq, hd))
    kk = rng.standard_normal((n + T, Hkv, hd))
    vv = rng.standard_normal((n + T, Hkv, hd))
    out = O.masked_attention(q, kk, vv, mask)
    for r in range(T):
        for h in range(Hq):
            g = h // (Hq // Hkv)
            ref = _brute_row(q[r, h].tolist(), kk[:, g].tolist(), vv[:, g].tolist(), mask[r].tolist(), hd)
            np.testing.assert_allclose(out[r, h], ref, rtol=1e-12, atol=1e-13)


def test_attention_matches_torch_sdpa():
    rng = np.random.default_rng(1)
    n, k, Hq, Hkv, hd = 9, 4, 6, 2, 16
    T = O.n_slots(k)
    mask = O.build_decode_mask(n, k)
    q = rng.standard_normal((T, Hq, hd)); kk = rng.standard_normal((n + T, Hkv, hd)); vv = rng.standard_normal((n + T, Hkv, hd))
    out = O.masked_attention(q, kk, vv, mask)
    tq = torch.from_numpy(q).permute(1, 0, 2)[None]
    tk = torch.from_numpy(kk).permute(1, 0, 2)[None].repeat_interleave(Hq // Hkv, dim=1)
    tv = torch.from_numpy(vv).permute(1, 0, 2)[None].repeat_interleave(Hq // Hkv, dim=1)
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, attn_mask=torch.from_numpy(mask)[None, None])
    np.testing.assert_allclose(out, ref[0].permute(1, 0, 2).numpy(), rtol=1e-11, atol=1e-12)


def test_attention_zero_query_is_mean_of_visible_values():
    rng = np.random.default_rng(2)
    n, k = 4, 2
    T = O.n_slots(k)
    mask = O.build_decode_mask(n, k)
    vv = rng.standard_normal((n + T, 1, 4))
    out = O.masked_attention(np.zeros((T, 1, 4)), rng.standard_normal((n + T, 1, 4)), vv, mask)
    for r in range(T):
        np.testing.assert_allclose(out[r, 0], vv[mask[r], 0].mean(axis=0), rtol=1e-13)


def test_attention_sharp_query_picks_one_key():
    # one key aligned with a huge query: the output is that key's value (softmax limit)
    hd = 4
    kk = np.eye(4)[:, None, :]
    vv = np.arange(16, dtype=float).reshape(4, 1, 4)
    q = (1e4 * np.eye(4)[2])[None, None, :]
    out = O.masked_attention(q, kk, vv, np.ones((1, 4), dtype=bool))
    np.testing.assert_allclose(out[0, 0], vv[2, 0], atol=1e-9)
    # ... and a masked key is never picked
    m = np.ones((1, 4), dtype=bool); m[0, 2] = False
    out = O.masked_attention(q, kk, vv, m)
    np.testing.assert_allclose(out[0, 0], vv[[0, 1, 3], 0].mean(axis=0), atol=1e-9)


# ---------------------------------------------------------------- rope
def test_rope_position_zero_is_identity_and_norm_preserved():
    rng = np.random.default_rng(3)
    x = rng.standard_normal((5, 3, 8))
    np.testing.assert_array_equal(O.rope(x, np.zeros(5, dtype=np.int64), 1e4), x)
    y = O.rope(x, np.array([1, 7, 100, 4095, 32767]), 1e6)
    np.testing.assert_allclose(np.linalg.norm(y, axis=-1), np.linalg.norm(x, axis=-1), rtol=1e-12)


def test_rope_closed_form_pairs():
    # hd = 4: pair (0, 2) turns by pos * theta^0, pair (1, 3) by pos * theta^(-1/2)
    theta, p = 100.0, 3
    x = np.array([[[1.0, 2.0, 0.0, 0.0]]])
    y = O.rope(x, np.array([p]), theta)[0, 0]
    a0, a1 = p * 1.0, p * theta ** -0.5
    np.testing.assert_allclose(y, [math.cos(a0), 2 * math.cos(a1), math.sin(a0), 2 * math.sin(a1)], rtol=1e-14)


def test_rope_scores_depend_on_relative_position_only():
    rng = np.random.default_rng(4)
    q = rng.standard_normal((1, 1, 16)); kk = rng.standard_normal((1, 1, 16))
    def score(m, n):
        return float(np.sum(O.rope(q, np.array([m]), 1e4) * O.rope(kk, np.array([n]), 1e4)))
    assert abs(score(10, 3) - score(107, 100)) < 1e-12
    assert abs(score(10, 3) - score(11, 3)) > 1e-6


# ---------------------------------------------------------------- norm / ffn
def test_rmsnorm_properties_and_library():
    rng = np.random.default_rng(5)
    x = rng.standard_normal((7, 32)) * 3.0
    g = 1.0 + 0.1 * rng.standard_normal(32)
    y = O.rmsnorm(x, np.ones(32), 0.0)
    np.testing.assert_allclose(np.mean(y * y, axis=-1), 1.0, rtol=1e-13)
    np.testing.assert_allclose(O.rmsnorm(5.0 * x, g, 0.0), O.rmsnorm(x, g, 0.0), rtol=1e-13)
    ref = torch.nn.functional.rms_norm(torch.from_numpy(x), (32,), torch.from_numpy(g), eps=1e-6).numpy()
    np.testing.assert_allclose(O.rmsnorm(x, g, 1e-6), ref, rtol=1e-12)
    # eps matters for tiny inputs: x = 0 stays 0, |x| << sqrt(eps) scales by 1/sqrt(eps)
    np.testing.assert_allclose(O.rmsnorm(np.full((1, 4), 1e-9), np.ones(4), 1e-6), np.full((1, 4), 1e-9 / 1e-3), rtol=1e-6)


def test_swiglu_library_and_points():
    rng = np.random.default_rng(6)
    a, b = rng.standard_normal((3, 9)), rng.standard_normal((3, 9))
    ref = (torch.nn.functional.silu(torch.from_numpy(a)) * torch.from_numpy(b)).numpy()
    np.testing.assert_allclose(O.swiglu(a, b), ref, rtol=1e-13)
    assert O.swiglu(np.array([0.0]), np.array([7.0]))[0] == 0.0
    np.testing.assert_allclose(O.swiglu(np.array([50.0]), np.array([2.0])), [100.0], rtol=1e-12)   # silu(x) -> x


# ---------------------------------------------------------------- whole causal pass vs a library decoder
@pytest.mark.parametrize("tied", [True, False])
def test_causal_forward_matches_transformers_llama(tied):
    tf = pytest.importorskip("transformers")
    from dataclasses import replace
    sh = replace(CONFIGS["tiny"], tie_lm_head=tied)
    wt = gen_model_weights(sh)
    cfg = _cfg(sh)
    w = O.weights_to_f64(wt)
    ids = gen_token_ids(3, tensor_id("prompt"), 23, sh.vocab - 1).numpy().astype(np.int64)
    fo = O.causal_forward(cfg, w, ids)

    c = tf.LlamaConfig(vocab_size=sh.vocab, hidden_size=sh.d_model, intermediate_size=sh.d_ffn,
                       num_hidden_layers=sh.n_layers, num_attention_heads=sh.n_q_heads,
                       num_key_value_heads=sh.n_kv_heads, head_dim=sh.head_dim, rms_norm_eps=sh.rms_eps,
                       rope_theta=sh.rope_theta, tie_word_embeddings=tied, attention_bias=False,
                       mlp_bias=False, max_position_embeddings=512, attn_implementation="eager")
    m = tf.LlamaForCausalLM(c).double().eval()
    sd = {"model.embed_tokens.weight": wt["embed"], "model.norm.weight": wt["final_norm"],
          "lm_head.weight": wt["lm_head"]}
    names = {"wq": "self_attn.q_proj", "wk": "self_attn.k_proj", "wv": "self_attn.v_proj", "wo": "self_attn.o_proj",
             "w_gate": "mlp.gate_proj", "w_up": "mlp.up_proj", "w_down": "mlp.down_proj",
             "attn_norm": "input_layernorm", "ffn_norm": "post_attention_layernorm"}
    for l, L in enumerate(wt["layers"]):
        for k_, v_ in names.items():
            sd[f"model.layers.{l}.{v_}.weight"] = L[k_]
    missing = m.load_state_dict({k_: v_.double() for k_, v_ in sd.items()}, strict=False)
    assert not [x for x in missing.missing_keys if "rotary" not in x]
    with torch.no_grad():
        ref = m(torch.from_numpy(ids)[None]).logits[0].numpy()
    # the library builds its rotary tables in float32, so agreement stops near 1e-7;
    # any structural mistake (pairing, head mapping, norm placement) is >= 1e-2
    np.testing.assert_allclose(fo.logits, ref, rtol=0, atol=2e-6)


# ---- optional bf16 storage of activations (OracleConfig.act_dtype) -------------------------------
def test_round_bf16_is_round_to_nearest_even_bfloat16():
    """Pinned against torch's float32 -> bfloat16 conversion and against hand-worked bit patterns."""
    rng = np.random.default_rng(3)
    x = np.concatenate([rng.standard_normal(4096) * 10.0 ** rng.integers(-6, 6, 4096), [0.0, -0.0, 1.0, -1.0, 3.0e38, 1e-40]])
    want = torch.tensor(x, dtype=torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    np.testing.assert_array_equal(O.round_bf16(x), want)
    # 1 + 2^-8 lies exactly between 1 and 1 + 2^-7: ties go to the even mantissa (1.0);
    # 1 + 3 * 2^-8 lies between 1 + 2^-7 (odd) and 1 + 2^-6 (even): up
    np.testing.assert_array_equal(O.round_bf16(np.array([1 + 2.0 ** -8, 1 + 3 * 2.0 ** -8, 1 + 2.0 ** -8 + 2.0 ** -20])),
                                  [1.0, 1 + 2.0 ** -6, 1 + 2.0 ** -7])


def test_bf16_storage_mode_rounds_only_what_is_stored():
    """With act_dtype = "bf16" the K/V a pass returns are exact bf16 values, the results move by the
    size of bf16 rounding noise and no more, and the default mode is untouched."""
    from dataclasses import replace
    from tests.helpers import make_model, oracle_cfg, prompt_ids
    sh, wt = make_model("tiny")
    cfg = oracle_cfg(sh)
    w = O.weights_to_f64(wt)
    ids = prompt_ids(sh, 24)
    a = O.causal_forward(cfg, w, ids)
    b = O.causal_forward(replace(cfg, act_dtype="bf16"), w, ids)
    c = O.causal_forward(replace(cfg, act_dtype="f64"), w, ids)
    np.testing.assert_array_equal(a.logits, c.logits)
    for l in range(cfg.n_layers):
        np.testing.assert_array_equal(b.k_new[l], O.round_bf16(b.k_new[l]))
        np.testing.assert_array_equal(b.v_new[l], O.round_bf16(b.v_new[l]))
        assert not np.array_equal(a.k_new[l], O.round_bf16(a.k_new[l]))
    d = np.abs(a.logits - b.logits).max()
    assert 1e-5 < d < 3e-2, d
    np.testing.assert_array_equal(a.hidden[0], b.hidden[0])        # the embedding rows are not an activation store


# ---- optional projection biases and per-head Q/K norm: pinned against library decoders that have them
def _hf_state(wt, extra):
    sd = {"model.embed_tokens.weight": wt["embed"], "model.norm.weight": wt["final_norm"], "lm_head.weight": wt["lm_head"]}
    names = {"wq": "self_attn.q_proj.weight", "wk": "self_attn.k_proj.weight", "wv": "self_attn.v_proj.weight", "wo": "self_attn.o_proj.weight",
             "w_gate": "mlp.gate_proj.weight", "w_up": "mlp.up_proj.weight", "w_down": "mlp.down_proj.weight",
             "attn_norm": "input_layernorm.weight", "ffn_norm": "post_attention_layernorm.weight", **extra}
    for l, L in enumerate(wt["layers"]):
        for k_, v_ in names.items():
            sd[f"model.layers.{l}.{v_}"] = L[k_]
    return {k_: v_.double() for k_, v_ in sd.items()}


@pytest.mark.parametrize("family", ["qwen2_bias", "qwen3_qk_norm"])
def test_causal_forward_with_bias_or_qk_norm_matches_transformers(family):
    tf = pytest.importorskip("transformers")
    from dataclasses import replace
    sh = replace(CONFIGS["tiny"], tie_lm_head=False, qkv_bias=family == "qwen2_bias", qk_norm=family == "qwen3_qk_norm")
    wt = gen_model_weights(sh)
    cfg = _cfg(sh)
    w = O.weights_to_f64(wt)
    ids = gen_token_ids(4, tensor_id("prompt"), 19, sh.vocab - 1).numpy().astype(np.int64)
    fo = O.causal_forward(cfg, w, ids)
    common = dict(vocab_size=sh.vocab, hidden_size=sh.d_model, intermediate_size=sh.d_ffn, num_hidden_layers=sh.n_layers,
                  num_attention_heads=sh.n_q_heads, num_key_value_heads=sh.n_kv_heads, rms_norm_eps=sh.rms_eps, rope_theta=sh.rope_theta,
                  tie_word_embeddings=False, max_position_embeddings=512, attn_implementation="eager", use_sliding_window=False)
    if family == "qwen2_bias":
        m = tf.Qwen2ForCausalLM(tf.Qwen2Config(**common)).double().eval()
        extra = {"bq": "self_attn.q_proj.bias", "bk": "self_attn.k_proj.bias", "bv": "self_attn.v_proj.bias"}
    else:
        m = tf.Qwen3ForCausalLM(tf.Qwen3Config(head_dim=sh.head_dim, attention_bias=False, **common)).double().eval()
        extra = {"q_norm": "self_attn.q_norm.weight", "k_norm": "self_attn.k_norm.weight"}
    missing = m.load_state_dict(_hf_state(wt, extra), strict=False)
    assert not [x for x in missing.missing_keys if "rotary" not in x] and not missing.unexpected_keys
    with torch.no_grad():
        ref = m(torch.from_numpy(ids)[None]).logits[0].numpy()
    np.testing.assert_allclose(fo.logits, ref, rtol=0, atol=2e-6)
    # and the option does something: the same weights without it give different logits
    plain = {**w, "layers": [{k_: v_ for k_, v_ in L.items() if k_ not in extra} for L in w["layers"]]}
    assert np.abs(O.causal_forward(cfg, plain, ids).logits - fo.logits).max() > 1e-3
