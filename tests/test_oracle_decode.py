"""Pins for the oracle's decode procedure: the invariants the paper's method implies."""
import itertools
from dataclasses import replace

import numpy as np
import pytest

from oracle import tidar_oracle as O
from tidar_synth import CONFIGS, gen_model_weights, gen_token_ids, tensor_id


def _cfg(sh, beta=1.0):
    return O.OracleConfig(sh.n_layers, sh.d_model, sh.n_q_heads, sh.n_kv_heads, sh.head_dim, sh.d_ffn,
                          sh.vocab, sh.rope_theta, sh.rms_eps, sh.mask_token_id, beta)


@pytest.fixture(scope="module", params=["tied", "untied"])
def model(request):
    # the tied tiny model repeats one token under random weights; the untied twin
    # wanders, so both degenerate and non-degenerate sequences are covered
    sh = replace(CONFIGS["tiny"], tie_lm_head=(request.param == "tied"))
    w = O.weights_to_f64(gen_model_weights(sh))
    prompt = gen_token_ids(sh.seed, tensor_id("prompt"), sh.prompt_len, sh.vocab - 1).numpy().astype(np.int64)
    return sh, _cfg(sh), w, prompt


N_NEW = 24


@pytest.fixture(scope="module")
def ar_tokens(model):
    sh, cfg, w, prompt = model
    return O.ar_generate(cfg, w, prompt, N_NEW + 2 * sh.k)


# ---------------------------------------------------------------- acceptance rule
def _accept_brute(block, targets):
    k = len(block)
    best = 0
    for m in range(k):
        if all(block[i] == targets[i - 1] for i in range(1, m + 1)):
            best = max(best, m)
    return best + 1


@pytest.mark.parametrize("k", [1, 2, 4, 8])
def test_accept_length_exhaustive(k):
    targets = list(range(100, 100 + k))
    for pattern in itertools.product([True, False], repeat=k - 1):
        block = [7] + [targets[i] if ok else -1 for i, ok in enumerate(pattern)]
        L = O.accept_length(block, targets)
        assert L == _accept_brute(block, targets)
        assert 1 <= L <= k
        first_bad = next((i for i, ok in enumerate(pattern) if not ok), k - 1)
        assert L == first_bad + 1


def test_accept_forced_and_select():
    block = [5, 6, 7, 8]
    targets = [6, 9, 9, 9]
    assert O.accept_length(block, targets) == 2
    assert O.accept_length(block, targets, forced=4) == 4
    d = np.arange(16).reshape(4, 4) + 100
    np.testing.assert_array_equal(O.select_next(2, targets, d), [9, 105, 106, 107])


# ---------------------------------------------------------------- greedy TiDAR == greedy AR
def test_tidar_equals_ar_natural_drafts(model, ar_tokens):
    sh, cfg, w, prompt = model
    out, Ls, _ = O.generate(cfg, w, prompt, sh.k, N_NEW)
    assert out == ar_tokens[:N_NEW]
    assert all(1 <= L <= sh.k for L in Ls)


def test_tidar_equals_ar_garbage_drafts(model, ar_tokens):
    sh, cfg, w, prompt = model

    def hook(st):                      # drafts that can never match
        st.block[1:] = cfg.mask_token_id

    out, Ls, _ = O.generate(cfg, w, prompt, sh.k, N_NEW, draft_hook=hook)
    assert out == ar_tokens[:N_NEW]
    assert set(Ls) == {1}


def test_tidar_equals_ar_perfect_and_partial_drafts(model, ar_tokens):
    sh, cfg, w, prompt = model
    k = sh.k
    n0 = len(prompt)

    def perfect(st):
        e = st.n - n0                  # tokens emitted before block[0]
        st.block[1:] = ar_tokens[e + 1:e + k]

    out, Ls, _ = O.generate(cfg, w, prompt, k, N_NEW, draft_hook=perfect)
    assert out == ar_tokens[:N_NEW]
    assert set(Ls) == {k}

    def two_right(st):
        e = st.n - n0
        st.block[1:] = ar_tokens[e + 1:e + k]
        st.block[3] = (st.block[3] + 1) % (sh.vocab - 1)

    out, Ls, _ = O.generate(cfg, w, prompt, k, N_NEW, draft_hook=two_right)
    assert out == ar_tokens[:N_NEW]
    assert set(Ls) == {3}


# ---------------------------------------------------------------- causal section is plain AR
def test_causal_slots_equal_plain_causal_forward(model):
    sh, cfg, w, prompt = model
    st, _ = O.prefill(cfg, w, prompt, sh.k)
    st.block[1:] = [11, 22, 33]
    seq = list(prompt) + [int(t) for t in st.block]
    so = O.step(cfg, w, st)
    ref = O.causal_forward(cfg, w, seq)
    n = len(prompt)
    np.testing.assert_allclose(so.fwd.logits[:sh.k], ref.logits[n:n + sh.k], rtol=1e-9, atol=1e-11)
    for l in range(cfg.n_layers):
        np.testing.assert_allclose(so.fwd.k_new[l][:sh.k], ref.k_new[l][n:n + sh.k], rtol=1e-9, atol=1e-12)


# ---------------------------------------------------------------- exact KV cache
def test_kv_cache_equals_one_causal_pass(model):
    sh, cfg, w, prompt = model
    out, Ls, st = O.generate(cfg, w, prompt, sh.k, N_NEW)
    assert st.n == len(prompt) + sum(Ls)
    ref = O.causal_forward(cfg, w, st.tokens[:st.n])
    for l in range(cfg.n_layers):
        assert st.k_cache[l].shape == (st.n, cfg.n_kv_heads, cfg.head_dim)
        np.testing.assert_allclose(st.k_cache[l], ref.k_new[l], rtol=1e-9, atol=1e-12)
        np.testing.assert_allclose(st.v_cache[l], ref.v_new[l], rtol=1e-9, atol=1e-12)


# ---------------------------------------------------------------- pre-drafts
@pytest.mark.parametrize("forced", [1, 2, 4])
def test_selected_predraft_equals_fresh_first_pass(model, forced):
    sh, cfg, w, prompt = model
    st, _ = O.prefill(cfg, w, prompt, sh.k)
    so = O.step(cfg, w, st, forced=forced)
    # a first pass over everything committed so far drafts from the same context
    st2, c2, fo2 = O.prefill(cfg, w, st.tokens[:st.n], sh.k, return_forward=True)
    assert c2 == st.block[0]
    np.testing.assert_array_equal(st2.block, st.block)
    g_step = so.fwd.logits[sh.k + (forced - 1) * sh.k: sh.k + forced * sh.k]
    np.testing.assert_allclose(g_step, fo2.logits[st.n:], rtol=1e-9, atol=1e-11)


def test_first_mask_slot_and_ar_row_predict_the_same_position(model):
    # Section 4.4.3: with beta = 0 the verified token comes from the first slot of
    # the block; the positions line up, so the layout's position ids must agree.
    sh, cfg, w, prompt = model
    _, _, _, pos = O.slot_layout(len(prompt), sh.k)
    for b in range(sh.k):
        assert pos[sh.k + b * sh.k] == pos[b] + 1


def test_beta_endpoints_select_one_head_each(model):
    """Section 4.4.3 pinned without the oracle's own mixing formula: at beta = 1 the verified targets are
    the argmax of the causal rows alone, at beta = 0 the argmax of the first slot of each block alone
    (each compared with the logits of an UNMIXED run), and the settled first token of the prefill
    switches between the last prompt row and the first mask row in the same way."""
    sh, cfg, w, prompt = model
    n, k = len(prompt), sh.k
    runs = {}
    for beta in (1.0, 0.0):
        cfg_b = replace(cfg, beta=beta)
        st, c, fo = O.prefill(cfg_b, w, prompt, k, return_forward=True)
        st.block = np.array(runs[1.0][0] if beta == 0.0 else st.block)      # same drafts in both runs
        block = st.block.copy()
        so = O.step(cfg_b, w, st)
        runs[beta] = (block, c, fo, so)
    _, c1, fo1, so1 = runs[1.0]
    _, c0, fo0, so0 = runs[0.0]
    np.testing.assert_array_equal(fo1.logits, fo0.logits)                   # beta does not touch the forward pass
    assert c1 == int(np.argmax(fo1.logits[n - 1])) and c0 == int(np.argmax(fo1.logits[n]))
    a = so1.fwd.logits[:k]
    g0 = so1.fwd.logits[k:].reshape(k, k, -1)[:, 0]
    np.testing.assert_array_equal(so1.targets, a.argmax(-1))
    # the beta = 0 run starts from a different settled token, so compare on its own unmixed logits
    a_0 = so0.fwd.logits[:k]; g0_0 = so0.fwd.logits[k:].reshape(k, k, -1)[:, 0]
    np.testing.assert_array_equal(so0.targets, g0_0.argmax(-1))
    assert not np.array_equal(a_0.argmax(-1), g0_0.argmax(-1)) or not np.array_equal(a.argmax(-1), g0.argmax(-1)), \
        "the two heads agree everywhere on this input: the endpoints are not told apart"


def test_beta_mix_on_hand_built_logits():
    """The mixing rule on three-logit rows worked by hand (not by the oracle's expression): the
    autoregressive row prefers id 0, the diffusion row id 2."""
    a = np.array([[2.0, 1.0, 0.0]]); g0 = np.array([[0.0, 1.0, 4.0]])
    # beta = 0.5: [1.0, 1.0, 2.0] -> id 2;  beta = 0.75: [1.5, 1.0, 1.0] -> id 0;  beta = 2/3: [4/3, 1, 4/3] ties -> lowest id 0
    hand = {1.0: 0, 0.0: 2, 0.5: 2, 0.75: 0}
    for beta, want in hand.items():
        mixed = np.array([[beta * 2.0 + (1 - beta) * 0.0, 1.0, (1 - beta) * 4.0]])
        assert int(O.argmax_lowest(mixed)[0]) == want
        assert int(O.argmax_lowest(beta * a + (1.0 - beta) * g0)[0]) == want
    assert int(O.argmax_lowest(np.array([[1.25, 1.0, 1.25]]))[0]) == 0      # ties go to the lowest id


def test_beta_half_step_uses_the_mixed_row(model):
    """beta = 0.5 in a real step: the targets are neither head's argmax in general, and on every slot
    they beat both heads' choices under the mixed score (checked through the scores, not the argmax)."""
    sh, cfg, w, prompt = model
    k = sh.k
    cfg_b = replace(cfg, beta=0.5)
    st, _ = O.prefill(cfg_b, w, prompt, k)
    so = O.step(cfg_b, w, st)
    a = so.fwd.logits[:k]
    g0 = so.fwd.logits[k:].reshape(k, k, -1)[:, 0]
    for j in range(k):
        score = lambda v: 0.5 * a[j, v] + 0.5 * g0[j, v]
        tj = int(so.targets[j])
        assert score(tj) >= score(int(a[j].argmax())) and score(tj) >= score(int(g0[j].argmax()))
        assert score(tj) >= max(score(v) for v in range(0, sh.vocab, 7))


# ---------------------------------------------------------------- planted mistakes must be caught
def _with_mask(monkeypatch, fn):
    orig = O.build_decode_mask

    def patched(n, k):
        m = orig(n, k).copy()
        fn(m, n, k)
        return m

    monkeypatch.setattr(O, "build_decode_mask", patched)


def test_planted_causal_sees_mask_slot_breaks_ar_equivalence(model, ar_tokens, monkeypatch):
    sh, cfg, w, prompt = model
    _with_mask(monkeypatch, lambda m, n, k: m.__setitem__((slice(0, k), slice(n + k, n + 2 * k)), True))
    st, _ = O.prefill(cfg, w, prompt, sh.k)
    seq = list(prompt) + [int(t) for t in st.block]
    so = O.step(cfg, w, st)
    ref = O.causal_forward(cfg, w, seq)
    assert np.abs(so.fwd.logits[:sh.k] - ref.logits[len(prompt):len(prompt) + sh.k]).max() > 1e-6


def test_planted_block_sees_one_more_draft_breaks_predraft_pin(model, monkeypatch):
    sh, cfg, w, prompt = model

    def widen(m, n, k):               # block b also sees causal slot b+1
        for b in range(k - 1):
            m[k + b * k:k + (b + 1) * k, n + b + 1] = True

    _with_mask(monkeypatch, widen)
    st, _ = O.prefill(cfg, w, prompt, sh.k)
    st.block[1:] = [11, 22, 33]
    so = O.step(cfg, w, st, forced=2)
    monkeypatch.undo()
    _, _, fo2 = O.prefill(cfg, w, st.tokens[:st.n], sh.k, return_forward=True)
    g_step = so.fwd.logits[sh.k + sh.k: sh.k + 2 * sh.k]
    assert np.abs(g_step - fo2.logits[st.n:]).max() > 1e-6


def test_planted_wrong_mask_position_breaks_predraft_pin(model, monkeypatch):
    sh, cfg, w, prompt = model
    orig = O.slot_layout

    def shifted(n, k):
        kind, blk, idx, pos = orig(n, k)
        pos = pos.copy()
        pos[k:] -= 1                  # label-shifted positions: the reading the paper rules out
        return kind, blk, idx, pos

    monkeypatch.setattr(O, "slot_layout", shifted)
    st, _ = O.prefill(cfg, w, prompt, sh.k)
    so = O.step(cfg, w, st, forced=1)
    monkeypatch.undo()
    _, _, fo2 = O.prefill(cfg, w, st.tokens[:st.n], sh.k, return_forward=True)
    assert np.abs(so.fwd.logits[sh.k:2 * sh.k] - fo2.logits[st.n:]).max() > 1e-6


# ---------------------------------------------------------------- seeded sampling
def test_hash_functions_match_their_published_values():
    # SplitMix64 started at 0 produces 0xE220A8397B1DCDAF, 0x6E789E6AA1B965F4, 0x06C45D188009454F (the reference
    # implementation's first outputs): output i is mix64 of i+1 times the golden-ratio increment
    g = 0x9E3779B97F4A7C15
    assert [O.mix64((i + 1) * g) for i in range(3)] == [0xE220A8397B1DCDAF, 0x6E789E6AA1B965F4, 0x06C45D188009454F]
    # MurmurHash3's 32-bit finaliser: 0 is a fixed point, fmix32(1) = 0x514E28B7; it is a bijection, so
    # 2^16 distinct inputs give 2^16 distinct outputs
    np.testing.assert_array_equal(O.fmix32(np.array([0, 1], dtype=np.uint32)), np.array([0, 0x514E28B7], dtype=np.uint32))
    assert len(np.unique(O.fmix32(np.arange(1 << 16, dtype=np.uint32)))) == 1 << 16


def test_gumbel_noise_is_standard_gumbel_and_keyed_by_position_only():
    g = np.concatenate([O.gumbel_noise(11, 0, p, 4096) for p in range(64)])
    # standard Gumbel: mean = Euler's constant, variance = pi^2 / 6, median = -ln ln 2
    assert abs(g.mean() - 0.5772156649) < 0.01 and abs(g.var() - np.pi ** 2 / 6) < 0.03
    assert abs(np.median(g) + np.log(np.log(2.0))) < 0.01
    np.testing.assert_array_equal(O.gumbel_noise(11, 3, 77, 100), O.gumbel_noise(11, 3, 77, 1000)[:100])   # a pure function of (seed, seq, pos, id)
    for other in (O.gumbel_noise(12, 3, 77, 100), O.gumbel_noise(11, 4, 77, 100), O.gumbel_noise(11, 3, 78, 100)):
        assert np.abs(other - O.gumbel_noise(11, 3, 77, 100)).min() > 0 or not np.array_equal(other, O.gumbel_noise(11, 3, 77, 100))


def test_draws_follow_softmax_of_the_tempered_logits():
    """Gumbel-max sampling pinned by what it must reproduce: over many positions the frequency of every token
    is its softmax(logits / temperature) probability; temperature -> 0 gives the argmax."""
    from dataclasses import replace
    sh = CONFIGS["tiny"]
    base = _cfg(sh)
    logits = np.array([2.0, 1.0, 0.5, 0.0, -1.0, -3.0])
    for temp in (1.0, 0.5):
        cfg = replace(base, temperature=temp, sample_seed=5)
        n = 20000
        draws = O.choose_tokens(cfg, np.tile(logits, (n, 1)), np.arange(n))
        p = np.exp(logits / temp); p /= p.sum()
        freq = np.bincount(draws, minlength=len(logits)) / n
        assert np.abs(freq - p).max() < 4.5 * np.sqrt(p.max() * (1 - p.max()) / n) + 1e-3, (freq, p)
    cold = replace(base, temperature=1e-4, sample_seed=5)
    assert (O.choose_tokens(cold, np.tile(logits, (50, 1)), np.arange(50)) == 0).all()
    assert (O.choose_tokens(base, np.tile(logits, (3, 1)), np.arange(3)) == 0).all()         # temperature 0: argmax


@pytest.mark.parametrize("drafts", ["natural", "garbage"])
def test_sampled_tidar_equals_sampled_autoregressive_decoding(model, drafts):
    """The noise of a draw depends on the predicted position only, so with beta = 1 sampled TiDAR must emit
    exactly what one-token-per-pass sampled decoding emits, whatever the drafts were; and the draws differ
    from greedy decoding (the temperature is live)."""
    from dataclasses import replace
    sh, cfg, w, prompt = model
    cfg_s = replace(cfg, temperature=0.9, sample_seed=21)
    ar = O.ar_generate(cfg_s, w, prompt, 24)
    rng = np.random.default_rng(0)

    def garbage(st):
        st.block[1:] = rng.integers(0, sh.vocab - 1, len(st.block) - 1)
    out, Ls, _ = O.generate(cfg_s, w, prompt, sh.k, 24, draft_hook=garbage if drafts == "garbage" else None)
    assert out == ar
    assert ar != O.ar_generate(cfg, w, prompt, 24)
    if drafts == "garbage":
        assert max(Ls) <= 2
    # another sequence slot or seed draws differently
    assert O.ar_generate(replace(cfg_s, seq=1), w, prompt, 24) != ar and O.ar_generate(replace(cfg_s, sample_seed=22), w, prompt, 24) != ar
