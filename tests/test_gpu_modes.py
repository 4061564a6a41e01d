"""Autoregressive mode, likelihood scoring, per-step block length and beta < 1 on the GPU
(needs a B200): every entry point through the C ABI against the oracle."""
from dataclasses import replace

import numpy as np
import pytest
import torch  # noqa: F401

from oracle import tidar_oracle as O
from tests.helpers import MARGIN, TOL_LOGITS, check_rows, make_model, oracle_cfg, prompt_ids, top1_margin

pytestmark = pytest.mark.gpu

IMPLS = [0, 1]


def _gpu(sh, wt, impl, k_max, debug=0, max_batch=1, max_seq_len=512, beta=1.0):
    from paper_2511_08923_b200 import Tidar, pack_weights
    return Tidar(sh, pack_weights(wt, "cuda:0"), k_max=k_max, max_batch=max_batch, max_seq_len=max_seq_len, debug=debug, impl=impl,
                 guard_bytes=64 * 1024, beta=beta)


def _close(t):
    assert t.arena_guard_intact()
    t.close()


@pytest.fixture(scope="module")
def tiny():
    sh, wt = make_model("tiny", tied=False)
    return sh, wt, oracle_cfg(sh), O.weights_to_f64(wt), prompt_ids(sh)


@pytest.mark.parametrize("impl", IMPLS)
def test_autoregressive_steps_match_plain_greedy_decoding(tiny, impl):
    """tidar_ar_step (one causal slot, no mask slots) against the oracle's one-token-per-pass decoder."""
    sh, wt, cfg, w, prompt = tiny
    n_new = 24
    ar = O.ar_generate(cfg, w, prompt, n_new)
    t = _gpu(sh, wt, impl, k_max=4)
    first = t.prefill(0, prompt, 1)
    fo = O.causal_forward(cfg, w, list(prompt) + ar)
    m = top1_margin(fo.logits[len(prompt) - 1:len(prompt) - 1 + n_new])      # margin of the prediction of new token i
    if m[0] > MARGIN:
        assert first == ar[0]
    launches0 = t.launch_count()
    checked = 0
    for i in range(n_new - 1):                      # teacher-forced with the oracle's tokens: the caches stay comparable
        t.set_block(0, [ar[i]])
        nxt = t.ar_step([0])
        if m[i + 1] > MARGIN:
            assert nxt == [ar[i + 1]], (i, nxt, ar[i + 1])
            checked += 1
    assert checked >= n_new // 2
    per_step = (t.launch_count() - launches0) / (n_new - 1)
    assert t.seq_len(0) == len(prompt) + n_new - 1
    # the committed cache is the one a causal pass over the same tokens gives
    from paper_2511_08923_b200 import bf16_bits_to_f32
    n = t.seq_len(0)
    for l in range(cfg.n_layers):
        kk, vv = t.kv(0, l, 0, n)
        assert np.abs(bf16_bits_to_f32(kk) - fo.k_new[l][:n]).max() <= TOL_LOGITS
        assert np.abs(bf16_bits_to_f32(vv) - fo.v_new[l][:n]).max() <= TOL_LOGITS
    # a TiDAR step after autoregressive steps finds no drafts: it accepts one token and leaves a full block
    toks, L = t.step_k([0], 4)
    assert L == [1] and len(t.get_block(0, 4)) == 4
    toks2, L2 = t.step([0])
    assert 1 <= L2[0] <= 4
    assert per_step < 60, per_step            # one slot per sequence: no mask-slot work
    _close(t)


@pytest.mark.parametrize("impl", IMPLS)
def test_likelihood_scoring_matches_causal_log_softmax(tiny, impl):
    """tidar_score: log p(next token) of every position from one causal pass (the model's
    autoregressive mode), against log-softmax of the oracle's causal logits; also across chunks."""
    sh, wt, cfg, w, prompt = tiny
    rng = np.random.default_rng(5)
    for n in (2, 37, 300):                          # 300 rows: more than one chunk of the row capacity
        ids = rng.integers(0, sh.vocab - 1, n)
        fo = O.causal_forward(cfg, w, ids)
        lg = fo.logits[:-1]
        lse = np.log(np.exp(lg - lg.max(-1, keepdims=True)).sum(-1)) + lg.max(-1)
        want = lg[np.arange(n - 1), ids[1:]] - lse
        t = _gpu(sh, wt, impl, k_max=4)
        got = t.score(0, ids)
        assert got.shape == (n - 1,)
        assert np.abs(got - want).max() <= TOL_LOGITS, np.abs(got - want).max()
        # the slot was scratch: nothing is left in it, and it can be prefilled afterwards
        from paper_2511_08923_b200 import TidarError
        with pytest.raises(TidarError):
            t.step([0])
        t.prefill(0, prompt, 4); t.step([0])
        _close(t)


def test_autoregressive_mode_at_the_benchmark_widths():
    """The one-slot step and the scoring pass at the 8B-class widths (two layers, 8192-entry vocabulary so
    that the oracle stays fast): one-row projections (a 16-row MMA block), 4096-wide rows, 32 / 8 heads.
    Logits of every autoregressive step and the log-probabilities of a 300-token pass against the oracle."""
    from dataclasses import replace as _r
    from tidar_synth import CONFIGS as CONFIGS_, gen_model_weights as gen_model_weights_
    sh = _r(CONFIGS_["8b"].reduced(2), vocab=8192)
    wt = gen_model_weights_(sh)
    cfg, w = oracle_cfg(sh), O.weights_to_f64(wt)
    prompt = prompt_ids(sh, n=90)
    n_new = 8
    ar = O.ar_generate(cfg, w, prompt, n_new)
    fo = O.causal_forward(cfg, w, list(prompt) + ar)
    m = top1_margin(fo.logits[len(prompt) - 1:len(prompt) - 1 + n_new])
    t = _gpu(sh, wt, 0, k_max=4, debug=1, max_seq_len=512)
    first = t.prefill(0, prompt, 1)
    if m[0] > MARGIN:
        assert first == ar[0]
    for i in range(n_new - 1):
        t.set_block(0, [ar[i]])                     # teacher-forced with the oracle's tokens
        nxt = t.ar_step([0])
        n_rows, _ = t.last_rows()
        assert n_rows == 1
        check_rows(t.logits(0, 1), fo.logits[len(prompt) + i:len(prompt) + i + 1], f"AR step {i} logits")
        if m[i + 1] > MARGIN:
            assert nxt == [ar[i + 1]], (i, nxt, ar[i + 1])
    _close(t)
    rng = np.random.default_rng(11)
    ids = rng.integers(0, sh.vocab - 1, 300)
    lg = O.causal_forward(cfg, w, ids).logits[:-1]
    lse = np.log(np.exp(lg - lg.max(-1, keepdims=True)).sum(-1)) + lg.max(-1)
    want = lg[np.arange(len(ids) - 1), ids[1:]] - lse
    t = _gpu(sh, wt, 0, k_max=4, max_seq_len=512)
    got = t.score(0, ids)
    # a log-probability is a logit minus a log-sum-exp, and the log-sum-exp moves by at most the largest
    # logit error: twice the per-row logit bound of the full-width comparisons (check_rows)
    bound = 2 * TOL_LOGITS * np.maximum(1.0, np.maximum(np.abs(lg).max(-1), 4 * np.sqrt((lg ** 2).mean(-1))))
    assert (np.abs(got - want) <= bound).all(), (np.abs(got - want) / bound).max()
    assert np.sqrt(((got - want) ** 2).mean()) <= 0.5 * TOL_LOGITS            # and far better on average
    _close(t)


@pytest.mark.parametrize("impl", IMPLS)
def test_block_length_chosen_per_step(tiny, impl):
    """tidar_step_k: shorter and longer blocks than the previous pass left.  Greedy TiDAR with beta = 1
    emits the autoregressive continuation whatever the block lengths are; a step that asks for more
    drafts than the sequence holds feeds mask tokens for the missing ones and never accepts them."""
    sh, wt, cfg, w, prompt = tiny
    n_new = 40
    ar = O.ar_generate(cfg, w, prompt, n_new + 8)
    fo = O.causal_forward(cfg, w, list(prompt) + ar)
    m = top1_margin(fo.logits[len(prompt) - 1:len(prompt) - 1 + n_new])
    unsure = np.nonzero(m <= MARGIN)[0]
    upto = int(unsure[0]) if len(unsure) else n_new
    t = _gpu(sh, wt, impl, k_max=8, max_seq_len=256)
    out = [t.prefill(0, prompt, 4)]
    held = 4
    for k in (2, 8, 8, 3, 1, 5, 8, 4, 4, 8, 8, 8):
        toks, L = t.step_k([0], k)
        assert 1 <= L[0] <= min(k, held), (k, held, L)         # only drafts the sequence holds can be accepted
        out.extend(toks[0]); held = k
        assert t.seq_len(0) == len(prompt) + len(out) - 1
        if len(out) >= n_new:
            break
    assert out[:upto] == ar[:upto]
    assert t.ridge_k(1) == 8 and t.ridge_k(4) == 8 and t.ridge_k(8, 288) == 5 and t.ridge_k(32, 288) == 2 and t.ridge_k(1000) == 1
    _close(t)


@pytest.mark.parametrize("impl", IMPLS)
def test_block_length_per_sequence_within_one_step(tiny, impl):
    """tidar_step_ks: three sequences with block lengths 2, 4 and 3 share one pass (20 + 6 + 12 slots laid
    out sequence after sequence).  Per sequence the logits, the acceptance and the committed cache are
    those of the oracle's own step with that sequence's block length."""
    from paper_2511_08923_b200 import TidarError, bf16_bits_to_f32
    sh, wt, cfg, w, prompt = tiny
    ks = [4, 2, 3]
    prompts = [prompt, prompt_ids(sh, n=sh.prompt_len - 5, seed=sh.seed + 1), prompt_ids(sh, n=sh.prompt_len + 9, seed=sh.seed + 2)]
    t = _gpu(sh, wt, impl, k_max=4, debug=1, max_batch=3, max_seq_len=256)
    states = []
    for q, (p, k) in enumerate(zip(prompts, ks)):
        t.prefill(q, p, k)
        states.append(O.prefill(cfg, w, p, k)[0])
    order = [2, 0, 1]                                              # listed order need not be slot order
    for step in range(5):
        forced = [0, 0, 0] if step != 2 else [1, 2, 1]
        blocks, outs = [], []
        for q in order:
            t.set_block(q, states[q].block)                        # teacher-forced: the caches stay comparable
            blocks.append(states[q].block.copy())
        for i, q in enumerate(order):
            outs.append(O.step(cfg, w, states[q], forced=forced[i]))
        toks, L = t.step_ks(order, [ks[q] for q in order], forced if step == 2 else None)
        n_rows, _ = t.last_rows()
        assert n_rows == sum(ks[q] * (ks[q] + 1) for q in order)
        lg = t.logits(0, n_rows)
        ids = t.argmax(0, n_rows)
        r0 = 0
        for i, q in enumerate(order):
            k = ks[q]; T = k * (k + 1)
            assert np.abs(lg[r0:r0 + T] - outs[i].fwd.logits).max() <= TOL_LOGITS, (step, q)
            L_ref = O.accept_length(blocks[i], ids[r0:r0 + k], forced[i])
            assert L[i] == L_ref
            assert toks[i] == [int(x) for x in blocks[i][1:L_ref]] + [int(ids[r0 + L_ref - 1])]
            if L[i] != outs[i].L or toks[i] != outs[i].emitted:    # only a near-tie may be decided the other way
                assert top1_margin(outs[i].fwd.logits[:k]).min() <= MARGIN, (step, q, L[i], outs[i].L)
                pytest.skip("near-tie in a verified position of the synthetic model")
            assert t.seq_len(q) == states[q].n
            assert t.get_block(q, k)[0] == int(states[q].block[0])
            r0 += T
    for q in range(3):
        n = t.seq_len(q)
        for l in range(cfg.n_layers):
            K, V = t.kv(q, l, 0, n)
            check_rows(bf16_bits_to_f32(K).reshape(n, -1), states[q].k_cache[l].reshape(n, -1), f"K seq {q} layer {l}")
            check_rows(bf16_bits_to_f32(V).reshape(n, -1), states[q].v_cache[l].reshape(n, -1), f"V seq {q} layer {l}")
    with pytest.raises(TidarError):
        t.step_ks([0, 1], [4, 5])                                  # above k_max
    with pytest.raises(TidarError):
        t.step_ks([0, 1], [2, 3], [3, 1])                          # forced acceptance above that sequence's length
    toks, L = t.step_ks([0, 1, 2], [3, 3, 3])                      # equal lengths: the ordinary step
    assert all(1 <= x <= 3 for x in L)
    _close(t)


@pytest.mark.parametrize("impl", IMPLS)
def test_block_length_per_sequence_with_beta_mixing(tiny, impl):
    """beta < 1 in a step of mixed block lengths: the mixed verification rows (one per verified position,
    sequence after sequence) follow the slots; per sequence the mixed logits, the acceptance and the tokens
    are those of the oracle's own step at that block length (paper Section 4.4.3)."""
    sh, wt, cfg, w, prompt = tiny
    beta = 0.5
    cfg_b = replace(cfg, beta=beta)
    ks = [3, 4, 2]
    prompts = [prompt, prompt_ids(sh, n=sh.prompt_len - 4, seed=sh.seed + 5), prompt_ids(sh, n=sh.prompt_len + 6, seed=sh.seed + 6)]
    t = _gpu(sh, wt, impl, k_max=4, debug=1, max_batch=3, max_seq_len=256, beta=beta)
    states = []
    for q, (p, k) in enumerate(zip(prompts, ks)):
        t.prefill(q, p, k)
        states.append(O.prefill(cfg_b, w, p, k)[0])
    R = sum(k * (k + 1) for k in ks)
    for step in range(3):
        blocks = []
        for q in range(3):
            t.set_block(q, states[q].block)
            blocks.append(states[q].block.copy())
        outs = [O.step(cfg_b, w, states[q]) for q in range(3)]
        toks, L = t.step_ks([0, 1, 2], ks)
        n_rows, _ = t.last_rows()
        assert n_rows == R + sum(ks)
        lg = t.logits(0, n_rows)
        ids = t.argmax(0, n_rows)
        r0, m0 = 0, R
        for q, k in enumerate(ks):
            T = k * (k + 1)
            fo = outs[q].fwd.logits
            ref_mixed = beta * fo[:k] + (1 - beta) * fo[k:].reshape(k, k, -1)[:, 0, :]
            assert np.abs(lg[r0:r0 + T] - fo).max() <= TOL_LOGITS
            assert np.abs(lg[m0:m0 + k] - ref_mixed).max() <= TOL_LOGITS, (step, q)
            tg = ids[m0:m0 + k]
            L_ref = O.accept_length(blocks[q], tg)
            assert L[q] == L_ref and toks[q] == [int(x) for x in blocks[q][1:L_ref]] + [int(tg[L_ref - 1])]
            if top1_margin(ref_mixed).min() > MARGIN:
                assert L[q] == outs[q].L and toks[q] == outs[q].emitted
            r0 += T; m0 += k
        if any(L[q] != outs[q].L for q in range(3)):
            break                                   # a near-tie went the other way: the caches have parted
    _close(t)


@pytest.mark.parametrize("impl", IMPLS)
def test_mixed_block_lengths_keep_the_autoregressive_continuation(tiny, impl):
    """With beta = 1 and greedy decoding every sequence of a mixed step still emits the model's
    autoregressive continuation, whatever lengths the steps choose (changing from step to step)."""
    sh, wt, cfg, w, prompt = tiny
    n_new = 28
    prompts = [prompt, prompt_ids(sh, n=sh.prompt_len + 3, seed=sh.seed + 7)]
    refs, upto = [], []
    for p in prompts:
        ar = O.ar_generate(cfg, w, p, n_new + 8)
        m = top1_margin(O.causal_forward(cfg, w, list(p) + ar).logits[len(p) - 1:len(p) - 1 + n_new])
        unsure = np.nonzero(m <= MARGIN)[0]
        refs.append(ar); upto.append(int(unsure[0]) if len(unsure) else n_new)
    t = _gpu(sh, wt, impl, k_max=8, max_batch=2, max_seq_len=256)
    out = [[t.prefill(q, p, 4)] for q, p in enumerate(prompts)]
    plan = [(2, 8), (8, 3), (5, 5), (1, 7), (8, 8), (3, 6), (6, 2), (8, 4), (4, 8), (7, 7), (8, 8), (8, 8)]
    for ka, kb in plan:
        toks, L = t.step_ks([0, 1], [ka, kb])
        for q in range(2):
            out[q].extend(toks[q])
            assert t.seq_len(q) == len(prompts[q]) + len(out[q]) - 1
        if min(len(o) for o in out) >= n_new:
            break
    for q in range(2):
        assert out[q][:upto[q]] == refs[q][:upto[q]], q
    _close(t)


def test_mixed_step_graph_replay_matches_plain_launches():
    """A step of mixed block lengths replays one captured graph for every length vector with the same
    row and tile count ((3, 4, 2) and (2, 3, 4) here, the layout living in device memory); the same
    teacher-forced steps launched kernel by kernel give identical tokens and bit-identical cached K/V."""
    from dataclasses import replace as _r
    from tidar_synth import CONFIGS as CONFIGS_, gen_model_weights as gen_model_weights_
    sh = _r(CONFIGS_["8b"].reduced(2), vocab=8192)
    wt = gen_model_weights_(sh)
    prompts = [prompt_ids(sh, n=150 + 37 * q, seed=sh.seed + q) for q in range(3)]
    plan = [([3, 4, 2], [2, 1, 2]), ([2, 3, 4], [1, 3, 4]), ([3, 4, 2], [3, 2, 1]), ([4, 4, 4], [4, 1, 2]), ([4, 2, 3], [2, 2, 3])]
    runs = {}
    for tag, debug in (("graph", 0), ("plain", 8)):
        t = _gpu(sh, wt, 0, k_max=4, debug=debug, max_batch=3, max_seq_len=512)
        rec = [t.prefill(q, p, 4) for q, p in enumerate(prompts)]
        blocks = [[t.get_block(q, 4) for q in range(3)]]
        l0 = t.launch_count()
        for i, (ks, forced) in enumerate(plan):
            if tag == "plain":
                for q in range(3):
                    t.set_block(q, runs["graph"]["blocks"][i][q])
            rec.append(t.step_ks([0, 1, 2], ks, forced))
            blocks.append([t.get_block(q, ks[q]) + [0] * (4 - ks[q]) for q in range(3)])
        kv = [[t.kv(q, l, 0, t.seq_len(q)) for l in range(sh.n_layers)] for q in range(3)]
        runs[tag] = {"rec": rec, "blocks": blocks, "kv": kv, "launches": t.launch_count() - l0}
        _close(t)
    assert runs["graph"]["rec"] == runs["plain"]["rec"]
    assert runs["graph"]["blocks"] == runs["plain"]["blocks"]
    assert runs["graph"]["launches"] == runs["plain"]["launches"]              # replayed launches are counted like recorded ones
    for q in range(3):
        for (k0, v0), (k1, v1) in zip(runs["graph"]["kv"][q], runs["plain"]["kv"][q]):
            np.testing.assert_array_equal(k0, k1); np.testing.assert_array_equal(v0, v1)


@pytest.mark.parametrize("impl", IMPLS)
def test_continuous_batching_with_planned_block_lengths(tiny, impl):
    """Sequences that want different numbers of tokens share steps whose block lengths come from
    tidar_plan_ks under a small slot budget; a finished sequence is released and the next prompt takes its
    slot.  Every request still receives exactly the model's greedy autoregressive continuation."""
    from paper_2511_08923_b200 import plan_ks
    sh, wt, cfg, w, prompt = tiny
    wants = [9, 21, 5, 14, 12]
    prompts = [prompt_ids(sh, n=sh.prompt_len - 7 + 3 * r, seed=sh.seed + 11 + r) for r in range(len(wants))]
    refs, sure = [], []
    for p, n_new in zip(prompts, wants):
        ar = O.ar_generate(cfg, w, p, n_new + 1)
        m = top1_margin(O.causal_forward(cfg, w, list(p) + ar).logits[len(p) - 1:len(p) - 1 + n_new])
        unsure = np.nonzero(m <= MARGIN)[0]
        refs.append(ar[:n_new]); sure.append(int(unsure[0]) if len(unsure) else n_new)
    k_max, budget = 6, 44
    t = _gpu(sh, wt, impl, k_max=k_max, max_batch=2, max_seq_len=256)
    waiting = list(range(len(wants)))
    slot_req = {}                                   # slot -> request
    out = {r: [] for r in range(len(wants))}
    steps = 0
    while waiting or slot_req:
        for slot in range(2):                       # admit
            if slot not in slot_req and waiting:
                r = waiting.pop(0)
                out[r].append(t.prefill(slot, prompts[r], 1))
                slot_req[slot] = r
        slots = sorted(s for s in slot_req if len(out[slot_req[s]]) < wants[slot_req[s]])
        if slots:
            remaining = [wants[slot_req[s]] - len(out[slot_req[s]]) for s in slots]
            ks = plan_ks(len(slots), k_max, budget, remaining)
            assert sum(k * (k + 1) for k in ks) <= budget and all(k <= rem for k, rem in zip(ks, remaining))
            toks, L = t.step_ks(slots, ks)
            for s, tk in zip(slots, toks):
                out[slot_req[s]].extend(tk)
            steps += 1
        for s in list(slot_req):                    # retire
            r = slot_req[s]
            if len(out[r]) >= wants[r]:
                assert len(out[r]) == wants[r]      # the cap keeps a step from running past the request
                t.release(s)
                del slot_req[s]
        assert steps < 200
    for r in range(len(wants)):
        assert out[r][:sure[r]] == refs[r][:sure[r]], r
    with pytest.raises(Exception):
        t.step([0])                                 # released slots hold nothing
    _close(t)


# ---- beta < 1 ------------------------------------------------------------------------------------
@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("beta", [0.0, 0.5])
def test_beta_mixed_verification(tiny, impl, beta):
    """beta < 1 (paper Section 4.4.3): drafts are verified against argmax(beta * logits_ar + (1 - beta) *
    logits_diff).  beta = 0 trusts the diffusion prediction alone: the verified targets must equal the
    argmax of the first slot of each block, which the GPU also reports on its own rows."""
    sh, wt, cfg, w, prompt = tiny
    k = sh.k
    cfg_b = replace(cfg, beta=beta)
    t = _gpu(sh, wt, impl, k_max=k, debug=1, beta=beta)
    first = t.prefill(0, prompt, k)
    st, c, fo = O.prefill(cfg_b, w, prompt, k, return_forward=True)
    n = len(prompt)
    mixed = beta * fo.logits[n - 1] + (1 - beta) * fo.logits[n]
    if top1_margin(mixed) > MARGIN:
        assert first == c
    T = k * (k + 1)
    for s in range(4):
        t.set_block(0, st.block)
        block = st.block.copy()
        so = O.step(cfg_b, w, st)
        toks, L = t.step([0])
        n_rows, _ = t.last_rows()
        assert n_rows == T + k                      # the k mixed rows follow the slots
        lg = t.logits(0, n_rows)
        ids = t.argmax(0, n_rows)
        ref_mixed = beta * so.fwd.logits[:k] + (1 - beta) * so.fwd.logits[k:].reshape(k, k, -1)[:, 0, :]
        assert np.abs(lg[:T] - so.fwd.logits).max() <= TOL_LOGITS
        assert np.abs(lg[T:] - ref_mixed).max() <= TOL_LOGITS          # mixing the LM head's input rows = mixing the logits
        tg = ids[T:]
        if beta == 0.0:                             # the diffusion prediction alone
            np.testing.assert_array_equal(lg[T:].argmax(-1), lg[k:T:k].argmax(-1))
        L_ref = O.accept_length(block, tg)
        assert L[0] == L_ref and toks[0] == [int(x) for x in block[1:L_ref]] + [int(tg[L_ref - 1])]
        if (top1_margin(ref_mixed) > MARGIN).all():
            assert L[0] == so.L and toks[0] == so.emitted
        elif L[0] != so.L:
            break
    _close(t)


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("family,hd", [("bias", 64), ("qk_norm", 64), ("bias", 128), ("qk_norm", 128)])
def test_projection_bias_and_per_head_qk_norm(impl, family, hd):
    """The two attention-block details in which the decoder families the paper starts from differ
    (Section 4.1): biases on Q/K/V, or an RMSNorm over each Q / K head before RoPE.  First pass and
    teacher-forced steps against the oracle, for both head widths the kernels support."""
    from paper_2511_08923_b200 import bf16_bits_to_f32
    from tidar_synth import CONFIGS, gen_model_weights
    over = dict(head_dim=hd, n_q_heads=4, n_kv_heads=2, d_model=256) if hd == 64 else dict(head_dim=hd, n_q_heads=6, n_kv_heads=2, d_model=512, d_ffn=768)
    sh = replace(CONFIGS["tiny"], name=f"{family}{hd}", tie_lm_head=False, qkv_bias=family == "bias", qk_norm=family == "qk_norm", **over)
    wt = gen_model_weights(sh)
    cfg, w = oracle_cfg(sh), O.weights_to_f64(wt)
    prompt = prompt_ids(sh, 70)
    k, n = sh.k, 70
    t = _gpu(sh, wt, impl, k_max=k, debug=1)
    t.prefill(0, prompt, k)
    st, c, fo = O.prefill(cfg, w, prompt, k, return_forward=True)
    assert np.abs(t.logits(0, n + k) - fo.logits).max() <= TOL_LOGITS
    for l in range(cfg.n_layers):                   # normed K reaches |x| ~ 5, where one bf16 ulp is 0.03: bound by the row's scale
        kk, vv = t.kv(0, l, 0, n)
        check_rows(bf16_bits_to_f32(kk).reshape(n, -1), st.k_cache[l].reshape(n, -1), f"K({l})")
        check_rows(bf16_bits_to_f32(vv).reshape(n, -1), st.v_cache[l].reshape(n, -1), f"V({l})")
    # the same weights without the extra tensors give clearly different logits: the option is live on the GPU
    plain = {**wt, "layers": [{a: b for a, b in L.items() if a not in ("bq", "bk", "bv", "q_norm", "k_norm")} for L in wt["layers"]]}
    t0 = _gpu(sh, plain, impl, k_max=k, debug=1)
    t0.prefill(0, prompt, k)
    assert np.abs(t0.logits(0, n + k) - fo.logits).max() > 10 * TOL_LOGITS
    _close(t0)
    for s in range(2):
        t.set_block(0, st.block)
        so = O.step(cfg, w, st, forced=2)
        toks, L = t.step([0], forced=[2])
        assert np.abs(t.logits(0, k * (k + 1)) - so.fwd.logits).max() <= TOL_LOGITS
        if (top1_margin(so.fwd.logits[:k]) > MARGIN).all():
            assert toks[0] == so.emitted
    _close(t)


@pytest.mark.parametrize("impl", IMPLS)
def test_seeded_sampling_draws_what_the_oracle_draws(tiny, impl):
    """temperature > 0: every prediction is a Gumbel-max draw keyed by (seed, slot, predicted position,
    token id).  The GPU's draws of every row equal the argmax of its own tempered logits plus the
    oracle's noise for that position, and follow the oracle's step wherever the noisy margin is clear;
    free-running sampled TiDAR equals sampled one-token-per-pass decoding of the GPU itself."""
    sh, wt, cfg, w, prompt = tiny
    k, temp, seed = sh.k, 0.8, 33
    cfg_s = replace(cfg, temperature=temp, sample_seed=seed, seq=0)
    t = _gpu(sh, wt, impl, k_max=k, debug=1, max_batch=1)
    t.close()
    from paper_2511_08923_b200 import Tidar, pack_weights
    t = Tidar(sh, pack_weights(wt, "cuda:0"), k_max=k, max_seq_len=512, debug=1, impl=impl, temperature=temp, sample_seed=seed, guard_bytes=64 * 1024)
    n = len(prompt)
    T = k * (k + 1)

    def noisy(lg, positions):
        return np.stack([lg[r] / temp + O.gumbel_noise(seed, 0, int(p), sh.vocab) for r, p in enumerate(positions)])

    first = t.prefill(0, prompt, k)
    st, c, fo = O.prefill(cfg_s, w, prompt, k, return_forward=True)
    lg = t.logits(0, n + k)
    pred = np.concatenate([np.arange(1, n + 1), n + np.arange(k)])       # prompt row g predicts g + 1, mask row i predicts n + i
    sc = noisy(lg.astype(np.float64), pred)
    ids = t.argmax(0, n + k)
    m = top1_margin(sc)
    sure = m > 1e-3
    np.testing.assert_array_equal(ids[sure], sc.argmax(-1)[sure])        # the GPU's draw from its own logits
    assert sure.mean() > 0.95
    assert (ids != lg.argmax(-1)).mean() > 0.2                           # and they are draws, not argmaxes
    if top1_margin(noisy(fo.logits[n - 1:n], [n]))[0] > 2 * TOL_LOGITS / temp:
        assert first == c
    for s in range(4):
        t.set_block(0, st.block)
        block = st.block.copy()
        so = O.step(cfg_s, w, st)
        toks, L = t.step([0])
        lg = t.logits(0, T)
        _, _, _, pos = O.slot_layout(st.n - so.L, k)
        pred = np.concatenate([pos[:k] + 1, pos[k:]])
        sc = noisy(lg.astype(np.float64), pred)
        ids = t.argmax(0, T)
        sure = top1_margin(sc) > 1e-3
        np.testing.assert_array_equal(ids[sure], sc.argmax(-1)[sure])
        L_ref = O.accept_length(block, ids[:k])
        assert L[0] == L_ref and toks[0] == [int(x) for x in block[1:L_ref]] + [int(ids[L_ref - 1])]
        ref_sc = noisy(so.fwd.logits, pred)
        if (top1_margin(ref_sc[:k]) > 2 * TOL_LOGITS / temp).all():
            assert L[0] == so.L and toks[0] == so.emitted
        elif L[0] != so.L:
            break
    # free running: sampled TiDAR steps against sampled autoregressive steps on the same GPU kernels
    out = [t.prefill(0, prompt, k)]
    while len(out) < 24:
        out.extend(t.step([0])[0][0])
    ar = [t.prefill(0, prompt, 1)]
    while len(ar) < 24:
        ar.extend(t.ar_step([0]))
    agree = next((i for i, (a, b) in enumerate(zip(out, ar)) if a != b), 24)
    assert agree >= 12, (out, ar)        # identical up to a near-tie of two differently rounded passes
    _close(t)


@pytest.mark.parametrize("impl", IMPLS)
def test_seeded_sampling_with_per_sequence_block_lengths(tiny, impl):
    """temperature > 0 in a step of mixed block lengths: the draw of every row is keyed by its own sequence
    slot and predicted position, so each row of the mixed pass equals the argmax of its tempered logits plus
    the oracle's noise for (slot, position), whatever the neighbours' block lengths are."""
    from paper_2511_08923_b200 import Tidar, pack_weights
    sh, wt, cfg, w, prompt = tiny
    temp, seed = 0.7, 91
    ks = [2, 4, 3]
    prompts = [prompt_ids(sh, n=sh.prompt_len + 2 * q, seed=sh.seed + 20 + q) for q in range(3)]
    t = Tidar(sh, pack_weights(wt, "cuda:0"), k_max=4, max_batch=3, max_seq_len=256, debug=1, impl=impl, temperature=temp, sample_seed=seed,
              guard_bytes=64 * 1024)
    for q in range(3):
        t.prefill(q, prompts[q], ks[q])
    for step in range(3):
        n_before = [t.seq_len(q) for q in range(3)]
        toks, L = t.step_ks([0, 1, 2], ks)
        n_rows, _ = t.last_rows()
        lg = t.logits(0, n_rows).astype(np.float64)
        ids = t.argmax(0, n_rows)
        r0, checked = 0, 0
        for q, k in enumerate(ks):
            _, _, _, pos = O.slot_layout(n_before[q], k)
            pred = np.concatenate([pos[:k] + 1, pos[k:]])          # a causal slot predicts the next position, a mask slot its own
            T = k * (k + 1)
            sc = np.stack([lg[r0 + r] / temp + O.gumbel_noise(seed, q, int(p), sh.vocab) for r, p in enumerate(pred)])
            sure = top1_margin(sc) > 1e-3
            np.testing.assert_array_equal(ids[r0:r0 + T][sure], sc.argmax(-1)[sure])
            checked += int(sure.sum())
            assert 1 <= L[q] <= k and t.seq_len(q) == n_before[q] + L[q]
            r0 += T
        assert checked >= 0.9 * n_rows
    assert t.arena_guard_intact()
    t.close()
