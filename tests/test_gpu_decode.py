"""CUDA path vs oracle on the decode step, through the C ABI (needs a B200)."""
import itertools

import numpy as np
import pytest
import torch

from oracle import tidar_oracle as O
from tests.helpers import MARGIN, TOL_LOGITS, make_model, oracle_cfg, prompt_ids, top1_margin
from tidar_synth import CONFIGS as CONFIGS_, gen_model_weights as gen_model_weights_

pytestmark = pytest.mark.gpu

IMPLS = [0, 1]


def _gpu(sh, wt, impl, k_max=None, debug=1, max_batch=1, max_seq_len=512, prefill_rows=0):
    """A context whose arena is followed by 64 KiB of sentinel bytes; _close() checks them."""
    from paper_2511_08923_b200 import Tidar, pack_weights
    packed = pack_weights(wt, "cuda:0")
    return Tidar(sh, packed, k_max=k_max or sh.k, max_batch=max_batch, max_seq_len=max_seq_len, debug=debug, impl=impl,
                 guard_bytes=64 * 1024, prefill_rows=prefill_rows)


def _close(t):
    assert t.arena_guard_intact(), "a kernel wrote past the end of the arena"
    t.close()


@pytest.fixture(scope="module", params=[True, False], ids=["tied", "untied"])
def tiny(request):
    sh, wt = make_model("tiny", tied=request.param)
    return sh, wt, oracle_cfg(sh), O.weights_to_f64(wt), prompt_ids(sh)


def _compare_pass(t, fo, rows, tol=TOL_LOGITS):
    """logits / hidden of the last GPU pass against an oracle ForwardOut restricted to rows."""
    n_rows, _ = t.last_rows()
    assert n_rows == len(rows)
    lg = t.logits(0, n_rows)
    ref = fo.logits[rows]
    assert np.isfinite(lg).all()
    assert np.abs(lg - ref).max() <= tol
    for l in range(len(fo.hidden)):
        h = t.hidden(l, 0, n_rows)
        assert np.abs(h - fo.hidden[l][rows]).max() <= tol
    ids = t.argmax(0, n_rows)
    np.testing.assert_array_equal(ids, lg.argmax(-1))          # fused argmax == argmax of its own logits
    sure = top1_margin(ref) > MARGIN
    np.testing.assert_array_equal(ids[sure], ref.argmax(-1)[sure])
    return lg, ids


@pytest.mark.parametrize("impl", IMPLS)
def test_tiny_prefill_and_teacher_forced_steps(tiny, impl):
    sh, wt, cfg, w, prompt = tiny
    k = sh.k
    t = _gpu(sh, wt, impl)
    first = t.prefill(0, prompt, k)
    st, c, fo = O.prefill(cfg, w, prompt, k, return_forward=True)
    lg, ids = _compare_pass(t, fo, np.arange(len(prompt) + k))
    n = len(prompt)
    assert first == int(lg[n - 1].argmax())
    blk = t.get_block(0, k)
    assert blk == [int(lg[n - 1].argmax())] + [int(x) for x in lg[n + 1:n + k].argmax(-1)]
    # KV of the prompt
    for l in range(cfg.n_layers):
        from paper_2511_08923_b200 import bf16_bits_to_f32
        kk, vv = t.kv(0, l, 0, n)
        assert np.abs(bf16_bits_to_f32(kk) - st.k_cache[l]).max() <= TOL_LOGITS
        assert np.abs(bf16_bits_to_f32(vv) - st.v_cache[l]).max() <= TOL_LOGITS
    # decode steps, teacher-forced: the GPU gets the oracle's block before every step
    ar = O.ar_generate(cfg, w, prompt, 40)
    for s in range(6):
        e = st.n - n
        if s % 3 == 1:                       # perfect drafts -> L = k
            st.block[1:] = ar[e + 1:e + k]
        elif s % 3 == 2:                     # two right, then wrong
            st.block[1:] = ar[e + 1:e + k]
            st.block[3] = (st.block[3] + 1) % (sh.vocab - 1)
        t.set_block(0, st.block)
        block_before = st.block.copy()
        n_before = st.n
        so = O.step(cfg, w, st)
        toks, Ls = t.step([0])
        lg, ids = _compare_pass(t, so.fwd, np.arange(k * (k + 1)))
        # integer logic, bit-exact given the GPU's own argmax ids
        tg = ids[:k]
        L_ref = O.accept_length(block_before, tg)
        assert Ls[0] == L_ref
        assert toks[0] == [int(x) for x in block_before[1:L_ref]] + [int(tg[L_ref - 1])]
        nxt = O.select_next(L_ref, tg, ids[k:].reshape(k, k))
        assert t.get_block(0, k) == [int(x) for x in nxt]
        assert t.seq_len(0) == n_before + L_ref
        if (top1_margin(so.fwd.logits[:k]) > MARGIN).all():
            assert Ls[0] == so.L and toks[0] == so.emitted
        elif Ls[0] != so.L:                   # a low-margin row flipped: the two states part ways here
            break
    _close(t)


@pytest.mark.parametrize("impl", IMPLS)
def test_tiny_free_running_generation_matches_ar(tiny, impl):
    sh, wt, cfg, w, prompt = tiny
    k = sh.k
    ar = O.ar_generate(cfg, w, prompt, sh.max_new_tokens)
    t = _gpu(sh, wt, impl)
    out = [t.prefill(0, prompt, k)]
    Ls = []
    while len(out) < sh.max_new_tokens:
        toks, L = t.step([0])
        out.extend(toks[0]); Ls.append(L[0])
    out = out[:sh.max_new_tokens]
    # compare up to the first position where the oracle itself is not sure
    fo = O.causal_forward(cfg, w, list(prompt) + ar)
    m = top1_margin(fo.logits[len(prompt) - 1:len(prompt) - 1 + sh.max_new_tokens])
    unsure = np.nonzero(m <= MARGIN)[0]
    upto = int(unsure[0]) if len(unsure) else sh.max_new_tokens
    assert out[:upto] == ar[:upto]
    assert all(1 <= L <= k for L in Ls)
    assert t.seq_len(0) == len(prompt) + sum(Ls)
    _close(t)


def _drive_pattern(t, sh, prompt, k, first_block0, pattern):
    """Builds, slot by slot, a draft block whose draft i agrees (pattern[i-1]) or disagrees with
    the verified prediction given the slots before it, then runs the natural step on it."""
    block = [first_block0]
    for i in range(1, k):
        t.prefill(0, prompt, k)
        t.set_block(0, block + [sh.mask_token_id] * (k - len(block)))
        toks_i, _ = t.step([0], forced=[i])
        tgt = toks_i[0][-1]                          # verified prediction after i slots
        block.append(tgt if pattern[i - 1] else (tgt + 1) % (sh.vocab - 1))
    t.prefill(0, prompt, k)
    t.set_block(0, block)
    toks, L = t.step([0])
    expect = next((i for i, ok in enumerate(pattern) if not ok), k - 1) + 1
    assert L[0] == expect, (pattern, block)
    assert toks[0][:expect - 1] == block[1:expect]
    targets = t.argmax(0, k)                         # the step's own argmax ids of the causal slots
    assert L[0] == O.accept_length(block, targets) and toks[0][-1] == int(targets[expect - 1])
    return block, L[0]


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("k", [4, 8])
def test_acceptance_scan_all_patterns(tiny, impl, k):
    """Every agree/disagree pattern of the k-1 drafts, driven through the real step (k = 4 and 8)."""
    sh, wt, cfg, w, prompt = tiny
    t = _gpu(sh, wt, impl, k_max=k, debug=0)
    t.prefill(0, prompt, k)
    b0 = t.get_block(0, k)[0]
    for pattern in itertools.product([True, False], repeat=k - 1):
        _drive_pattern(t, sh, prompt, k, b0, pattern)
    _close(t)


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("k", [16, 32])
def test_acceptance_scan_wide_blocks(tiny, impl, k):
    """k = 16 and k = 32 (every lane of the verifying warp in use at 32): all drafts agree, the
    first disagrees, only the last disagrees, and a seeded sample of mixed patterns."""
    sh, wt, cfg, w, prompt = tiny
    t = _gpu(sh, wt, impl, k_max=k, debug=0, max_seq_len=256)
    t.prefill(0, prompt, k)
    b0 = t.get_block(0, k)[0]
    rng = np.random.default_rng(k)
    patterns = [tuple([True] * (k - 1)), tuple([False] + [True] * (k - 2)), tuple([True] * (k - 2) + [False]),
                tuple([True] * (k // 2) + [False] * (k - 1 - k // 2))]
    patterns += [tuple(bool(x) for x in rng.random(k - 1) < 0.85) for _ in range(4 if k == 16 else 2)]
    seen = set()
    for pattern in patterns:
        _, L = _drive_pattern(t, sh, prompt, k, b0, pattern)
        seen.add(L)
    assert k in seen and 1 in seen and (k - 1) in seen
    _close(t)


@pytest.mark.parametrize("impl", IMPLS)
def test_forced_acceptance_and_poisoned_eviction(tiny, impl):
    """Forced L commits exactly L slots; NaN-filling evicted slots changes nothing."""
    sh, wt, cfg, w, prompt = tiny
    k = sh.k
    runs = []
    for debug in (1, 3):
        t = _gpu(sh, wt, impl, debug=debug)
        t.prefill(0, prompt, k)
        rec = []
        for L in (1, 3, 2, 4, 1):
            toks, Ls = t.step([0], forced=[L])
            assert Ls == [L] and len(toks[0]) == L
            rec.append((toks[0], t.get_block(0, k), t.logits(0, k * (k + 1)).copy()))
        n = t.seq_len(0)
        assert n == len(prompt) + 11
        rec.append([t.kv(0, l, 0, n) for l in range(cfg.n_layers)])
        runs.append(rec)
        _close(t)
    for a, b in zip(runs[0][:-1], runs[1][:-1]):
        assert a[0] == b[0] and a[1] == b[1]
        np.testing.assert_array_equal(a[2], b[2])
    for (k0, v0), (k1, v1) in zip(runs[0][-1], runs[1][-1]):
        np.testing.assert_array_equal(k0, k1); np.testing.assert_array_equal(v0, v1)


@pytest.mark.parametrize("impl", IMPLS)
def test_committed_kv_is_exact_and_never_rewritten(tiny, impl):
    """The cache after decoding equals, bit for bit, what a fresh first pass over the
    final sequence writes for layer 0 (row-wise deterministic kernels), stays within
    tolerance of the oracle for every layer, and committed rows never change later."""
    from paper_2511_08923_b200 import bf16_bits_to_f32
    sh, wt, cfg, w, prompt = tiny
    k = sh.k
    t = _gpu(sh, wt, impl, debug=0)
    seq = list(prompt) + [t.prefill(0, prompt, k)]
    snaps = []
    for L in (2, 4, 1, 3):
        toks, _ = t.step([0], forced=[L])
        seq.extend(toks[0])
        n = t.seq_len(0)
        snaps.append((n, [t.kv(0, l, 0, n) for l in range(cfg.n_layers)]))
    n_final = t.seq_len(0)
    final = [t.kv(0, l, 0, n_final) for l in range(cfg.n_layers)]
    for n, kv in snaps:
        for l in range(cfg.n_layers):
            np.testing.assert_array_equal(kv[l][0], final[l][0][:n]); np.testing.assert_array_equal(kv[l][1], final[l][1][:n])
    ref = O.causal_forward(cfg, w, seq[:n_final])
    for l in range(cfg.n_layers):
        assert np.abs(bf16_bits_to_f32(final[l][0]) - ref.k_new[l]).max() <= TOL_LOGITS
        assert np.abs(bf16_bits_to_f32(final[l][1]) - ref.v_new[l]).max() <= TOL_LOGITS
    # replay: a first pass over the same tokens on a fresh sequence slot
    t2 = _gpu(sh, wt, impl, debug=0)
    t2.prefill(0, seq[:n_final], k)
    k0, v0 = t2.kv(0, 0, 0, n_final)
    np.testing.assert_array_equal(k0, final[0][0]); np.testing.assert_array_equal(v0, final[0][1])
    _close(t); _close(t2)


@pytest.mark.parametrize("impl", IMPLS)
def test_batched_step_equals_single_sequence_steps(impl):
    sh, wt = make_model("tiny", tied=False)
    k = sh.k
    prompts = [prompt_ids(sh, n, seed=s) for n, s in ((64, 0), (37, 5), (1, 6))]
    single = []
    for p in prompts:
        t = _gpu(sh, wt, impl, debug=0)
        out = [t.prefill(0, p, k)]
        for L in (2, 1, 4):
            out.extend(t.step([0], forced=[L])[0][0])
        single.append(out); _close(t)
    t = _gpu(sh, wt, impl, debug=0, max_batch=3)
    outs = [[t.prefill(i, p, k)] for i, p in enumerate(prompts)]
    for L in (2, 1, 4):
        toks, _ = t.step([0, 1, 2], forced=[L, L, L])
        for i in range(3):
            outs[i].extend(toks[i])
    assert outs == single
    _close(t)


@pytest.mark.parametrize("impl", IMPLS)
def test_errors_are_reported_before_launch(impl):
    from paper_2511_08923_b200 import TidarError
    sh, wt = make_model("tiny")
    t = _gpu(sh, wt, impl, debug=0, max_seq_len=80)
    with pytest.raises(TidarError) as e:
        t.step([0])
    assert e.value.code == -1
    with pytest.raises(TidarError) as e:
        t.prefill(0, prompt_ids(sh, 73), 4)             # 73 + 8 > 80
    assert e.value.code == -2
    t.prefill(0, prompt_ids(sh, 70), 4)
    t.step([0], forced=[2])
    with pytest.raises(TidarError) as e:                 # 72 + 8 = 80 fits, then 73.. does not
        t.step([0], forced=[1]); t.step([0], forced=[1])
    assert e.value.code == -2
    with pytest.raises(TidarError):
        t.prefill(0, [5000], 4)
    with pytest.raises(TidarError):
        t.step([0], forced=[9])
    _close(t)


@pytest.mark.parametrize("name,over", [
    # 2*d_ffn/128 = 151 weight tiles > 148 SMs: whole-wave tiles fused, leftover tiles K-split
    ("wide_ffn", dict(d_model=1024, n_q_heads=8, n_kv_heads=2, head_dim=128, d_ffn=9664, n_layers=1, vocab=1024)),
    # six query heads per KV head (the 1.5B-class grouping): 21 slots x 6 heads per attention tile
    ("group6", dict(d_model=768, n_q_heads=6, n_kv_heads=1, head_dim=128, d_ffn=1024, n_layers=2, vocab=2048)),
])
def test_other_shapes_prefill_and_steps(name, over):
    from dataclasses import replace
    from tidar_synth import CONFIGS, gen_model_weights
    sh = replace(CONFIGS["tiny"], name=name, tie_lm_head=False, k=8, **over)
    wt = gen_model_weights(sh)
    cfg, w = oracle_cfg(sh), O.weights_to_f64(wt)
    prompt = prompt_ids(sh, 70)
    k = sh.k
    t = _gpu(sh, wt, 0, max_seq_len=256)
    t.prefill(0, prompt, k)
    st, c, fo = O.prefill(cfg, w, prompt, k, return_forward=True)
    _compare_pass(t, fo, np.arange(len(prompt) + k))
    for s in range(2):
        t.set_block(0, st.block)
        so = O.step(cfg, w, st, forced=3)
        toks, Ls = t.step([0], forced=[3])
        _compare_pass(t, so.fwd, np.arange(k * (k + 1)))
        assert Ls == [3]
    _close(t)


@pytest.mark.parametrize("name", ["tiny", "1.5b", "8b"])
def test_graph_replay_plain_launches_and_replay_kernels_agree(name):
    """The benchmark times the captured-graph path with programmatic dependent launches; the
    logits / hidden-state comparisons run with plain launches.  The same teacher-forced steps
    through (a) graph replay, (b) plain launches and (c) the fp32 CUDA-core kernels must give
    identical acceptance lengths, tokens and next blocks, and (a) and (b) bit-identical cached
    K/V in every layer (same kernels, same order: a kernel that read its input before the
    previous kernel finished would show here)."""
    from dataclasses import replace
    if name == "tiny":
        sh, k, n_prompt = CONFIGS_["tiny"], 4, 64
    else:
        sh = replace(CONFIGS_[name].reduced(2), vocab=8192)          # the benchmark's widths, two layers, small head
        k, n_prompt = 16, 200
    wt = gen_model_weights_(sh)
    prompt = prompt_ids(sh, n_prompt)
    forced = [3, k, 1, k // 2, 2]
    runs = {}
    for tag, impl, debug in (("graph", 0, 0), ("plain", 0, 8), ("replay", 1, 0)):
        t = _gpu(sh, wt, impl, k_max=k, debug=debug, max_seq_len=n_prompt + 8 * k + 64)
        rec = [t.prefill(0, prompt, k)]
        blocks = [t.get_block(0, k)]
        for f in forced:
            if tag != "graph":
                t.set_block(0, runs["graph"]["blocks"][len(rec) - 1])          # teacher-forced from run (a)
            toks, L = t.step([0], forced=[f])
            rec.append((toks[0], L[0]))
            blocks.append(t.get_block(0, k))
        n = t.seq_len(0)
        kv = [t.kv(0, l, 0, n) for l in range(sh.n_layers)] if impl == 0 else None
        runs[tag] = {"rec": rec, "blocks": blocks, "kv": kv, "n": n, "launches": t.launch_count()}
        _close(t)
    assert runs["graph"]["rec"] == runs["plain"]["rec"] and runs["graph"]["blocks"] == runs["plain"]["blocks"]
    assert runs["graph"]["n"] == runs["plain"]["n"]
    for (k0, v0), (k1, v1) in zip(runs["graph"]["kv"], runs["plain"]["kv"]):
        np.testing.assert_array_equal(k0, k1); np.testing.assert_array_equal(v0, v1)
    # the CUDA-core kernels round differently: tokens can only differ on a near-tie, which the
    # tiny model's margins make rare; lengths are forced, so the shapes must match exactly
    assert [r[1] for r in runs["replay"]["rec"][1:]] == [r[1] for r in runs["graph"]["rec"][1:]]
    same = sum(a == b for a, b in zip(runs["replay"]["rec"], runs["graph"]["rec"]))
    assert same >= len(forced), (runs["replay"]["rec"], runs["graph"]["rec"])


@pytest.mark.parametrize("impl", IMPLS)
def test_device_timeout_status_is_reported_and_sequences_released(tiny, impl):
    """The status word a kernel sets when one of its bounded waits gives up reaches the caller as
    TIDAR_EDEVICE_TIMEOUT, and the sequences of the failed step must be prefilled again.  The word
    is set through a debug hook: no kernel is made to wait."""
    from paper_2511_08923_b200 import TidarError
    sh, wt, cfg, w, prompt = tiny
    k = sh.k
    t = _gpu(sh, wt, impl, debug=0)
    t.prefill(0, prompt, k)
    t.step([0], forced=[2])
    if impl != 0:                                   # the replay kernels have no bounded waits and no status word to read
        _close(t)
        return
    t.force_status(2)
    with pytest.raises(TidarError) as e:
        t.step([0], forced=[1])
    assert e.value.code == -5
    with pytest.raises(TidarError) as e:            # released: not prefilled any more
        t.step([0], forced=[1])
    assert e.value.code == -1
    first = t.prefill(0, prompt, k)                 # and usable again
    toks, L = t.step([0], forced=[2])
    assert L == [2]
    t.force_status(1)
    with pytest.raises(TidarError) as e:
        t.sync()
    assert e.value.code == -5
    t.sync()                                        # the word was cleared by the report
    # a real bounded wait that runs out: a barrier nothing arrives on, a limit of 2^14 polls
    t.wait_probe(1 << 14)
    with pytest.raises(TidarError) as e:
        t.sync()
    assert e.value.code == -5 and "status 9" in str(e.value)
    t.prefill(0, prompt, k)                         # the context is still usable
    assert t.step([0], forced=[1])[1] == [1]
    _close(t)


@pytest.mark.parametrize("impl", IMPLS)
def test_long_first_pass_in_one_chunk(tiny, impl):
    """prefill_rows: a 700-token prompt encoded in ONE pass of 704 rows (three row blocks of the
    projections, weight tiles shared between them; the LM head on the trailing rows only) against the
    oracle, and against the same prompt encoded in the default chunks of 256 rows."""
    from paper_2511_08923_b200 import bf16_bits_to_f32
    sh, wt, cfg, w, _ = tiny
    k = sh.k
    prompt = prompt_ids(sh, 700, seed=9)
    n = len(prompt)
    st, c, fo = O.prefill(cfg, w, prompt, k, return_forward=True)
    outs = []
    for rows in (768, 0):
        t = _gpu(sh, wt, impl, max_seq_len=1024, prefill_rows=rows)
        first = t.prefill(0, prompt, k)
        n_rows, row0 = t.last_rows()
        assert row0 + n_rows == n + k and row0 <= n - 1
        if rows:
            assert n_rows == 256 and row0 == n + k - 256          # logits for the trailing rows of the single chunk
        lg = t.logits(0, n_rows)
        assert np.abs(lg - fo.logits[row0:]).max() <= TOL_LOGITS
        for l in range(cfg.n_layers + 1):
            assert np.abs(t.hidden(l, 0, n_rows) - fo.hidden[l][row0:]).max() <= TOL_LOGITS
        ids = t.argmax(0, n_rows)
        np.testing.assert_array_equal(ids, lg.argmax(-1))
        assert first == int(lg[n - 1 - row0].argmax())
        assert t.get_block(0, k) == [first] + [int(x) for x in lg[n + 1 - row0:n + k - row0].argmax(-1)]
        kv = []
        for l in range(cfg.n_layers):
            kk, vv = t.kv(0, l, 0, n)
            assert np.abs(bf16_bits_to_f32(kk) - st.k_cache[l]).max() <= TOL_LOGITS
            assert np.abs(bf16_bits_to_f32(vv) - st.v_cache[l]).max() <= TOL_LOGITS
            kv.append((kk, vv))
        toks, L = t.step([0], forced=[2])
        outs.append((first, kv, toks, t.get_block(0, k)))
        _close(t)
    # layer 0's cache does not depend on how the prompt was cut into passes
    np.testing.assert_array_equal(outs[0][1][0][0], outs[1][1][0][0]); np.testing.assert_array_equal(outs[0][1][0][1], outs[1][1][0][1])
    if top1_margin(fo.logits[n - 1]) > MARGIN:
        assert outs[0][0] == outs[1][0] == c


def test_two_steps_in_flight_match_one_at_a_time():
    """tidar_step_async accepts a second step while the first is in flight (forced lengths): the results,
    handed out oldest first, the blocks and the cached K/V are bit-identical to the same steps run one at a
    time; a third step, a step without forced lengths behind one in flight, and every other entry point
    are refused until the queue is drained."""
    from paper_2511_08923_b200 import TidarError
    sh, wt = make_model("tiny", tied=False)
    k = sh.k
    prompts = [prompt_ids(sh, n=sh.prompt_len - 3 * q, seed=sh.seed + q) for q in range(2)]
    forced = [[2, 1], [k, 3], [1, 1], [3, k], [2, 2], [k, k], [1, 2]]
    runs = {}
    for tag in ("serial", "pipelined"):
        t = _gpu(sh, wt, 0, k_max=k, debug=0, max_batch=2, max_seq_len=256)     # diagnostics off: they allow one step in flight only
        for q, p in enumerate(prompts):
            t.prefill(q, p, k)
        res = []
        if tag == "serial":
            for f in forced:
                res.append(t.step([0, 1], forced=f))
        else:
            t.step_async([0, 1], forced[0])
            for f in forced[1:]:
                t.step_async([0, 1], f)
                if f is forced[1]:
                    with pytest.raises(TidarError):
                        t.step_async([0, 1], f)                   # a third step
                    with pytest.raises(TidarError):
                        t.prefill(0, prompts[0], k)               # anything else that touches sequences
                    assert t.seq_len(0) == len(prompts[0]) + forced[0][0] + forced[1][0]      # lengths advance when a step is enqueued
                res.append(t.step_wait())
            res.append(t.step_wait())
            with pytest.raises(TidarError):
                t.step_wait()                                     # nothing left in flight
            t.step_async([0, 1], [1, 1])
            with pytest.raises(TidarError):
                t.step([0, 1])                                    # unforced lengths cannot follow a step in flight
            t.step_wait()
            res.append(None)
        n = [t.seq_len(q) for q in range(2)]
        blocks = [t.get_block(q, k) for q in range(2)]
        upto = [len(prompts[q]) + sum(f[q] for f in forced) for q in range(2)]
        kv = [[t.kv(q, l, 0, upto[q]) for l in range(sh.n_layers)] for q in range(2)]
        runs[tag] = (res[:len(forced)], upto, kv, blocks if tag == "serial" else None)
        assert n[0] >= upto[0] and n[1] >= upto[1]
        _close(t)
    assert runs["serial"][0] == runs["pipelined"][0]
    for q in range(2):
        for (k0, v0), (k1, v1) in zip(runs["serial"][2][q], runs["pipelined"][2][q]):
            np.testing.assert_array_equal(k0, k1); np.testing.assert_array_equal(v0, v1)
