"""Parity at the benchmark's sizes (needs a B200 and a host with tens of GB of RAM).

The 1.5B-class model runs at full depth and full vocabulary: one first pass over the
512-token prompt and one decode step (k = 16, 272 slots), in the launch configuration the
benchmark times.  The oracle computes every hidden state but only a sample of LM-head rows
(151936-wide logits for 528 rows would not fit a test).  The 8B-class widths run as a
2-layer twin with the full vocabulary, for the same reason.
"""
import numpy as np
import pytest
import torch  # noqa: F401

from oracle import tidar_oracle as O
from tests.helpers import MARGIN, TOL_LOGITS, depth_tol, oracle_cfg, prompt_ids, top1_margin
from tidar_synth import CONFIGS, gen_model_weights

pytestmark = pytest.mark.gpu


def _run(sh, n_sample=12):
    from paper_2511_08923_b200 import Tidar, pack_weights
    k = sh.k
    wt = gen_model_weights(sh)
    cfg, w = oracle_cfg(sh), O.weights_to_f64(wt)
    prompt = prompt_ids(sh)
    n = len(prompt)
    t = Tidar(sh, pack_weights(wt, "cuda:0"), k_max=k, max_seq_len=n + 8 * k, debug=1, impl=0)
    del wt
    # ---- first pass ----
    first = t.prefill(0, prompt, k)
    # the first pass runs in chunks of the context's row capacity; the read-back calls see the last chunk
    n_rows, row0 = t.last_rows()
    assert row0 + n_rows == n + k and row0 <= n - 1
    ids = np.concatenate([prompt, np.full(k, cfg.mask_token_id, dtype=np.int64)])
    rows = np.unique(np.concatenate([np.arange(n - 1, n + k), np.random.default_rng(0).integers(row0, n, n_sample)]))
    kc, vc = O._empty_cache(cfg)
    fo = O.forward(cfg, w, ids, np.arange(n + k, dtype=np.int64), O.build_prefill_mask(n, k), kc, vc, logit_rows=rows)
    for l in (0, cfg.n_layers // 2, cfg.n_layers):
        assert np.abs(t.hidden(l, 0, n_rows) - fo.hidden[l][row0:]).max() <= depth_tol(fo.hidden[l][row0:])
    for r in rows:
        lg = t.logits(int(r) - row0, 1)[0]
        assert np.abs(lg - fo.logits[r]).max() <= depth_tol(fo.logits[r])
        if top1_margin(fo.logits[r]) > max(MARGIN, 2 * depth_tol(fo.logits[r])):
            assert int(t.argmax(int(r) - row0, 1)[0]) == int(fo.logits[r].argmax())
    # cached K/V of the whole prompt (first chunk included), first and last layer
    from paper_2511_08923_b200 import bf16_bits_to_f32
    for l in (0, cfg.n_layers - 1):
        kk, vv = t.kv(0, l, 0, n)
        assert np.abs(bf16_bits_to_f32(kk) - fo.k_new[l][:n]).max() <= depth_tol(fo.k_new[l][:n])
        assert np.abs(bf16_bits_to_f32(vv) - fo.v_new[l][:n]).max() <= depth_tol(fo.v_new[l][:n])
    a = fo.logits[n - 1]
    if top1_margin(a) > max(MARGIN, 2 * depth_tol(a)):
        assert first == int(a.argmax())
    # ---- one decode step, teacher-forced from the oracle's state ----
    block = np.empty(k, dtype=np.int64)
    block[0] = int(a.argmax()); block[1:] = fo.logits[n + 1:n + k].argmax(-1)
    st = O.OracleState(n=n, k_cache=[x[:n].copy() for x in fo.k_new], v_cache=[x[:n].copy() for x in fo.v_new], block=block)
    t.set_block(0, block)
    T = k * (k + 1)
    _, _, _, pos = O.slot_layout(n, k)
    sids = np.concatenate([block, np.full(k * k, cfg.mask_token_id, dtype=np.int64)])
    srows = np.unique(np.concatenate([np.arange(k), np.random.default_rng(1).integers(k, T, n_sample)]))
    so = O.forward(cfg, w, sids, pos, O.build_decode_mask(n, k), st.k_cache, st.v_cache, logit_rows=srows)
    toks, Ls = t.step([0])
    for l in (0, cfg.n_layers // 2, cfg.n_layers):
        assert np.abs(t.hidden(l, 0, T) - so.hidden[l]).max() <= depth_tol(so.hidden[l])
    for r in srows:
        assert np.abs(t.logits(int(r), 1)[0] - so.logits[r]).max() <= depth_tol(so.logits[r])
    gpu_ids = t.argmax(0, T)
    L_ref = O.accept_length(block, gpu_ids[:k])
    assert Ls[0] == L_ref and toks[0] == [int(x) for x in block[1:L_ref]] + [int(gpu_ids[L_ref - 1])]
    if (top1_margin(so.logits[:k]) > max(MARGIN, 2 * depth_tol(so.logits[:k]))).all():
        assert L_ref == O.accept_length(block, so.logits[:k].argmax(-1))
    t.close()


def test_1p5b_class_full_depth_prefill_and_step():
    _run(CONFIGS["1.5b"])


def test_8b_class_widths_two_layer_twin():
    _run(CONFIGS["8b"].reduced(2))
