"""Parity at the benchmark's sizes (needs a B200 and a host with tens of GB of RAM).

The 1.5B-class model runs at full depth and full vocabulary: one first pass over the
512-token prompt and one decode step (k = 16, 272 slots), in the launch configuration the
benchmark times.  The 8B-class model runs at full depth as well (36 layers, full
vocabulary): a first pass over a 128-token prompt and one decode step.  The oracle computes
every hidden state but only a sample of LM-head rows (151936-wide logits for hundreds of
rows would not fit a test); for the 8B-class model its weights are handed to it one layer
at a time, generated on demand, so that the host holds one layer in float64 and not 36.

Every comparison is per row (3e-2 x max(1, max |reference row|)) and in rms (2.5 % of the
reference's rms); the measured errors are printed and written to
gpurun_out/fullsize_errors.json when that folder exists.
"""
import json
import os

import numpy as np
import pytest
import torch  # noqa: F401

from oracle import tidar_oracle as O
from tests.helpers import MARGIN, RMS_REL, check_rows, depth_tol, oracle_cfg, prompt_ids, top1_margin
from tidar_synth import CONFIGS, gen_model_weights, lazy_model_weights

pytestmark = pytest.mark.gpu


def _oracle_weights(sh, wt, lazy):
    """float64 weights for the oracle: everything at once (from the tensors the GPU got), or the final
    norm now, embedding and head upcast where they are read, and the layers on demand."""
    return lazy_model_weights(sh, "cuda:0") if lazy else O.weights_to_f64(wt)


# How the tolerances are set (measured on a B200; see the error table these tests print).
#
# Against the oracle with bf16-STORED activations (act_dtype = "bf16": the oracle rounds at the same
# places as the kernels, all arithmetic float64) a single stage agrees almost exactly: the K/V a layer
# caches to 1e-4 rms (a rounding flips where fp32 and float64 sums straddle a bf16 boundary), a layer
# without attention to 2e-4, the tensor-core attention to 2e-3 (its probability operand is bf16).
# That is the sharp check, and it is applied to the first layer: cached K/V(0) and hidden(1).
#
# It cannot be carried through the depth: once the two sides differ by a fraction of a bf16 ulp
# their later roundings decorrelate (one FFN turns a 4e-4 difference into 2.5e-3), so after a few
# layers each side carries its own rounding noise whatever the oracle emulates.  That noise is a
# random walk over the layers whose step depends on the model's activation statistics (sharper
# attention and wider FFNs in the 8B-class model: 0.78 % per layer against 0.35 %).  At depth the
# float64 oracle is therefore compared with a bound calibrated on the model's own first layer:
# rms error after l layers <= 1.5 x (rms error after one layer) x sqrt(l), the per-row bound of
# check_rows scaled alike; the first-layer error itself must stay under 1.2 %.
FIRST_LAYER_RMS_MAX = 0.012
BF16_KV_RMS_MAX, BF16_HIDDEN1_RMS_MAX = 5e-4, 7e-3


def _run(sh, n_prompt=None, n_sample=12, lazy=False, tag=""):
    report = {}
    try:
        _run_checks(sh, n_prompt, n_sample, lazy, tag, report)
    finally:                                       # the measured errors are kept whatever the outcome
        for what, v in report.items():
            print(f"{what}: max |err| {v['max_abs']:.4f} (reference max {v['max_ref']:.2f}), rms err / rms ref {v['rms_rel']:.4f}, "
                  f"worst row at {v['worst_row_err_over_tol']:.2f} of its bound")
        out_dir = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "gpurun_out")
        if os.path.isdir(out_dir):
            path = os.path.join(out_dir, "fullsize_errors.json")
            prev = json.load(open(path)) if os.path.exists(path) else {}
            prev.update(report)
            json.dump(prev, open(path, "w"), indent=1)


def _depth_bounds(sigma1, l):
    """(rms bound, row-bound factor) after l layers, from the first-layer rms error sigma1."""
    rms = max(RMS_REL, 1.5 * sigma1 * np.sqrt(max(l, 1)))
    return dict(rms_rel_max=rms, row_factor=rms / RMS_REL)


def _run_checks(sh, n_prompt, n_sample, lazy, tag, report):
    from dataclasses import replace
    from paper_2511_08923_b200 import Tidar, pack_weights, bf16_bits_to_f32
    k = sh.k
    prompt = prompt_ids(sh, n_prompt)
    n = len(prompt)
    T = k * (k + 1)
    wt = gen_model_weights(sh, device="cuda:0")
    t = Tidar(sh, pack_weights(wt, "cuda:0"), k_max=k, max_seq_len=n + 8 * k, debug=1, impl=0, guard_bytes=64 * 1024)
    w = _oracle_weights(sh, wt, lazy)
    del wt
    L = sh.n_layers
    layers_checked = sorted({0, 1, L // 2, L})
    cfg = oracle_cfg(sh)
    # ---- first pass on the GPU ----
    first = t.prefill(0, prompt, k)
    # the first pass runs in chunks of the context's row capacity; the read-back calls see the last chunk
    n_rows, row0 = t.last_rows()
    assert row0 + n_rows == n + k and row0 <= n - 1
    rows = np.unique(np.concatenate([np.arange(n - 1, n + k), np.random.default_rng(0).integers(row0, n, n_sample)]))
    g_hidden = {l: t.hidden(l, 0, n_rows) for l in layers_checked}
    g_logits = np.stack([t.logits(int(r) - row0, 1)[0] for r in rows])
    g_argmax = t.argmax(0, n_rows)
    g_kv = {l: t.kv(0, l, 0, n) for l in (0, L - 1)}
    ids = np.concatenate([prompt, np.full(k, sh.mask_token_id, dtype=np.int64)])
    pos = np.arange(n + k, dtype=np.int64)
    kc, vc = O._empty_cache(cfg)
    # ---- the sharp check: first layer against the oracle that stores its activations in bf16 ----
    if not lazy:
        cfg1 = replace(cfg, n_layers=1, act_dtype="bf16")
        w1 = dict(w); w1["layers"] = w["layers"][:1]
        f1 = O.forward(cfg1, w1, ids, pos, O.build_prefill_mask(n, k), kc[:1], vc[:1], logit_rows=np.array([], dtype=np.int64))
        kk, vv = g_kv[0]
        check_rows(bf16_bits_to_f32(kk).reshape(n, -1), f1.k_new[0][:n].reshape(n, -1), f"{tag}[bf16 oracle] cached K(0)", report,
                   rms_rel_max=BF16_KV_RMS_MAX, row_factor=0.2)
        check_rows(bf16_bits_to_f32(vv).reshape(n, -1), f1.v_new[0][:n].reshape(n, -1), f"{tag}[bf16 oracle] cached V(0)", report,
                   rms_rel_max=BF16_KV_RMS_MAX, row_factor=0.2)
        check_rows(g_hidden[1], f1.hidden[1][row0:], f"{tag}[bf16 oracle] prefill hidden(1)", report, rms_rel_max=BF16_HIDDEN1_RMS_MAX, row_factor=0.5)
        del f1
    # ---- the whole depth against the float64 definition ----
    fo = O.forward(cfg, w, ids, pos, O.build_prefill_mask(n, k), kc, vc, logit_rows=rows)
    _, sigma1 = check_rows(g_hidden[1], fo.hidden[1][row0:], f"{tag}prefill hidden(1)", report, rms_rel_max=FIRST_LAYER_RMS_MAX)
    for l in layers_checked:
        if l != 1:
            check_rows(g_hidden[l], fo.hidden[l][row0:], f"{tag}prefill hidden({l})", report, **_depth_bounds(sigma1, l))
    check_rows(g_logits, fo.logits[rows], f"{tag}prefill logits", report, **_depth_bounds(sigma1, L + 1))
    for r in rows:
        if top1_margin(fo.logits[r]) > max(MARGIN, 2 * depth_tol(fo.logits[r])):
            assert int(g_argmax[int(r) - row0]) == int(fo.logits[r].argmax())
    for l, (kk, vv) in g_kv.items():
        check_rows(bf16_bits_to_f32(kk).reshape(n, -1), fo.k_new[l][:n].reshape(n, -1), f"{tag}cached K({l})", report, **_depth_bounds(sigma1, l + 1))
        check_rows(bf16_bits_to_f32(vv).reshape(n, -1), fo.v_new[l][:n].reshape(n, -1), f"{tag}cached V({l})", report, **_depth_bounds(sigma1, l + 1))
    a = fo.logits[n - 1]
    if top1_margin(a) > max(MARGIN, 2 * depth_tol(a)):
        assert first == int(a.argmax())
    block = np.empty(k, dtype=np.int64)
    block[0] = int(a.argmax()); block[1:] = fo.logits[n + 1:n + k].argmax(-1)
    kc, vc = [x[:n].copy() for x in fo.k_new], [x[:n].copy() for x in fo.v_new]
    del fo
    # ---- one decode step, teacher-forced from the oracle's state ----
    t.set_block(0, block)
    toks, Ls = t.step([0])
    srows = np.unique(np.concatenate([np.arange(k), np.random.default_rng(1).integers(k, T, n_sample)]))
    g_hidden = {l: t.hidden(l, 0, T) for l in layers_checked}
    g_logits = np.stack([t.logits(int(r), 1)[0] for r in srows])
    gpu_ids = t.argmax(0, T)
    L_ref = O.accept_length(block, gpu_ids[:k])
    assert Ls[0] == L_ref and toks[0] == [int(x) for x in block[1:L_ref]] + [int(gpu_ids[L_ref - 1])]
    nxt = O.select_next(L_ref, gpu_ids[:k], gpu_ids[k:].reshape(k, k))
    assert t.get_block(0, k) == [int(x) for x in nxt]
    assert t.arena_guard_intact()
    t.close()
    _, _, _, spos = O.slot_layout(n, k)
    sids = np.concatenate([block, np.full(k * k, sh.mask_token_id, dtype=np.int64)])
    so = O.forward(cfg, w, sids, spos, O.build_decode_mask(n, k), kc, vc, logit_rows=srows)
    _, sigma1 = check_rows(g_hidden[1], so.hidden[1], f"{tag}step hidden(1)", report, rms_rel_max=FIRST_LAYER_RMS_MAX)
    for l in layers_checked:
        if l != 1:
            check_rows(g_hidden[l], so.hidden[l], f"{tag}step hidden({l})", report, **_depth_bounds(sigma1, l))
    check_rows(g_logits, so.logits[srows], f"{tag}step logits", report, **_depth_bounds(sigma1, L + 1))
    if (top1_margin(so.logits[:k]) > max(MARGIN, 2 * depth_tol(so.logits[:k]))).all():
        assert L_ref == O.accept_length(block, so.logits[:k].argmax(-1))


def test_1p5b_class_full_depth_prefill_and_step():
    _run(CONFIGS["1.5b"], tag="1.5b ")


def test_8b_class_widths_two_layer_twin():
    _run(CONFIGS["8b"].reduced(2), tag="8b-L2 ")


def test_8b_class_full_depth_prefill_and_step():
    """The benchmark's own model (36 layers, full vocabulary), short prompt: the oracle takes the
    layers one at a time (about two minutes of float64 NumPy on the host)."""
    _run(CONFIGS["8b"], n_prompt=128, n_sample=6, lazy=True, tag="8b ")
