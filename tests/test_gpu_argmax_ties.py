"""Ties in the fused LM-head argmax: the lowest vocabulary id wins (needs a B200).

The LM head's running argmax is reduced across the 32 lanes of a warp, the four lane
quadrants of a weight tile, the tiles one CTA walks through, the CTAs, and finally the
merge kernel.  Duplicated LM-head rows give bit-identical logits at several ids, placed so
that each of those reduction levels has to break a tie: same lane group, another quadrant
of the same tile, another tile of the same CTA, another CTA, id 0 and the last id.
"""
from dataclasses import replace

import numpy as np
import pytest
import torch

from oracle import tidar_oracle as O
from tests.helpers import MARGIN, oracle_cfg, prompt_ids
from tidar_synth import CONFIGS, gen_model_weights, gen_normal_bf16, tensor_id

pytestmark = pytest.mark.gpu

N_SMS = 148            # the LM-head kernel runs one CTA per SM; CTA c walks tiles c, c + 148, ...
TILE = 128


def _model():
    sh = replace(CONFIGS["tiny"], name="ties", tie_lm_head=False, vocab=TILE * 300, k=4)
    wt = gen_model_weights(sh)
    lm = wt["lm_head"].clone()
    V, d = lm.shape
    groups = [
        # (ids that share one row vector), lowest id first
        [0, 1, 40, TILE * N_SMS + 5, TILE * 1 + 7, V - 1],              # id 0 ... the last id
        [3, 35, 64 + 3, TILE * 2 + 3],                                   # quadrants 0, 1, 2 of tile 0; another CTA
        [TILE * 150 + 65, TILE * 151 + 2, TILE * (150 + N_SMS) + 9],     # lowest id not in the first wave of tiles
    ]
    # One direction per group, built from the oracle's final hidden states (the untied LM head does
    # not feed back into them) so that the group is certain to hold the maximum of one chosen prompt
    # row: v = c * (y_r - mean y) with c set for a logit of 6 on row r, far above the other logits.
    cfg, w = oracle_cfg(sh), O.weights_to_f64(wt)
    _, _, fo = O.prefill(cfg, w, prompt_ids(sh, 40), sh.k, return_forward=True)
    y = O.rmsnorm(fo.hidden[-1], w["final_norm"], cfg.rms_eps)
    rows = []
    for r in (5, 17, 29):
        v = y[r] - y.mean(0)
        rows.append(torch.tensor(v * (6.0 / float(v @ y[r])), dtype=torch.float32).to(torch.bfloat16))
    for ids, v in zip(groups, rows):
        for i in ids:
            lm[i] = v
    wt["lm_head"] = lm
    return sh, wt, groups


@pytest.mark.parametrize("impl", [0, 1])
def test_lowest_id_wins_ties_at_every_reduction_level(impl):
    from paper_2511_08923_b200 import Tidar, pack_weights
    sh, wt, groups = _model()
    k = sh.k
    cfg, w = oracle_cfg(sh), O.weights_to_f64(wt)
    prompt = prompt_ids(sh, 40)
    t = Tidar(sh, pack_weights(wt, "cuda:0"), k_max=k, max_seq_len=256, debug=1, impl=impl)
    hit = set()

    def check(ref):
        n_rows, _ = t.last_rows()
        lg = t.logits(0, n_rows)
        ids = t.argmax(0, n_rows)
        # duplicated rows give bit-identical logits, so ties are real
        for g in groups:
            for i in g[1:]:
                np.testing.assert_array_equal(lg[:, g[0]], lg[:, i])
        np.testing.assert_array_equal(ids, lg.argmax(-1))             # np.argmax returns the first (lowest) maximum
        top = lg.max(-1)
        for r in range(n_rows):
            for g in groups:
                if lg[r, g[0]] == top[r]:
                    assert ids[r] == g[0]
                    hit.add(g[0])
        # the oracle (float64, ties to the lowest id as well) agrees wherever the winning VALUE is clear
        top_ref = ref.max(-1)
        runner = np.array([row[row < tv].max() for row, tv in zip(ref, top_ref)])
        sure = (top_ref - runner) > MARGIN
        np.testing.assert_array_equal(ids[sure], ref.argmax(-1)[sure])

    t.prefill(0, prompt, k)
    st, _, fo = O.prefill(cfg, w, prompt, k, return_forward=True)
    check(fo.logits)
    t.set_block(0, st.block)
    so = O.step(cfg, w, st)
    t.step([0])
    check(so.fwd.logits)
    assert len(hit) == len(groups), f"only the tie groups starting at {sorted(hit)} ever held a row maximum: widen the test"
    t.close()
