"""Pins for the oracle's masks and slot layout (CPU only)."""
import os

import numpy as np
import pytest

from oracle import tidar_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _read_mask(name):
    rows = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            rows.append([c == "1" for c in line.replace(" ", "")])
    return np.array(rows, dtype=bool)


def test_slot_count_matches_paper_footnote():
    # Section 3.3 footnote: q_len = block_len * (1 + block_len)
    assert [O.n_slots(k) for k in (3, 4, 8, 16)] == [12, 20, 72, 272]


def test_decode_mask_worked_example_shape_and_rows():
    m = O.build_decode_mask(3, 3)
    assert m.shape == (12, 15)                      # (q_len, q_len + prefix)
    np.testing.assert_array_equal(m, _read_mask("decode_mask_k3_n3.txt"))


def test_prefill_mask_example():
    m = O.build_prefill_mask(4, 3)
    assert m.shape == (7, 7)                        # (prompt + block)^2
    np.testing.assert_array_equal(m, _read_mask("prefill_mask_k3_n4.txt"))


@pytest.mark.parametrize("k", [1, 2, 4, 8, 16])
@pytest.mark.parametrize("n", [0, 1, 5, 64])
def test_decode_mask_invariants(n, k):
    m = O.build_decode_mask(n, k)
    T = k * (k + 1)
    assert m.shape == (T, n + T)
    kind, blk, idx, pos = O.slot_layout(n, k)
    # every row sees the whole committed prefix
    assert m[:, :n].all()
    loc = m[:, n:]
    # causal rows: exactly the causal slots up to themselves, never a mask slot
    for j in range(k):
        assert loc[j, :k].tolist() == [c <= j for c in range(k)]
        assert not loc[j, k:].any()
        assert m[j].sum() == n + j + 1
    # mask rows: causal 0..b, own block, nothing else
    for b in range(k):
        for i in range(k):
            r = k + b * k + i
            assert loc[r, :k].tolist() == [c <= b for c in range(k)]
            own = np.zeros(k * k, dtype=bool)
            own[b * k:(b + 1) * k] = True
            np.testing.assert_array_equal(loc[r, k:], own)
            assert m[r].sum() == n + (b + 1) + k
    # of the (k+1)^2 local k x k tiles exactly 2k+1 are non-empty
    nonempty = 0
    for tr in range(k + 1):
        for tc in range(k + 1):
            nonempty += loc[tr * k:(tr + 1) * k, tc * k:(tc + 1) * k].any()
    assert nonempty == 2 * k + 1
    # positions: causal j at n+j; mask (b,i) at n+b+1+i, i.e. block b starts at the
    # position causal slot b predicts (no label shift)
    assert pos[:k].tolist() == [n + j for j in range(k)]
    for b in range(k):
        assert pos[k + b * k] == pos[b] + 1
        assert pos[k + b * k:k + (b + 1) * k].tolist() == list(range(n + b + 1, n + b + 1 + k))
    # a visible key is never at a later position than the row unless it is in the
    # row's own bidirectional block
    for r in range(T):
        for c in range(T):
            if loc[r, c] and not (kind[r] == 1 and kind[c] == 1 and blk[r] == blk[c]):
                assert pos[c] <= pos[r]


@pytest.mark.parametrize("n,k", [(1, 1), (3, 3), (17, 4), (64, 16)])
def test_prefill_mask_invariants(n, k):
    m = O.build_prefill_mask(n, k)
    assert m.shape == (n + k, n + k)
    np.testing.assert_array_equal(m[:n, :n], np.tril(np.ones((n, n), dtype=bool)))
    assert not m[:n, n:].any()
    assert m[n:, :].all()


def test_prefill_mask_is_block_zero_of_a_decode_step():
    # The mask rows of a first pass over n tokens see what block L-1 of a decode
    # step sees after L accepted slots: all committed tokens plus their own block.
    n, k, L = 7, 4, 3
    dm = O.build_decode_mask(n, k)
    rows = dm[k + (L - 1) * k: k + L * k]
    seen_committed = rows[:, :n + L]                   # cache + causal 0..L-1
    assert seen_committed.all()
    assert not rows[:, n + L:n + k].any()              # later causal slots invisible
    pm = O.build_prefill_mask(n + L, k)
    assert pm[n + L:, :n + L].all() and pm[n + L:, n + L:].all()
