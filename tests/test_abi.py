"""Host-side checks of the C-ABI library: builds, loads, exports what the header declares."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from paper_2511_08923_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    names = set()
    inc = os.path.join(ROOT, "include")
    for f in os.listdir(inc):
        if f.endswith(".h"):
            src = open(os.path.join(inc, f)).read()
            src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
            names |= set(re.findall(r"\b(tidar_[a-z0-9_]+)\s*\(", src))
    return sorted(names)


def test_library_builds_and_exports_every_declared_symbol():
    path = build.build()
    assert os.path.exists(path)
    lib = C.CDLL(path)
    names = _declared()
    assert {"tidar_init", "tidar_prefill", "tidar_step", "tidar_free"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} declared in include/*.h but not exported"


def _cfg(**over):
    base = dict(n_layers=2, d_model=256, n_q_heads=4, n_kv_heads=2, head_dim=64, d_ffn=704, vocab=1024, tie_lm_head=1,
                rms_eps=1e-6, rope_theta=1e4, mask_token_id=1023, k_max=4, max_batch=1, max_seq_len=256, page_size=64,
                beta=1.0, temperature=0.0, sample_seed=0, debug=0, impl=1, prefill_rows=0)
    base.update(over)
    return binding.tidar_config(**base)


def test_arena_bytes_and_validation_run_on_the_host():
    lib = binding.load()
    n = C.c_size_t(0)
    assert lib.tidar_arena_bytes(C.byref(_cfg()), C.byref(n)) == 0
    small = n.value
    assert small > 2 * 2 * 4 * 64 * 2 * 64 * 2          # at least the KV pages
    assert lib.tidar_arena_bytes(C.byref(_cfg(debug=1)), C.byref(n)) == 0
    assert n.value > small
    for bad in (dict(head_dim=96), dict(page_size=32), dict(k_max=0), dict(k_max=33), dict(n_q_heads=3),
                dict(mask_token_id=5000), dict(beta=1.5), dict(beta=-0.1), dict(temperature=-1.0), dict(d_model=100),
                dict(max_seq_len=8), dict(n_q_heads=0, n_kv_heads=1), dict(n_q_heads=256, n_kv_heads=1),
                dict(d_model=12352)):
        assert lib.tidar_arena_bytes(C.byref(_cfg(**bad)), C.byref(n)) == -1, bad
        assert lib.tidar_last_error(None)


def test_init_without_gpu_fails_loudly():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    lib = binding.load()
    w = binding.tidar_weights()
    ctx = C.c_void_p()
    rc = lib.tidar_init(C.byref(_cfg()), C.byref(w), C.c_void_p(256), C.c_size_t(1 << 30), None, C.byref(ctx))
    assert rc == -4 and b"no CUDA device" in lib.tidar_last_error(None)


def test_block_length_plan_is_optimal_under_the_row_budget():
    """tidar_plan_ks (host only) against brute force: among all length vectors within the caps whose
    slots sum_i k_i (k_i + 1) fit the budget, the plan has the largest sum of lengths; infeasible budgets
    give all ones; the plan never exceeds a cap."""
    import itertools
    from paper_2511_08923_b200 import TidarError, plan_ks
    rng = np.random.default_rng(5)
    for trial in range(60):
        n = int(rng.integers(1, 5)); k_max = int(rng.integers(1, 7))
        want = [int(x) for x in rng.integers(1, 9, size=n)] if trial % 2 else None
        budget = int(rng.integers(1, 120))
        ks = plan_ks(n, k_max, budget, want)
        caps = [min(k_max, w) for w in want] if want else [k_max] * n
        assert all(1 <= k <= c for k, c in zip(ks, caps))
        feasible = [v for v in itertools.product(*[range(1, c + 1) for c in caps]) if sum(k * (k + 1) for k in v) <= budget]
        if not feasible:
            assert ks == [1] * n
        else:
            assert sum(k * (k + 1) for k in ks) <= budget
            assert sum(ks) == max(sum(v) for v in feasible), (n, k_max, budget, want, ks)
            assert max(ks) - min(k for k, c in zip(ks, caps) if k < c or k == max(ks)) <= 1      # blocks that may still grow stay level
    assert plan_ks(1, 16) == [16] and plan_ks(8, 16) == [6] * 4 + [5] * 4 and plan_ks(32, 16) == [3] * 16 + [2] * 16      # the default budget of 288 slots, used in full
    assert plan_ks(3, 16, 288, [2, 16, 16]) == [2, 11, 11]                                            # 6 + 132 + 132 = 270 <= 288 < 270 + 24
    for bad in [(0, 4, 10, None), (2, 0, 10, None), (2, 4, 10, [1, 0])]:
        with pytest.raises(TidarError):
            plan_ks(*bad)
