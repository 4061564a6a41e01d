"""Host-side checks of the C-ABI library: builds, loads, exports what the header declares."""
import ctypes as C
import os
import re

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
