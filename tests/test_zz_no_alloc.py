"""tidar_attention_static against tidar_attention (needs a B200).

tidar_attention_static serves hosts that hold device tensors but cannot allocate
device memory where they need attention (their pool belongs to another component, they
sit in a latency-critical loop, or they were handed buffers without an allocator): its
per-row table is a fixed array inside the library.  This file checks, through the C ABI,
that it gives what the arena-backed entry point gives, on two calls in a row (the second
with other shapes, so stale table entries of the first would show), that it rejects
oversized requests, and that it allocates nothing.  Collected last on purpose.
"""
from dataclasses import replace

import numpy as np
import pytest
import torch

from tidar_synth import CONFIGS, gen_model_weights, gen_normal_bf16, tensor_id

pytestmark = pytest.mark.gpu

TOL = 3e-2          # the tolerance of the attention parity tests


def _inputs(hd, Hq, Hkv, k, ns, seed, dev="cuda:0"):
    B, T, page = len(ns), k * (k + 1), 64
    pps = (max(ns) + k + page - 1) // page
    n_pages = B * pps + 2
    q = gen_normal_bf16(seed, tensor_id("q"), B * T * Hq * hd, 1.0).view(B * T, Hq, hd)
    kl = gen_normal_bf16(seed, tensor_id("k", 1), B * k * k * Hkv * hd, 1.0).view(B * k * k, Hkv, hd)
    vl = gen_normal_bf16(seed, tensor_id("v", 1), B * k * k * Hkv * hd, 1.0).view(B * k * k, Hkv, hd)
    kp = gen_normal_bf16(seed, tensor_id("k", 2), n_pages * Hkv * page * hd, 1.0).view(n_pages, Hkv, page, hd)
    vp = gen_normal_bf16(seed, tensor_id("v", 2), n_pages * Hkv * page * hd, 1.0).view(n_pages, Hkv, page, hd)
    perm = torch.randperm(n_pages, generator=torch.Generator().manual_seed(seed))
    pt = perm[:B * pps].view(B, pps).to(torch.int32)
    sl = torch.tensor(ns, dtype=torch.int32)
    return [x.to(dev) for x in (q, kp, vp, pt, sl, kl, vl)]


def test_static_table_attention_matches_arena_attention_twice():
    from paper_2511_08923_b200 import Tidar, attention_static, pack_weights
    hd, Hq, Hkv = 128, 8, 2
    sh = replace(CONFIGS["tiny"], head_dim=hd, n_q_heads=Hq, n_kv_heads=Hkv, n_layers=1, vocab=64, d_ffn=64, d_model=64)
    t = Tidar(sh, pack_weights(gen_model_weights(sh), "cuda:0"), k_max=8, max_batch=3, max_seq_len=512, impl=1)
    cases = [(8, [200, 5], 31), (4, [0, 63, 130], 32)]
    prepared = []
    for k, ns, seed in cases:                           # every buffer exists before the calls under test
        ins = _inputs(hd, Hq, Hkv, k, ns, seed)
        R = len(ns) * k * (k + 1)
        ref = torch.full((R, Hq * hd), float("nan"), dtype=torch.bfloat16, device="cuda:0")
        got = torch.full((R, Hq * hd), float("nan"), dtype=torch.bfloat16, device="cuda:0")
        prepared.append((k, ns, ins, ref, got))
    for k, ns, ins, ref, got in prepared:
        t.attention(*ins, ref, len(ns), k)
    torch.cuda.synchronize()
    before = torch.cuda.memory_allocated()
    for k, ns, ins, ref, got in prepared:               # two calls in a row, different shapes
        attention_static(*ins, got, len(ns), k, Hq, Hkv, hd)
    torch.cuda.synchronize()
    assert torch.cuda.memory_allocated() == before
    for k, ns, ins, ref, got in prepared:
        a, b = got.float().cpu().numpy(), ref.float().cpu().numpy()
        assert np.isfinite(a).all() and np.isfinite(b).all()
        assert np.abs(a - b).max() <= TOL
    t.close()


def test_static_table_attention_rejects_what_does_not_fit():
    from paper_2511_08923_b200 import TidarError, attention_static
    hd, Hq, Hkv, k = 64, 4, 2, 16
    ins = _inputs(hd, Hq, Hkv, 2, [3], 33)
    out = torch.zeros(8, dtype=torch.bfloat16, device="cuda:0")
    with pytest.raises(TidarError) as e:                # 17 * 272 rows > 4352: refused before any launch
        attention_static(*ins, out, 17, k, Hq, Hkv, hd)
    assert e.value.code == -2 and "4352" in str(e.value)
    with pytest.raises(TidarError) as e:
        attention_static(*ins, out, 1, 2, Hq, Hkv, 96)
    assert e.value.code == -1
    torch.cuda.synchronize()
    assert float(out.float().abs().sum()) == 0.0
