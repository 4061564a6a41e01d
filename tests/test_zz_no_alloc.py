"""tidar_attention_static against the oracle and against tidar_attention (needs a B200).

tidar_attention_static serves hosts that hold device tensors but cannot allocate
device memory where they need attention (their pool belongs to another component, they
must stay out of the allocator, or they were handed buffers without one): its per-row
table is a fixed array inside the library.  This file checks, through the C ABI, on two
calls in a row (the second with other shapes, so stale table entries of the first would
show), that its output matches the oracle's dense-mask attention and what the arena-backed
entry point gives with the tensor-core kernel; that it rejects what it cannot run; and that
neither torch's allocator nor the driver's free-memory figure moves across the calls.
Collected last on purpose.
"""
from dataclasses import replace

import numpy as np
import pytest
import torch

from oracle import tidar_oracle as O
from tidar_synth import CONFIGS, gen_model_weights, gen_normal_bf16, tensor_id

pytestmark = pytest.mark.gpu

TOL = 3e-2          # the tolerance of the attention parity tests


def _inputs(hd, Hq, Hkv, k, ns, seed, dev="cuda:0"):
    """Seeded q / local K,V / cached K,V in shuffled pages, and the oracle's result for them."""
    B, T, page = len(ns), k * (k + 1), 64
    pps = (max(ns) + k + page - 1) // page
    n_pages = B * pps + 2
    q = gen_normal_bf16(seed, tensor_id("q"), B * T * Hq * hd, 1.0).view(B * T, Hq, hd)
    kl = gen_normal_bf16(seed, tensor_id("k", 1), B * k * k * Hkv * hd, 1.0).view(B * k * k, Hkv, hd)
    vl = gen_normal_bf16(seed, tensor_id("v", 1), B * k * k * Hkv * hd, 1.0).view(B * k * k, Hkv, hd)
    kp = torch.zeros(n_pages, Hkv, page, hd, dtype=torch.bfloat16)
    vp = torch.zeros(n_pages, Hkv, page, hd, dtype=torch.bfloat16)
    perm = torch.randperm(n_pages, generator=torch.Generator().manual_seed(seed))
    pt = perm[:B * pps].view(B, pps).to(torch.int32)
    refs = []
    for s, n in enumerate(ns):
        kc = gen_normal_bf16(seed, tensor_id("k", 2 + s), (n + k) * Hkv * hd, 1.0).view(n + k, Hkv, hd)
        vc = gen_normal_bf16(seed, tensor_id("v", 2 + s), (n + k) * Hkv * hd, 1.0).view(n + k, Hkv, hd)
        for p in range(n + k):
            kp[pt[s, p // page], :, p % page] = kc[p]
            vp[pt[s, p // page], :, p % page] = vc[p]
        k_all = torch.cat([kc, kl[s * k * k:(s + 1) * k * k]]).double().numpy()
        v_all = torch.cat([vc, vl[s * k * k:(s + 1) * k * k]]).double().numpy()
        refs.append(O.masked_attention(q[s * T:(s + 1) * T].double().numpy(), k_all, v_all, O.build_decode_mask(n, k)))
    sl = torch.tensor(ns, dtype=torch.int32)
    return [x.to(dev) for x in (q, kp, vp, pt, sl, kl, vl)], np.concatenate(refs).reshape(B * T, Hq * hd)


def test_static_table_attention_matches_oracle_and_arena_attention_twice():
    from paper_2511_08923_b200 import Tidar, attention_static, pack_weights
    hd, Hq, Hkv = 128, 8, 2
    sh = replace(CONFIGS["tiny"], head_dim=hd, n_q_heads=Hq, n_kv_heads=Hkv, n_layers=1, vocab=64, d_ffn=64, d_model=64)
    t = Tidar(sh, pack_weights(gen_model_weights(sh), "cuda:0"), k_max=8, max_batch=3, max_seq_len=512, impl=0)
    cases = [(8, [200, 5], 31), (4, [0, 63, 130], 32)]
    prepared = []
    for k, ns, seed in cases:                           # every buffer exists before the calls under test
        ins, ref = _inputs(hd, Hq, Hkv, k, ns, seed)
        R = len(ns) * k * (k + 1)
        arena_out = torch.full((R, Hq * hd), float("nan"), dtype=torch.bfloat16, device="cuda:0")
        got = torch.full((R, Hq * hd), float("nan"), dtype=torch.bfloat16, device="cuda:0")
        prepared.append((k, ns, ins, ref, arena_out, got))
    for k, ns, ins, ref, arena_out, got in prepared:    # the existing entry point, tensor-core kernel
        t.attention(*ins, arena_out, len(ns), k)
    k, ns, ins, ref, arena_out, got = prepared[0]
    attention_static(*ins, got, len(ns), k, Hq, Hkv, hd)        # warm-up: resolves the table's address on this device
    torch.cuda.synchronize()
    got.fill_(float("nan"))
    torch.cuda.synchronize()
    torch_before = torch.cuda.memory_allocated()
    free_before, _ = torch.cuda.mem_get_info()
    for k, ns, ins, ref, arena_out, got in prepared:    # two calls in a row, different shapes
        attention_static(*ins, got, len(ns), k, Hq, Hkv, hd)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert torch.cuda.memory_allocated() == torch_before
    assert free_after == free_before, "device free memory moved across tidar_attention_static calls"
    for k, ns, ins, ref, arena_out, got in prepared:
        a, b = got.float().cpu().numpy(), arena_out.float().cpu().numpy()
        assert np.isfinite(a).all() and np.isfinite(b).all()
        assert np.abs(a - ref).max() <= TOL             # the oracle's dense-mask attention
        assert np.abs(a - b).max() <= TOL               # the arena-backed entry point
    t.close()


def test_static_table_attention_rejects_what_it_cannot_run():
    from paper_2511_08923_b200 import TidarError, attention_static
    hd, Hq, Hkv, k = 64, 4, 2, 16
    ins, _ = _inputs(hd, Hq, Hkv, 2, [3], 33)
    out = torch.zeros(6 * Hq * hd + 8, dtype=torch.bfloat16, device="cuda:0")
    with pytest.raises(TidarError) as e:                # 17 * 272 rows > 4352: refused before any launch
        attention_static(*ins, out, 17, k, Hq, Hkv, hd)
    assert e.value.code == -2 and "4352" in str(e.value)
    with pytest.raises(TidarError) as e:
        attention_static(*ins, out, 1, 2, Hq, Hkv, 96)
    assert e.value.code == -1
    with pytest.raises(TidarError) as e:                # output not 16-byte aligned
        attention_static(*ins, out[1:], 1, 2, Hq, Hkv, hd)
    assert e.value.code == -1 and "aligned" in str(e.value)
    q, kp, vp, pt, sl, kl, vl = ins
    with pytest.raises(TidarError) as e:                # K pages not 16-byte aligned
        attention_static(q, kp.view(-1)[1:], vp, pt, sl, kl, vl, out, 1, 2, Hq, Hkv, hd)
    assert e.value.code == -1
    torch.cuda.synchronize()
    assert float(out.float().abs().sum()) == 0.0


def test_static_table_attention_clamps_lengths_and_skips_pages_outside_the_pool():
    """A length beyond what the page table backs is clamped, a page index outside the pool
    contributes nothing: the call stays inside the caller's buffers and returns finite values."""
    from paper_2511_08923_b200 import attention_static
    hd, Hq, Hkv, k = 64, 4, 2, 2
    ins, ref = _inputs(hd, Hq, Hkv, k, [70], 34)
    q, kp, vp, pt, sl, kl, vl = ins
    R = k * (k + 1)
    out = torch.full((R, Hq * hd), float("nan"), dtype=torch.bfloat16, device="cuda:0")
    big = torch.tensor([10 ** 6], dtype=torch.int32, device="cuda:0")
    attention_static(q, kp, vp, pt, big, kl, vl, out, 1, k, Hq, Hkv, hd)
    torch.cuda.synchronize()
    assert np.isfinite(out.float().cpu().numpy()).all()
    bad_pt = pt.clone(); bad_pt[0, 0] = 10 ** 6          # first page of the prefix is not in the pool
    attention_static(q, kp, vp, bad_pt, sl, kl, vl, out, 1, k, Hq, Hkv, hd)
    torch.cuda.synchronize()
    got = out.float().cpu().numpy()
    assert np.isfinite(got).all()
    # the same result as attention over the prefix without its first 64 positions
    pages = pt[0].cpu().numpy()
    n = 70
    kc = torch.stack([kp[int(pages[p // 64]), :, p % 64] for p in range(64, n + k)]).double().cpu().numpy()
    vc = torch.stack([vp[int(pages[p // 64]), :, p % 64] for p in range(64, n + k)]).double().cpu().numpy()
    k_all = np.concatenate([kc, kl.double().cpu().numpy()]); v_all = np.concatenate([vc, vl.double().cpu().numpy()])
    mask = O.build_decode_mask(n, k)[:, 64:]
    want = O.masked_attention(q.double().cpu().numpy(), k_all, v_all, mask).reshape(R, Hq * hd)
    assert np.abs(got - want).max() <= TOL
