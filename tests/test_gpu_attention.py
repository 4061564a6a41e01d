"""Structured-mask paged attention alone vs the oracle's dense-mask attention (needs a B200)."""
from dataclasses import replace

import numpy as np
import pytest
import torch

from oracle import tidar_oracle as O
from tests.helpers import make_model
from tidar_synth import CONFIGS, gen_normal_bf16, tensor_id

pytestmark = pytest.mark.gpu

IMPLS = [0, 1]
TOL = 3e-2          # unit-variance bf16 inputs; bf16 output rounding alone is ~1e-2 at |x| ~ 3


def _ctx(hd, Hq, Hkv, k_max, max_batch, impl):
    from paper_2511_08923_b200 import Tidar, pack_weights
    sh = replace(CONFIGS["tiny"], head_dim=hd, n_q_heads=Hq, n_kv_heads=Hkv, n_layers=1, vocab=64, d_ffn=64, d_model=64)
    from tidar_synth import gen_model_weights
    return Tidar(sh, pack_weights(gen_model_weights(sh), "cuda:0"), k_max=k_max, max_batch=max_batch, max_seq_len=128,
                 impl=impl)


def _case(t, hd, Hq, Hkv, k, ns, seed):
    B, T, page = len(ns), k * (k + 1), 64
    pps = (max(ns) + k + page - 1) // page
    n_pages = B * pps + 3
    dev = "cuda:0"
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
    out = torch.full((B * T, Hq * hd), float("nan"), dtype=torch.bfloat16, device=dev)
    sl = torch.tensor(ns, dtype=torch.int32, device=dev)
    t.attention(q.to(dev), kp.to(dev), vp.to(dev), pt.to(dev), sl, kl.to(dev), vl.to(dev), out, B, k)
    torch.cuda.synchronize()
    got = out.float().cpu().numpy().reshape(B * T, Hq, hd)
    ref = np.concatenate(refs)
    assert np.isfinite(got).all()
    assert np.abs(got - ref).max() <= TOL


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("hd,Hq,Hkv", [(64, 4, 2), (128, 8, 2), (128, 4, 4)])
def test_attention_small_lengths(impl, hd, Hq, Hkv):
    t = _ctx(hd, Hq, Hkv, 8, 3, impl)
    # prefix lengths around page boundaries, n = 0 included (first token of a sequence)
    _case(t, hd, Hq, Hkv, 4, [0, 1, 63], 11)
    _case(t, hd, Hq, Hkv, 4, [64, 65, 127], 12)
    _case(t, hd, Hq, Hkv, 8, [200, 5], 13)
    _case(t, hd, Hq, Hkv, 1, [9], 14)
    _case(t, hd, Hq, Hkv, 3, [700], 15)
    t.close()


@pytest.mark.parametrize("impl", IMPLS)
def test_attention_k16_long_prefix(impl):
    t = _ctx(128, 8, 2, 16, 1, impl)
    _case(t, 128, 8, 2, 16, [1500], 21)
    t.close()


def _case_sampled(t, hd, Hq, Hkv, k, n, seed, n_rows=24):
    """Config-2 sizes: the kernel runs on all rows, the oracle on a sample of query rows
    (each with its own dense-mask row), which covers every kind of slot and both ends."""
    T, page = k * (k + 1), 64
    pps = (n + k + page - 1) // page
    dev = "cuda:0"
    q = gen_normal_bf16(seed, tensor_id("q"), T * Hq * hd, 1.0).view(T, Hq, hd)
    kl = gen_normal_bf16(seed, tensor_id("k", 1), k * k * Hkv * hd, 1.0).view(k * k, Hkv, hd)
    vl = gen_normal_bf16(seed, tensor_id("v", 1), k * k * Hkv * hd, 1.0).view(k * k, Hkv, hd)
    kc = gen_normal_bf16(seed, tensor_id("k", 2), pps * page * Hkv * hd, 1.0).view(pps * page, Hkv, hd)
    vc = gen_normal_bf16(seed, tensor_id("v", 2), pps * page * Hkv * hd, 1.0).view(pps * page, Hkv, hd)
    perm = torch.randperm(pps + 5, generator=torch.Generator().manual_seed(seed))[:pps]
    kp = torch.zeros(pps + 5, Hkv, page, hd, dtype=torch.bfloat16)
    vp = torch.zeros(pps + 5, Hkv, page, hd, dtype=torch.bfloat16)
    kp[perm] = kc.view(pps, page, Hkv, hd).permute(0, 2, 1, 3)
    vp[perm] = vc.view(pps, page, Hkv, hd).permute(0, 2, 1, 3)
    out = torch.full((T, Hq * hd), float("nan"), dtype=torch.bfloat16, device=dev)
    t.attention(q.to(dev), kp.to(dev), vp.to(dev), perm.view(1, pps).to(torch.int32).to(dev),
                torch.tensor([n], dtype=torch.int32, device=dev), kl.to(dev), vl.to(dev), out, 1, k)
    torch.cuda.synchronize()
    got = out.float().cpu().numpy().reshape(T, Hq, hd)
    assert np.isfinite(got).all()
    rows = np.unique(np.concatenate([[0, k - 1, k, T - 1], np.random.default_rng(seed).integers(0, T, n_rows)]))
    mask = O.build_decode_mask(n, k)[rows]
    k_all = torch.cat([kc[:n + k], kl]).double().numpy()
    v_all = torch.cat([vc[:n + k], vl]).double().numpy()
    ref = O.masked_attention(q[rows].double().numpy(), k_all, v_all, mask)
    assert np.abs(got[rows] - ref).max() <= TOL


@pytest.mark.parametrize("n", [1024, 4096, 16384, 32768])
def test_attention_microbench_sizes_sampled_rows(n):
    """32 query / 8 KV heads, head_dim 128, k = 16: the stand-alone attention workload."""
    from paper_2511_08923_b200 import Tidar, pack_weights
    from tidar_synth import gen_model_weights
    sh = replace(CONFIGS["tiny"], head_dim=128, n_q_heads=32, n_kv_heads=8, n_layers=1, vocab=64, d_ffn=64, d_model=64)
    t = Tidar(sh, pack_weights(gen_model_weights(sh), "cuda:0"), k_max=16, max_batch=1, max_seq_len=128, impl=0)
    _case_sampled(t, 128, 32, 8, 16, n, 40 + n % 97)
    t.close()
