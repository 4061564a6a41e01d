"""Weight-streaming projection kernel vs the float64 definition (needs a B200)."""
from dataclasses import replace

import numpy as np
import pytest
import torch

from tidar_synth import CONFIGS, gen_model_weights, gen_normal_bf16, tensor_id

pytestmark = pytest.mark.gpu

# bf16 x bf16 products are exact in fp32; what is left is the fp32 accumulation order.
# |out| ~ 0.02 * sqrt(K) <= 2.5, K <= 12288 terms.
TOL = 2e-3


@pytest.fixture(scope="module")
def ctx():
    from paper_2511_08923_b200 import Tidar, pack_weights
    sh = CONFIGS["tiny"]
    t = Tidar(sh, pack_weights(gen_model_weights(sh), "cuda:0"), k_max=16, max_batch=8, max_seq_len=128, impl=0)
    yield t
    t.close()


def _run(t, R, N, K, splits, seed):
    A = gen_normal_bf16(seed, tensor_id("q"), R * K, 1.0).view(R, K)
    W = gen_normal_bf16(seed, tensor_id("wq"), N * K, 0.02).view(N, K)
    ref = A.double().numpy() @ W.double().numpy().T
    out = torch.full((R, N), float("nan"), dtype=torch.float32, device="cuda:0")
    guard = torch.full((4096,), 7.0, dtype=torch.float32, device="cuda:0")      # allocated right after out
    t.gemm(A.cuda(), W.cuda(), out, splits)
    t.sync()
    got = out.cpu().numpy()
    assert np.isfinite(got).all()
    assert np.abs(got - ref).max() <= TOL
    assert bool((guard == 7.0).all())
    return got


@pytest.mark.parametrize("R,N,K", [
    (20, 512, 256),        # tiny model, one decode step
    (68, 1408, 256),       # tiny model prefill rows, N = 11 tiles
    (1, 256, 704),         # a single row, K = 11 blocks
    (72, 1100, 1536),      # k = 8 slots, ragged N tail
    (272, 1536, 8960),     # k = 16 slots (two MMA halves), 1.5B-class down projection
    (272, 2176, 4096),     # 8B-class width
    (300, 640, 512),       # two row blocks
    (601, 200, 1024),      # three row blocks, ragged everything
])
def test_gemm_matches_definition(ctx, R, N, K):
    a = _run(ctx, R, N, K, 0, 100 + R)
    b = _run(ctx, R, N, K, 1, 100 + R)
    kb = K // 64
    c = _run(ctx, R, N, K, min(3, kb), 100 + R)
    # a fixed summation order: repeated runs agree bit for bit
    np.testing.assert_array_equal(a, _run(ctx, R, N, K, 0, 100 + R))
    assert np.abs(b - c).max() <= TOL


def test_gemm_rejects_bad_arguments(ctx):
    from paper_2511_08923_b200 import TidarError
    A = torch.zeros(4, 100, dtype=torch.bfloat16, device="cuda:0")
    W = torch.zeros(8, 100, dtype=torch.bfloat16, device="cuda:0")
    out = torch.zeros(4, 8, dtype=torch.float32, device="cuda:0")
    with pytest.raises(TidarError) as e:
        ctx.gemm(A, W, out)                       # K not a multiple of 64
    assert e.value.code == -1
    A = torch.zeros(4, 128, dtype=torch.bfloat16, device="cuda:0")
    W = torch.zeros(8, 128, dtype=torch.bfloat16, device="cuda:0")
    with pytest.raises(TidarError):
        ctx.gemm(A, W, out, splits=99)
