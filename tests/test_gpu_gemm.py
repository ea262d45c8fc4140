"""The tensor-core projection kernel in isolation against the plain definition
Y = X W^T evaluated in fp64 on the CPU (building block of the forward of Sec. 3.2)."""
import numpy as np
import pytest
import torch

from paper_2502_08923_b200 import inputs
from helpers import make_pair

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    cfg = inputs.ModelConfig(n_layers=1, d_model=512, n_heads=4, n_kv_heads=4, head_dim=128, d_ffn=4096,
                             vocab=512, rope_theta=10000.0, rms_eps=1e-5)   # workspace large enough for the shapes below
    c, _ = make_pair(cfg, 256, 1, 10)
    yield c
    c.close()


@pytest.mark.parametrize("rows", [1, 11, 16, 17, 100, 176, 256])
@pytest.mark.parametrize("N,K", [(128, 64), (200, 256), (768, 256), (256, 1024), (4096, 4096), (1000, 520)])
def test_linear_matches_fp64_matmul(ctx, rows, N, K):
    g = torch.Generator().manual_seed(rows * 7919 + N + K)
    X = torch.randn(rows, K, generator=g).to(torch.bfloat16)
    W = (torch.randn(N, K, generator=g) * 0.05).to(torch.bfloat16)
    pad = (rows + 15) // 16 * 16
    Xd = torch.zeros(pad, K, dtype=torch.bfloat16, device="cuda")
    Xd[:rows] = X.cuda()
    Y = ctx.cs_linear(Xd, W.cuda(), rows=rows)
    assert ctx.cs_sync_status() == 0
    want = X.double().numpy() @ W.double().numpy().T
    got = Y.cpu().double().numpy()
    # bf16 products are exact in fp32; only the fp32 summation order differs
    tol = 1e-5 * np.sqrt(K) * max(1.0, np.abs(want).max())
    assert np.abs(got - want).max() <= tol


@pytest.mark.parametrize("rows", [1, 11, 40])
def test_lm_head_argmax_matches_fp64(rows):
    """LM-head stage alone: tile argmax in the GEMM epilogue + final reduction."""
    from helpers import argmax_consistent
    cfg = inputs.ModelConfig(n_layers=1, d_model=256, n_heads=8, n_kv_heads=8, head_dim=32, d_ffn=512,
                             vocab=5000, rope_theta=10000.0, rms_eps=1e-5)      # 5000 = 39 tiles + ragged tail
    c, _ = make_pair(cfg, 64, 4, 10, seed=3)
    g = torch.Generator().manual_seed(rows)
    X = torch.randn(rows, cfg.d_model, generator=g).to(torch.bfloat16)
    pad = (rows + 15) // 16 * 16
    Xd = torch.zeros(pad, cfg.d_model, dtype=torch.bfloat16, device="cuda")
    Xd[:rows] = X.cuda()
    logits = torch.zeros(rows, cfg.vocab, dtype=torch.float32, device="cuda")
    ids = c.cs_lm_head(Xd, rows=rows, logits_dbg=logits)
    assert c.cs_sync_status() == 0
    want = X.double().numpy() @ c.weights["lm_head"].cpu().double().numpy().T
    assert np.abs(logits.cpu().double().numpy() - want).max() <= 1e-4
    assert not argmax_consistent(want, ids.cpu().tolist(), tol=1e-4)
    ids2 = c.cs_lm_head(Xd, rows=rows)          # without the debug dump
    assert ids2.cpu().tolist() == ids.cpu().tolist()
    c.close()
