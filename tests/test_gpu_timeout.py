"""A bounded wait that runs out (every mbarrier wait of the TMA / MMA pipelines has a time limit
with a drain path behind it): the limit is shortened to 2 ms for this context and the producer
of one small GEMM launch leaves out one K block, so the tensor-core warp waits for a tile that
never arrives.  Nothing faults or hangs: the CTA records the timeout, lets its other copies
land, frees its tensor memory and returns; the host reads CS_ERR_TIMEOUT and the context goes
on working."""
import numpy as np
import pytest
import torch

from paper_2502_08923_b200 import binding as cs, inputs
from helpers import make_pair

pytestmark = pytest.mark.gpu


def _operands(rows, N, K, seed):
    g = torch.Generator().manual_seed(seed)
    X = torch.randn(rows, K, generator=g).to(torch.bfloat16)
    W = (torch.randn(N, K, generator=g) * 0.05).to(torch.bfloat16)
    Xd = torch.zeros((rows + 15) // 16 * 16, K, dtype=torch.bfloat16, device="cuda")
    Xd[:rows] = X.cuda()
    return X, W, Xd, W.cuda()


def test_wait_runs_out_and_the_context_stays_usable(monkeypatch):
    monkeypatch.setenv("CS_WAIT_LIMIT_US", "2000")
    cfg = inputs.ModelConfig(n_layers=1, d_model=256, n_heads=2, n_kv_heads=2, head_dim=128, d_ffn=512, vocab=512,
                             rope_theta=10000.0, rms_eps=1e-5)
    ctx, _ = make_pair(cfg, 256, 1, 10)
    rows, N, K = 8, 128, 256                 # one CTA, four K blocks, no split-K cluster
    X, W, Xd, Wd = _operands(rows, N, K, 1)
    want = X.double().numpy() @ W.double().numpy().T
    tol = 1e-5 * np.sqrt(K) * max(1.0, np.abs(want).max())
    assert np.abs(ctx.cs_linear(Xd, Wd, rows=rows).cpu().double().numpy() - want).max() <= tol
    assert ctx.cs_sync_status() == cs.CS_OK
    # K block 2 never arrives
    ctx.cs_debug_drop_tile(2)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    Y = ctx.cs_linear(Xd, Wd, rows=rows)
    ev1.record()
    assert ctx.cs_sync_status() == cs.CS_ERR_TIMEOUT
    assert 1.0 <= ev0.elapsed_time(ev1) <= 500.0          # waited about the limit, not 2 s, and returned
    assert float(Y.abs().max()) == 0.0                     # a CTA that gave up stores zeros, never partial sums
    assert ctx.cs_sync_status() == cs.CS_OK                # the status was reported once and cleared
    # the hook covered one launch; the same context computes correctly afterwards
    for seed in (2, 3):
        X, W, Xd, Wd = _operands(rows, N, K, seed)
        want = X.double().numpy() @ W.double().numpy().T
        assert np.abs(ctx.cs_linear(Xd, Wd, rows=rows).cpu().double().numpy() - want).max() <= tol
    assert ctx.cs_sync_status() == cs.CS_OK
    # the hook refuses launches that split K over a cluster (the cluster barrier has no time limit)
    X, W, Xd, Wd = _operands(rows, 256, 4096, 4)
    ctx.cs_debug_drop_tile(1)
    with pytest.raises(cs.CsError) as err:
        ctx.cs_linear(Xd, Wd, rows=rows)
    assert err.value.code == cs.CS_ERR_UNSUPPORTED
    want = X.double().numpy() @ W.double().numpy().T
    got = ctx.cs_linear(Xd, Wd, rows=rows).cpu().double().numpy()
    assert np.abs(got - want).max() <= 1e-5 * np.sqrt(4096) * max(1.0, np.abs(want).max())
    ctx.close()
