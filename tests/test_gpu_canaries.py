"""Write canaries (host-checked, no sanitizer needed): a step may only write the K/V rows of the
block it verifies (App. B.2: the block's keys and values are appended at positions kv_len ..
kv_len + draft_len) and its own workspace.  The cache lives inside a larger buffer with guard
bands, every cache byte outside the appended rows is compared with a copy taken before the call,
and the binding keeps guard bands around the workspace.  Shapes cover the three attention
kernels, short and tall GEMM launch shapes, ragged batches, sequences without a draft, the
generation loop and prefill."""
import numpy as np
import pytest
import torch

from paper_2502_08923_b200 import binding as cs, inputs
from helpers import PATTERN, assert_only_rows_written, guarded_kv, i32

pytestmark = pytest.mark.gpu

WIDE = inputs.ModelConfig(n_layers=2, d_model=512, n_heads=8, n_kv_heads=4, head_dim=128, d_ffn=1024,
                          vocab=1024, rope_theta=500000.0, rms_eps=1e-5)



@pytest.mark.parametrize("kernel", ["tc", "tcw", "default"])
@pytest.mark.parametrize("B,k,kv_max", [(1, 10, 700), (3, 10, 650), (16, 10, 900), (2, 40, 1100)])
def test_verify_step_writes_only_the_block_rows(kernel, B, k, kv_max, monkeypatch):
    if kernel != "default":
        monkeypatch.setenv("CS_ATTN_KERNEL", kernel)
    cfg = WIDE
    rng = np.random.default_rng(B * 100 + k)
    max_seq = kv_max + k + 1 + 37
    w = inputs.weights_to(inputs.make_weights(cfg, seed=5, gain_jitter=0.05), "cuda")
    ctx = cs.Context(cfg, w, max_seq=max_seq, max_batch=B, k_max=k)
    kv_lens = [kv_max] + [int(x) for x in rng.integers(kv_max // 2, kv_max + 1, size=B - 1)]
    draft_lens = [k] + [int(x) for x in rng.integers(0, k + 1, size=B - 1)]
    if B > 2:
        draft_lens[-1] = 0                                # a sequence without a draft: one row
    buf, kv = guarded_kv(cfg, B, max_seq, kv_max, seed=B)
    before = kv.clone()
    kvl = i32(kv_lens)
    ctx.cs_verify_step(i32(rng.integers(0, cfg.vocab, size=B)), i32(rng.integers(0, cfg.vocab, size=(B, k))),
                       i32(draft_lens), kv, kvl)
    assert ctx.cs_sync_status() == 0
    assert_only_rows_written(buf, kv, before, [(kv_lens[b], draft_lens[b] + 1) for b in range(B)])
    assert ctx.workspace_guards_intact()
    ctx.close()


@pytest.mark.parametrize("cfg", [inputs.TINY, inputs.ModelConfig(n_layers=2, d_model=256, n_heads=4, n_kv_heads=2, head_dim=64,
                                                                 d_ffn=512, vocab=512, rope_theta=10000.0, rms_eps=1e-5)],
                         ids=["head32-or-tiny", "head64"])
def test_verify_step_other_head_sizes(cfg):
    """The mma.sync attention path of the small configurations."""
    B, k, kv_max = 4, 7, 300
    rng = np.random.default_rng(3)
    max_seq = kv_max + k + 1 + 11
    w = inputs.weights_to(inputs.make_weights(cfg, seed=6, gain_jitter=0.05), "cuda")
    ctx = cs.Context(cfg, w, max_seq=max_seq, max_batch=B, k_max=k)
    kv_lens = [kv_max, 1, 129, 200]
    draft_lens = [k, 0, 3, k]
    buf, kv = guarded_kv(cfg, B, max_seq, kv_max, seed=2)
    before = kv.clone()
    kvl = i32(kv_lens)
    ctx.cs_verify_step(i32(rng.integers(0, cfg.vocab, size=B)), i32(rng.integers(0, cfg.vocab, size=(B, k))),
                       i32(draft_lens), kv, kvl)
    assert ctx.cs_sync_status() == 0
    assert_only_rows_written(buf, kv, before, [(kv_lens[b], draft_lens[b] + 1) for b in range(B)])
    assert ctx.workspace_guards_intact()
    ctx.close()


def test_loop_steps_and_prefill_write_only_their_rows():
    """Five loop steps (step graph, cached tiles requested early) after a prefill into a guarded cache."""
    cfg, B, k, gamma = WIDE, 4, 10, 3
    rng = np.random.default_rng(9)
    n0 = [600, 411, 257, 600]
    max_new = 6 * (k + 1)
    stride = (max(n0) + max_new + 67) // 4 * 4
    max_seq = max(n0) + max_new + k + 64
    w = inputs.weights_to(inputs.make_weights(cfg, seed=7, gain_jitter=0.05), "cuda")
    ctx = cs.Context(cfg, w, max_seq=max_seq, max_batch=B, k_max=k)
    h = np.zeros((B, stride), dtype=np.int32)
    for b in range(B):
        hh = rng.integers(0, cfg.vocab, size=n0[b], dtype=np.int32)
        src = int(rng.integers(n0[b] // 4, n0[b] // 2))
        hh[n0[b] - gamma:] = hh[src:src + gamma]           # the last gamma tokens repeat an earlier place
        h[b, :n0[b]] = hh
    buf, kv = guarded_kv(cfg, B, max_seq, 0, seed=0)
    hd, ld = i32(h), i32(n0)
    kvl = torch.zeros(B, dtype=torch.int32, device="cuda")
    before = kv.clone()
    ctx.cs_prefill(hd, ld, max(n0), kv, kvl)
    assert ctx.cs_sync_status() == 0
    assert kvl.cpu().tolist() == [n - 1 for n in n0]
    assert_only_rows_written(buf, kv, before, [(0, n - 1) for n in n0])
    before = kv.clone()
    ctx.cs_loop_begin(hd, ld, kv, kvl, gamma, k, max_new)
    ctx.cs_loop_steps(5)
    ctx.cs_loop_poll()
    ctx.cs_loop_end()
    assert ctx.cs_sync_status() == 0
    # a step writes the block's rows; rows past the accepted prefix are overwritten by later steps.
    # All writes lie between the old cache length and the new one plus one block.
    new_len = kvl.cpu().tolist()
    assert_only_rows_written(buf, kv, before, [(n0[b] - 1, new_len[b] - (n0[b] - 1) + k + 1) for b in range(B)])
    assert all(new_len[b] > n0[b] - 1 for b in range(B))
    assert ctx.workspace_guards_intact()
    ctx.close()
