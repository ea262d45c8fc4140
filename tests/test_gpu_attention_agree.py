"""The three attention kernels (mma.sync, tcgen05 with query rows as M, tcgen05 with keys and head
dims as M) on the same seeded random shapes: batch 1-16, windows 0-60 (blocks cut into row groups
from 33 rows on), cache depths 1-5,000 with ragged lengths and ragged draft lengths.  Logits of the
live rows and the whole K/V cache must agree across the kernels; parity with the oracle is the
business of the other GPU tests, this one sweeps many more shapes than the oracle could."""
import numpy as np
import pytest
import torch

from paper_2502_08923_b200 import binding as cs, inputs
from helpers import i32

pytestmark = pytest.mark.gpu

CFG = inputs.ModelConfig(n_layers=2, d_model=256, n_heads=8, n_kv_heads=2, head_dim=128, d_ffn=512,
                         vocab=512, rope_theta=500000.0, rms_eps=1e-5)


@pytest.fixture(scope="module")
def weights():
    return inputs.weights_to(inputs.make_weights(CFG, seed=11, gain_jitter=0.05), "cuda")


@pytest.mark.parametrize("seed", [1, 2, 3])
def test_kernels_agree_on_random_shapes(weights, seed, monkeypatch):
    rng = np.random.default_rng(seed)
    done = 0
    while done < 16:
        B = int(rng.choice([1, 2, 3, 5, 8, 16]))
        k = int(rng.choice([0, 1, 5, 10, 20, 33, 60]))
        if B * (max(k, 1) + 1) > 256:                      # rows of a step
            continue
        kv_max = int(rng.choice([1, 100, 129, 700, 1500, 3000, 5000]))
        kv_lens = [kv_max] + [int(x) for x in rng.integers(1, kv_max + 1, size=B - 1)]
        draft_lens = [int(x) for x in rng.integers(0, k + 1, size=B)]
        max_seq = kv_max + k + 1 + int(rng.integers(1, 70))
        last = rng.integers(0, CFG.vocab, size=B)
        draft = rng.integers(0, CFG.vocab, size=(B, max(k, 1)))[:, :k]
        kv0 = inputs.synthetic_kv(CFG, B, max_seq, kv_max, seed=done, device="cuda")
        outs = {}
        for kern in ("mma", "tc", "tcw"):
            monkeypatch.setenv("CS_ATTN_KERNEL", kern)
            ctx = cs.Context(CFG, weights, max_seq=max_seq, max_batch=B, k_max=max(k, 1))
            kv, kvl = kv0.clone(), i32(kv_lens)
            logits = torch.full((B, k + 1, CFG.vocab), float("nan"), dtype=torch.float32, device="cuda")
            dr = i32(draft) if k > 0 else torch.zeros((B, 0), dtype=torch.int32, device="cuda")
            ctx.cs_verify_step(i32(last), dr, i32(draft_lens), kv, kvl, logits_dbg=logits)
            assert ctx.cs_sync_status() == 0, (kern, B, k, kv_lens, draft_lens)
            lg = logits.cpu().numpy()
            outs[kern] = ([lg[b, :draft_lens[b] + 1] for b in range(B)], kv.float().cpu().numpy())
            ctx.close()
        for kern in ("tc", "tcw"):
            for b in range(B):
                got, ref = outs[kern][0][b], outs["mma"][0][b]
                assert np.isfinite(got).all(), (kern, b, B, k, kv_lens, draft_lens)
                assert float(np.abs(got - ref).max()) < 5e-3, (kern, b, B, k, kv_lens, draft_lens)
            assert float(np.abs(outs[kern][1] - outs["mma"][1]).max()) < 5e-2, (kern, B, k, kv_lens, draft_lens)
        done += 1
