"""The long-context and multi-turn workloads at their full shapes (8B-class model, batches of
8 and 16, 30k / 8k-token histories) in scripted-target mode: every integer the loop produces
(match positions through their effect, drafts, accepted lengths, emitted tokens, lengths,
counters) must equal the oracle's model-free simulator.  The forward runs in full at these
sizes (block of B*(k+1) rows, attention over the whole cache); its numerics are checked
elsewhere against the oracle."""
import numpy as np
import pytest
import torch

from oracle import copyspec_oracle as O
from paper_2502_08923_b200 import binding as cs, inputs
from helpers import i32

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def weights8b():
    return inputs.make_weights(inputs.LLAMA8B, seed=0, device="cuda")


def _run(weights8b, cases, k, max_new, policy=cs.LATEST):
    cfg = inputs.LLAMA8B
    B = len(cases)
    n0 = max(len(h) for h, _ in cases)
    stride = (n0 + max_new + 67) // 4 * 4
    max_seq = n0 + max_new + k + 64
    ctx = cs.Context(cfg, weights8b, max_seq=max_seq, max_batch=B, k_max=k)
    kv = torch.zeros(cfg.n_layers, 2, B, cfg.n_kv_heads, max_seq, cfg.head_dim, dtype=torch.bfloat16, device="cuda")
    g = torch.Generator(device="cuda"); g.manual_seed(1)
    for layer in range(cfg.n_layers):      # synthetic context K/V, one layer at a time to bound memory
        kv[layer, :, :, :, :n0 - 1, :] = torch.randn(2, B, cfg.n_kv_heads, n0 - 1, cfg.head_dim, device="cuda",
                                                      generator=g).to(torch.bfloat16)
    h = np.zeros((B, stride), dtype=np.int32)
    lens = np.array([len(hh) for hh, _ in cases], dtype=np.int32)
    script = np.stack([s[:max_new] for _, s in cases]).astype(np.int32)
    for b, (hh, _) in enumerate(cases):
        h[b, :len(hh)] = hh
    hd, ld, kvl = i32(h), i32(lens), i32(lens - 1)
    st = ctx.cs_decode_loop(hd, ld, kv, kvl, 3, k, max_new, policy=policy, script=i32(script))
    tot = O.new_stats()
    taus = []
    for b, (hh, s) in enumerate(cases):
        steps, so, h_sim = O.scripted_simulator(hh, s, 3, k, policy, max_new)
        assert hd[b, :int(ld[b])].cpu().tolist() == h_sim, b
        assert int(kvl[b]) == int(ld[b]) - 1 == len(hh) + max_new - 1
        taus += [x["tau"] for x in steps if x["p0"] >= 0]
        for key in ("steps", "attempts", "accepted", "emitted", "no_match"):
            tot[key] += so[key]
        for i, v in enumerate(so["tau_hist"]):
            tot["tau_hist"][i] += v
    for key in ("steps", "attempts", "accepted", "emitted", "no_match"):
        assert st[key] == tot[key], key
    assert st["tau_hist"] == tot["tau_hist"]
    ctx.close()
    del kv
    torch.cuda.empty_cache()
    return st, taus


def test_long_context_copy_decode_batch8_k20(weights8b):
    """30,720-token Zipf contexts, scripted continuation with 60 % verbatim spans, k = 20."""
    cases = [inputs.long_context_case(100 + b) for b in range(8)]
    st, taus = _run(weights8b, cases, k=20, max_new=384)
    assert st["accepted"] > 0.3 * st["emitted"]          # copying carries a good share of the tokens
    assert max(taus) == 20


def test_multi_turn_batch16_k10(weights8b):
    """8,192-token histories whose first-turn answer is re-emitted with edits, batch 16, k = 10."""
    cases = [inputs.multi_turn_case(200 + b)[:2] for b in range(16)]
    st, taus = _run(weights8b, cases, k=10, max_new=384)
    assert st["accepted"] > 0.3 * st["emitted"]
    assert max(taus) == 10 and min(taus) == 0
