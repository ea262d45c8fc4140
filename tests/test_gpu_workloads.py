"""The long-context and multi-turn workloads at their full shapes (8B-class model, batches of
8 and 16, 30k / 8k-token histories) in scripted-target mode: every integer the loop produces
(match positions through their effect, drafts, accepted lengths, emitted tokens, lengths,
counters) must equal the oracle's model-free simulator.  The forward runs in full at these
sizes (block of B*(k+1) rows, attention over the whole cache).  Its numerics are checked here
on the first step, whose greedy tokens (computed by all 32 layers and the full LM head although
the script decides acceptance) are compared with the oracle's logits for one of the sequences;
element-wise logit and K/V parity at these block heights and cache depths is in
test_gpu_long_shapes.py."""
import numpy as np
import pytest
import torch

from oracle import copyspec_oracle as O
from paper_2502_08923_b200 import binding as cs, inputs
from helpers import argmax_consistent, i32

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
    # ---- first step on its own: the forward's greedy tokens against the oracle (last sequence;
    # the step only writes cache rows from position len - 1 on, so the context rows are read after it)
    model = O.Model(cfg, weights8b, contract=True, cache_weights=False)
    ctx.cs_loop_begin(hd, ld, kv, kvl, 3, k, max_new, policy=policy, script=i32(script))
    ctx.cs_loop_steps(1)
    mp, dl, al, ot, am = (t.numpy() for t in ctx.cs_loop_last_step())
    ctx.cs_loop_end()
    for b in (B - 1,):
        hh, n = cases[b][0], int(lens[b])
        p0 = O.find_match(hh, n, 3, policy)
        draft = O.gather_draft(hh, n, p0, 3, k)
        assert int(mp[b]) == p0 and int(dl[b]) == len(draft)
        cache = O.KVCache(cfg, 1, n + k, dtype=np.float32)
        for layer in range(cfg.n_layers):
            cache.a[layer, :, 0, :, :n - 1, :] = kv[layer, :, b, :, :n - 1, :].float().cpu().numpy()
        lg = model.forward_block([int(hh[-1])] + draft, n - 1, cache, 0)
        assert not argmax_consistent(lg, am[b, :len(draft) + 1].tolist()), b
        assert all(am[b, len(draft) + 1:] == -1)
        del cache
    # ---- the whole scripted run from the start
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
