"""cs_decode_loop on the GPU against the oracle loop, greedy decoding and the model-free
simulator (App. B.3 steps 1, 2, 4; Sec. 3.2)."""
import numpy as np
import pytest
import torch

from oracle import copyspec_oracle as O
from paper_2502_08923_b200 import binding as cs, inputs
from helpers import COUNTERS, LOGIT_TOL, counters_for_streams, greedy_margins, i32, make_pair

pytestmark = pytest.mark.gpu


def _run_gpu(ctx, hists, lens, stride, gamma, k, max_new, policy, script=None, eos_id=-1):
    B = len(hists)
    h = np.zeros((B, stride), dtype=np.int32)
    for b in range(B):
        h[b, :lens[b]] = hists[b][:lens[b]]
    hd, ld = i32(h), i32(lens)
    kv = ctx.alloc_kv()
    kv_len = torch.zeros(ctx.max_batch, dtype=torch.int32, device="cuda")[:B].contiguous()
    ctx.cs_prefill(hd, ld, int(max(lens)), kv, kv_len)
    st = ctx.cs_decode_loop(hd, ld, kv, kv_len, gamma, k, max_new, policy=policy, eos_id=eos_id,
                            script=None if script is None else i32(script))
    return hd.cpu().numpy(), ld.cpu().numpy(), kv_len.cpu().numpy(), st


@pytest.mark.parametrize("policy", [cs.LATEST, cs.FIRST])
def test_tiny_config_scripted_mode(policy):
    """Small configuration: 512-token context with planted spans, gamma=3, k=10, scripted target."""
    cfg = inputs.TINY
    ctx, model = make_pair(cfg, 1024, 1, 10)
    ctxt, spans = inputs.tiny_context(seed=1)
    rng = np.random.default_rng(7)
    max_new = 200
    script = inputs.copy_script(rng, ctxt, max_new, 0.6, 5, 30, cfg.vocab, zipf_s=None)
    h, n, kvl, st = _run_gpu(ctx, [ctxt], [512], 1024, 3, 10, max_new, policy, script=script[None, :])
    steps, st_o, h_sim = O.scripted_simulator(ctxt, script, 3, 10, policy, max_new)
    assert n[0] == 512 + max_new and kvl[0] == n[0] - 1
    assert h[0, :n[0]].tolist() == h_sim
    for key in ("steps", "attempts", "accepted", "emitted", "no_match"):
        assert st[key] == st_o[key], key
    assert st["tau_hist"][:11] == st_o["tau_hist"][:11]
    assert st["accepted"] > 0 and len({s["tau"] for s in steps}) >= 5     # tau covers a spread of values
    ctx.close()


def test_tiny_config_real_mode_is_greedy_decoding():
    """64 decode steps in real mode; the emitted tokens equal the oracle's copy loop and
    plain greedy decoding (losslessness, Sec. 1 / App. B.2)."""
    cfg = inputs.TINY
    ctx, model = make_pair(cfg, 1024, 1, 10)
    ctxt, _ = inputs.tiny_context(seed=1)
    max_new = 64
    h, n, kvl, st = _run_gpu(ctx, [ctxt], [512], 1024, 3, 10, max_new, cs.LATEST)
    cache = O.KVCache(cfg, 1, 1024)
    model.prefill(ctxt.tolist(), cache, 0)
    h_o = ctxt.tolist()
    trace = []
    got_o, st_o = O.decode_loop(model, cache, 0, h_o, 3, 10, O.LATEST, max_new, trace=trace)
    gpu_tokens = h[0, 512:n[0]].tolist()
    # every emitted token is the oracle's greedy choice, or within the logit tolerance of it
    assert max(greedy_margins(model, cfg, ctxt, gpu_tokens)) < LOGIT_TOL
    assert n[0] == 512 + max_new and kvl[0] == n[0] - 1
    # the statistics are those of a loop whose targets are the emitted tokens (and the oracle
    # loop's own when the streams agree, which they do unless a near-tie flipped a token)
    want = counters_for_streams([ctxt], [gpu_tokens], 3, 10)
    for key in COUNTERS:
        assert st[key] == want[key], key
    assert st["tau_hist"][:11] == want["tau_hist"][:11]
    assert gpu_tokens != got_o or all(st[key] == st_o[key] for key in COUNTERS)
    # plain decoding from the same kernels (k = 0) gives the same tokens
    h0, n0, _, st0 = _run_gpu(ctx, [ctxt], [512], 1024, 3, 0, max_new, cs.LATEST)
    assert h0[0, 512:n0[0]].tolist() == gpu_tokens and st0["steps"] == max_new and st0["accepted"] == 0
    ctx.close()


def test_batch_of_sequences_with_eos_and_different_lengths():
    cfg = inputs.ModelConfig(n_layers=2, d_model=128, n_heads=4, n_kv_heads=2, head_dim=32, d_ffn=256, vocab=64,
                             rope_theta=10000.0, rms_eps=1e-5)
    B, k, max_new = 4, 5, 60
    ctx, model = make_pair(cfg, 256, B, k, seed=2)
    rng = np.random.default_rng(2)
    lens = [40, 25, 33, 8]
    hists = [rng.integers(0, cfg.vocab, size=n).astype(np.int32) for n in lens]
    # choose as EOS a token that plain decoding of sequence 0 produces somewhere in the middle
    c0 = O.KVCache(cfg, 1, 256); model.prefill(hists[0].tolist(), c0, 0)
    ref0 = O.greedy_decode(model, c0, 0, hists[0].tolist(), max_new)
    eos = ref0[max_new // 2]
    h, n, kvl, st = _run_gpu(ctx, hists, lens, 128, 3, k, max_new, cs.LATEST, eos_id=eos)
    gens, stopped = [], 0
    for b in range(B):
        gen = h[b, lens[b]:n[b]].tolist()
        assert kvl[b] == n[b] - 1
        assert max(greedy_margins(model, cfg, hists[b], gen)) < LOGIT_TOL, b
        assert len(gen) == max_new or gen[-1] == eos       # stops at max_new or at the first EOS
        assert eos not in gen[:-1]
        stopped += len(gen) < max_new
        gens.append(gen)
    assert stopped >= 1                                    # the EOS rule was exercised
    want = counters_for_streams(hists, gens, 3, k)        # per sequence, on the stream it emitted
    for key in COUNTERS:
        assert st[key] == want[key], key
    assert st["tau_hist"][:k + 1] == want["tau_hist"][:k + 1]
    assert st["emitted"] == int(sum(n[b] - lens[b] for b in range(B)))
    ctx.close()


def test_loop_without_graph_capture_gives_the_same_result(monkeypatch):
    """The step can also be enqueued launch by launch (CS_NO_GRAPH=1); overlapping launches of
    consecutive steps must not change any integer result."""
    monkeypatch.setenv("CS_NO_GRAPH", "1")
    cfg = inputs.TINY
    ctx, model = make_pair(cfg, 1024, 1, 10)
    ctxt, _ = inputs.tiny_context(seed=1)
    rng = np.random.default_rng(11)
    max_new = 200
    script = inputs.copy_script(rng, ctxt, max_new, 0.6, 5, 30, cfg.vocab, zipf_s=None)
    h, n, kvl, st = _run_gpu(ctx, [ctxt], [512], 1024, 3, 10, max_new, cs.LATEST, script=script[None, :])
    steps, st_o, h_sim = O.scripted_simulator(ctxt, script, 3, 10, O.LATEST, max_new)
    assert h[0, :n[0]].tolist() == h_sim
    for key in ("steps", "attempts", "accepted", "emitted", "no_match"):
        assert st[key] == st_o[key], key
    ctx.close()


def test_loop_capacity_is_reported():
    cfg = inputs.TINY
    ctx, _ = make_pair(cfg, 128, 1, 10)
    hist = np.zeros((1, 64), dtype=np.int32)
    kv = ctx.alloc_kv(); kv_len = i32([19])
    with pytest.raises(cs.CsError) as e:
        ctx.cs_decode_loop(i32(hist), i32([20]), kv, kv_len, 3, 10, 100)     # 20 + 100 > stride 64
    assert e.value.code == cs.CS_ERR_CAPACITY
    ctx.close()


def test_a_sequence_without_room_does_not_stop_the_others():
    """Batch of two: the second history leaves no room for max_new more tokens.  The loop reports
    CS_ERR_CAPACITY, leaves that sequence untouched and still runs the first one to its end."""
    cfg = inputs.TINY
    ctx, _ = make_pair(cfg, 1024, 2, 10)
    ctxt, _ = inputs.tiny_context(seed=1)
    max_new, stride = 120, 600
    lens = [400, 512]                      # 512 + 120 > 600
    script = inputs.copy_script(np.random.default_rng(3), ctxt[:400], max_new, 0.6, 5, 30, cfg.vocab, zipf_s=None)
    h = np.zeros((2, stride), dtype=np.int32)
    for b, n in enumerate(lens):
        h[b, :n] = ctxt[:n]
    hd, ld = i32(h), i32(lens)
    kv = ctx.alloc_kv()
    kvl = torch.zeros(2, dtype=torch.int32, device="cuda")
    ctx.cs_prefill(hd, ld, 512, kv, kvl)
    with pytest.raises(cs.CsError) as err:
        ctx.cs_decode_loop(hd, ld, kv, kvl, 3, 10, max_new, script=i32(np.stack([script, script])))
    assert err.value.code == cs.CS_ERR_CAPACITY
    _, _, h_sim = O.scripted_simulator(ctxt[:400], script, 3, 10, O.LATEST, max_new)
    assert ld.cpu().tolist() == [400 + max_new, 512] and kvl.cpu().tolist() == [400 + max_new - 1, 511]
    assert hd[0, :400 + max_new].cpu().tolist() == h_sim
    assert hd[1].cpu().tolist() == h[1].tolist()
    assert ctx.cs_sync_status() == 0       # the status was reported once and cleared
    ctx.close()


@pytest.mark.parametrize("k", [50, 100])
def test_wide_blocks_match_the_simulator(k):
    """Copy windows of 50 and 100 tokens (the sweep of Sec. 4 / App. B.1): blocks of 51 and 101
    rows through the same kernels; every integer of the scripted loop equals the simulator's."""
    cfg = inputs.TINY
    ctx, model = make_pair(cfg, 1536, 1, k)
    ctxt, spans = inputs.tiny_context(seed=1)
    rng = np.random.default_rng(11)
    max_new = 420
    script = inputs.copy_script(rng, ctxt, max_new, 0.7, 20, 160, cfg.vocab, zipf_s=None)
    h, n, kvl, st = _run_gpu(ctx, [ctxt], [512], 1024, 3, k, max_new, cs.LATEST, script=script[None, :])
    steps, st_o, h_sim = O.scripted_simulator(ctxt, script, 3, k, O.LATEST, max_new)
    assert n[0] == 512 + max_new and kvl[0] == n[0] - 1
    assert h[0, :n[0]].tolist() == h_sim
    for key in ("steps", "attempts", "accepted", "emitted", "no_match"):
        assert st[key] == st_o[key], key
    assert max(s["tau"] for s in steps) > 20          # the wide window is actually used
    ctx.close()


def test_real_mode_loop_with_wide_heads_and_caches_of_many_key_tiles():
    """Real-mode decoding with 128-wide heads (the tensor-core attention kernel) over caches of
    10-14 key tiles, batch 8: with 9 key slices per (sequence, KV head) several slices walk two
    tiles, and inside the loop the tiles of cached keys are fetched ahead of the dependency
    wait.  Every emitted token must be the oracle's greedy choice up to the logit tolerance
    (losslessness, Sec. 1 / App. B.2), so a wrong attention result cannot hide behind a script."""
    cfg = inputs.ModelConfig(n_layers=2, d_model=256, n_heads=8, n_kv_heads=4, head_dim=128, d_ffn=512, vocab=512,
                             rope_theta=500000.0, rms_eps=1e-5)
    B, k, max_new, max_seq = 8, 10, 16, 1792
    ctx, model = make_pair(cfg, max_seq, B, k, seed=5, gain_jitter=0.1)
    rng = np.random.default_rng(5)
    lens = [1700, 1301, 1536, 1663, 1409, 1280, 1599, 1688]
    hists = []
    for n in lens:
        h = rng.integers(0, cfg.vocab, size=n).astype(np.int32)
        src = int(rng.integers(0, n // 2))
        h[n - 40:] = h[src:src + 40]          # the context ends inside a replay of an earlier span
        hists.append(h)
    h, n, kvl, st = _run_gpu(ctx, hists, lens, 1728, 3, k, max_new, cs.LATEST)
    assert st["attempts"] >= B                 # every sequence opened with a match and a 10-token draft
    gens = []
    for b in range(B):
        gen = h[b, lens[b]:n[b]].tolist()
        assert len(gen) == max_new and kvl[b] == n[b] - 1
        assert max(greedy_margins(model, cfg, hists[b], gen)) < LOGIT_TOL, b
        gens.append(gen)
    want = counters_for_streams(hists, gens, 3, k)
    for key in COUNTERS:
        assert st[key] == want[key], key
    assert st["tau_hist"][:k + 1] == want["tau_hist"][:k + 1]
    ctx.close()


def test_steps_driven_from_host_memory():
    """cs_step_host: histories kept on the host, one call per step.  Scripted mode against the
    model-free simulator (two sequences of different lengths), then real mode against the
    oracle's greedy choice."""
    cfg = inputs.TINY
    ctx, model = make_pair(cfg, 1024, 2, 10)
    rng = np.random.default_rng(11)
    ctxt, _ = inputs.tiny_context(seed=1)
    lens = [512, 300]
    max_new, stride, k = 80, 640, 10
    scripts = [inputs.copy_script(rng, ctxt[:n], max_new, 0.6, 5, 30, cfg.vocab, zipf_s=None) for n in lens]

    def prefilled():
        h = np.zeros((2, stride), dtype=np.int32)
        for b, n in enumerate(lens):
            h[b, :n] = ctxt[:n]
        kv = ctx.alloc_kv()
        kvl = torch.zeros(2, dtype=torch.int32, device="cuda")
        ctx.cs_prefill(i32(h), i32(lens), max(lens), kv, kvl)
        return torch.from_numpy(h).pin_memory(), torch.tensor(lens, dtype=torch.int32).pin_memory(), kv, kvl

    hist_h, len_h, kv, kvl = prefilled()
    hist_d, len_d = torch.empty(2, stride, dtype=torch.int32, device="cuda"), torch.empty(2, dtype=torch.int32, device="cuda")
    acc, out = torch.zeros(2, dtype=torch.int32).pin_memory(), torch.zeros(2, k + 1, dtype=torch.int32).pin_memory()
    scr = torch.zeros(2, k + 1, dtype=torch.int32).pin_memory()
    pads = [np.concatenate([s, np.full(k + 1, -1, dtype=np.int32)]) for s in scripts]
    sims = [O.scripted_simulator(ctxt[:n], s, 3, k, O.LATEST, max_new + k + 1)[0] for n, s in zip(lens, pads)]
    for step in range(6):
        e = [int(len_h[b]) - lens[b] for b in range(2)]
        assert max(e) + k + 1 <= max_new          # every row of the block still has a script entry
        for b in range(2):
            scr[b] = torch.from_numpy(pads[b][e[b]:e[b] + k + 1])
        ctx.cs_step_host(hist_h, len_h, hist_d, len_d, kv, kvl, 3, k, acc, out, script_host=scr)
        for b in range(2):
            rec = sims[b][step]
            assert int(acc[b]) == rec["tau"] and out[b, :rec["tau"] + 1].tolist() == rec["out"], (step, b)
            assert int(len_h[b]) == rec["n"] + rec["tau"] + 1
    assert ctx.cs_sync_status() == 0
    assert kvl.cpu().tolist() == [int(len_h[b]) - 1 for b in range(2)]
    for b in range(2):
        n = int(len_h[b])
        assert hist_h[b, lens[b]:n].tolist() == scripts[b][:n - lens[b]].tolist()

    # real mode: every emitted token is the oracle's greedy choice up to the logit tolerance
    hist_h, len_h, kv, kvl = prefilled()
    for _ in range(8):
        ctx.cs_step_host(hist_h, len_h, hist_d, len_d, kv, kvl, 3, k, acc, out)
    assert ctx.cs_sync_status() == 0
    for b in range(2):
        gen = hist_h[b, lens[b]:int(len_h[b])].tolist()
        assert len(gen) >= 8 and max(greedy_margins(model, cfg, ctxt[:lens[b]], gen)) < LOGIT_TOL
    # a caller that rewrote a row in place says so; the next call uploads the rows in full again
    ctx.cs_step_host_reset()
    before = [int(len_h[b]) for b in range(2)]
    ctx.cs_step_host(hist_h, len_h, hist_d, len_d, kv, kvl, 3, k, acc, out)
    for b in range(2):
        assert int(len_h[b]) == before[b] + int(acc[b]) + 1
        assert hist_d[b, :before[b]].cpu().tolist() == hist_h[b, :before[b]].tolist()
    # a key longer than the search kernel compares, or an unknown policy, is refused on the host
    for bad in (dict(gamma=9), dict(gamma=3, policy=7)):
        with pytest.raises(cs.CsError) as err:
            ctx.cs_step_host(hist_h, len_h, hist_d, len_d, kv, kvl, bad["gamma"], k, acc, out, policy=bad.get("policy", cs.LATEST))
        assert err.value.code == cs.CS_ERR_ARG
    # a history row without room for one more block is refused on the host, nothing changes
    len_h[0] = stride - 5
    with pytest.raises(cs.CsError):
        ctx.cs_step_host(hist_h, len_h, hist_d, len_d, kv, kvl, 3, k, acc, out)
    assert int(len_h[0]) == stride - 5
    ctx.close()
