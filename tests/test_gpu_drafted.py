"""cs_decode_loop_drafted on the GPU against the oracle's CopySpec + draft-model loop
(Sec. 3.3; App. B.3 step 3): emitted tokens, per-kind statistics, both cache lengths and the
contents of both caches after the roll-backs."""
import numpy as np
import pytest
import torch

from oracle import copyspec_oracle as O
from paper_2502_08923_b200 import binding as cs, inputs
from helpers import LOGIT_TOL, counters_for_streams, greedy_margins, i32, make_pair

pytestmark = pytest.mark.gpu

TARGET = inputs.ModelConfig(n_layers=2, d_model=128, n_heads=4, n_kv_heads=2, head_dim=32, d_ffn=256, vocab=64,
                            rope_theta=10000.0, rms_eps=1e-5)
SMALL = inputs.ModelConfig(n_layers=1, d_model=64, n_heads=2, n_kv_heads=1, head_dim=32, d_ffn=128, vocab=64,
                           rope_theta=10000.0, rms_eps=1e-5)
KEYS = ("steps", "attempts", "accepted", "emitted", "no_match", "draft_attempts", "draft_accepted")


def _gpu_run(tctx, dctx, hist, stride, gamma, k, delta, max_new, script=None, eos_id=-1, drafter_prefix=None):
    n = len(hist)
    h = np.zeros((1, stride), dtype=np.int32)
    h[0, :n] = hist
    hd, ld = i32(h), i32([n])
    kv_t, kv_d = tctx.alloc_kv(), (dctx.alloc_kv() if dctx is not None else None)
    kvl_t = torch.zeros(1, dtype=torch.int32, device="cuda")
    tctx.cs_prefill(hd, ld, n, kv_t, kvl_t)
    kvl_d = None
    if dctx is not None:
        kvl_d = torch.zeros(1, dtype=torch.int32, device="cuda")
        m = n if drafter_prefix is None else drafter_prefix + 1     # the draft model may have seen only a prefix
        dctx.cs_prefill(hd, i32([m]), m, kv_d, kvl_d)
    st = tctx.cs_decode_loop_drafted(dctx, hd, ld, kv_t, kvl_t, kv_d, kvl_d, gamma, k, delta, max_new, eos_id=eos_id,
                                     script=None if script is None else i32(script))
    return hd.cpu().numpy()[0], int(ld[0]), kv_t, int(kvl_t[0]), kv_d, (int(kvl_d[0]) if kvl_d is not None else None), st


def _oracle_run(tm, dm, hist, cap, gamma, k, delta, max_new, script=None, eos_id=-1, drafter_prefix=None):
    tc, dc = O.KVCache(TARGET, 1, cap), O.KVCache(SMALL, 1, cap)
    tm.prefill(hist, tc, 0)
    d_len = len(hist) - 1 if drafter_prefix is None else drafter_prefix
    dm.forward_block(hist[:d_len], 0, dc, 0)
    h, trace = list(hist), []
    got, st, d_len = O.decode_loop_drafted(tm, tc, dm, dc, d_len, 0, h, gamma, k, delta, O.LATEST, max_new,
                                           eos_id=eos_id, script=script, trace=trace)
    return h, got, st, d_len, tc, dc, trace


def _cache_close(kv_gpu, cache, n, tol=2e-2):
    a = kv_gpu[:, :, 0, :, :n, :].float().cpu().numpy()
    b = cache.a[:, :, 0, :, :n, :]
    return float(np.abs(a - b).max()) <= tol


def _mixed_script(rng, dm, context, max_new):
    """A target stream that alternates spans lifted from the context (copy steps) with stretches
    that follow the draft model's own greedy choice four times out of five (drafted steps whose
    proposals are partly accepted)."""
    cap = len(context) + max_new + 8
    cache = O.KVCache(SMALL, 1, cap)
    seq = list(context)
    dm.forward_block(seq[:-1], 0, cache, 0)
    script = []
    while len(script) < max_new:
        if rng.random() < 0.5:
            src = int(rng.integers(0, len(context) - 24))
            span = [int(t) for t in context[src:src + int(rng.integers(12, 20))]]
        else:
            span = []
            for _ in range(int(rng.integers(8, 14))):
                lg = dm.forward_block(seq[-1:], len(seq) - 1, cache, 0)
                t = O.argmax_lowest(lg[0]) if rng.random() < 0.8 else int(rng.integers(0, 64))
                span.append(t)
                seq.append(t)
            script += span
            continue
        for t in span:                     # keep the draft model's cache in step with the stream
            dm.forward_block(seq[-1:], len(seq) - 1, cache, 0)
            seq.append(t)
        script += span
    return np.asarray(script[:max_new], dtype=np.int32)


@pytest.mark.parametrize("delta", [3, 5])
def test_real_mode_with_a_draft_model(delta):
    max_new, cap, stride = 80, 256, 192
    tctx, tm = make_pair(TARGET, cap, 1, 10, seed=2)
    dctx, dm = make_pair(SMALL, cap, 1, 3, seed=12)        # catches up four tokens per block
    hist = np.random.default_rng(2).integers(0, 64, size=40).astype(np.int32).tolist()
    h, n, kv_t, kvl_t, kv_d, kvl_d, st = _gpu_run(tctx, dctx, hist, stride, 3, 10, delta, max_new)
    gen = h[40:n].tolist()
    assert len(gen) == max_new and kvl_t == n - 1 and kvl_d <= n - 1
    assert max(greedy_margins(tm, TARGET, hist, gen)) < LOGIT_TOL      # losslessness (Sec. 1 / App. B.2)
    assert st["steps"] == st["attempts"] + st["no_match"] and st["draft_attempts"] == st["no_match"] > 0
    assert st["emitted"] == max_new == st["steps"] + st["accepted"] + st["draft_accepted"]
    h_o, got, st_o, d_len, tc, dc, trace = _oracle_run(tm, dm, hist, cap, 3, 10, delta, max_new)
    # The target's cache is that of the accepted tokens whatever the draft model proposed.
    t_ref = O.KVCache(TARGET, 1, cap)
    tm.forward_block([int(t) for t in h[:n - 1]], 0, t_ref, 0)
    assert _cache_close(kv_t, t_ref, n - 1)
    # Which steps drafted and how much of each proposal survived depends on the draft model's own
    # greedy choices, so the step counters are compared where the two runs took the same path: the
    # streams agree (they do unless a near-tie of the target flipped a token, which the margin
    # check above bounds) and so does the number of drafted steps.
    if gen == got and st["draft_attempts"] == st_o["draft_attempts"]:
        for key in KEYS:
            assert st[key] == st_o[key], key
        assert kvl_d == d_len and _cache_close(kv_d, dc, d_len)
    else:
        assert gen == got or max(greedy_margins(tm, TARGET, hist, gen)) < LOGIT_TOL
    tctx.close(); dctx.close()


def test_a_draft_model_equal_to_the_target_has_every_proposal_accepted():
    """Closed form: with the target's own weights as the draft model every drafted step accepts
    all delta proposals and nothing is rolled back."""
    max_new, cap, stride, delta = 61, 256, 128, 4
    w = inputs.make_weights(TARGET, seed=4)
    tctx, tm = make_pair(TARGET, cap, 1, 10, weights=w)
    dctx, _ = make_pair(TARGET, cap, 1, 3, weights=w)
    hist = np.random.default_rng(4).integers(0, 64, size=30).astype(np.int32).tolist()
    n0 = len(hist)
    h = np.zeros((1, stride), dtype=np.int32); h[0, :n0] = hist
    hd, ld = i32(h), i32([n0])
    kv_t, kv_d = tctx.alloc_kv(), dctx.alloc_kv()
    kvl_t, kvl_d = torch.zeros(1, dtype=torch.int32, device="cuda"), torch.zeros(1, dtype=torch.int32, device="cuda")
    tctx.cs_prefill(hd, ld, n0, kv_t, kvl_t)
    dctx.cs_prefill(hd, ld, n0, kv_d, kvl_d)
    st = tctx.cs_decode_loop_drafted(dctx, hd, ld, kv_t, kvl_t, kv_d, kvl_d, 3, 10, delta, max_new)
    n = int(ld[0])
    gen = hd[0, n0:n].cpu().tolist()
    assert len(gen) == max_new and max(greedy_margins(tm, TARGET, hist, gen)) < LOGIT_TOL
    assert st["draft_attempts"] > 0
    # every drafted step but a clipped last one emits delta + 1 tokens
    assert st["draft_accepted"] >= delta * (st["draft_attempts"] - 1)
    assert st["emitted"] == max_new == st["steps"] + st["accepted"] + st["draft_accepted"]
    tctx.close(); dctx.close()


@pytest.mark.parametrize("no_graph", [False, True])
def test_scripted_mode_mixes_copy_steps_and_drafted_steps(no_graph, monkeypatch):
    if no_graph:      # the forwards enqueued kernel by kernel instead of replayed from their graphs
        monkeypatch.setenv("CS_NO_GRAPH", "1")
    max_new, cap, stride = 120, 384, 320
    tctx, tm = make_pair(TARGET, cap, 1, 10, seed=3)
    dctx, dm = make_pair(SMALL, cap, 1, 3, seed=13)
    rng = np.random.default_rng(7)
    context = rng.integers(0, 64, size=150).astype(np.int32)
    script = _mixed_script(rng, dm, context.tolist(), max_new)
    # the draft model starts 30 tokens behind, as after a run of copy steps
    h, n, kv_t, kvl_t, kv_d, kvl_d, st = _gpu_run(tctx, dctx, context.tolist(), stride, 3, 10, 4, max_new, script=script,
                                                  drafter_prefix=119)
    assert h[150:n].tolist() == script.tolist() and kvl_t == n - 1       # the emitted stream is the script
    h_o, got, st_o, d_len, tc, dc, trace = _oracle_run(tm, dm, context.tolist(), cap, 3, 10, 4, max_new, script=script,
                                                       drafter_prefix=119)
    assert st_o["attempts"] > 0 and st_o["accepted"] > 0                 # copy steps happened
    assert st_o["draft_attempts"] > 0 and st_o["draft_accepted"] > 0     # and drafted steps with accepted proposals
    assert any(r["drafted"] and r["tau"] < 4 for r in trace)             # and roll-backs of the draft cache
    for key in KEYS:
        assert st[key] == st_o[key], key
    assert st["tau_hist"][:11] == st_o["tau_hist"][:11]
    assert kvl_d == d_len
    assert _cache_close(kv_t, tc, n - 1) and _cache_close(kv_d, dc, d_len)
    tctx.close(); dctx.close()


def test_delta_zero_needs_no_draft_model_and_eos_stops_the_loop():
    max_new, cap, stride = 60, 256, 128
    tctx, tm = make_pair(TARGET, cap, 1, 10, seed=2)
    hist = np.random.default_rng(2).integers(0, 64, size=40).astype(np.int32).tolist()
    c0 = O.KVCache(TARGET, 1, cap); tm.prefill(hist, c0, 0)
    ref = O.greedy_decode(tm, c0, 0, list(hist), max_new)
    eos = ref[max_new // 2]
    h, n, kv_t, kvl_t, _, _, st = _gpu_run(tctx, None, hist, stride, 3, 10, 0, max_new, eos_id=eos)
    gen = h[40:n].tolist()
    assert max(greedy_margins(tm, TARGET, hist, gen)) < LOGIT_TOL
    assert gen[-1] == eos and eos not in gen[:-1] and kvl_t == n - 1 and st["draft_attempts"] == 0
    c1 = O.KVCache(TARGET, 1, cap); tm.prefill(hist, c1, 0)
    got, st_o = O.decode_loop(tm, c1, 0, list(hist), 3, 10, O.LATEST, max_new, eos_id=eos)
    want = counters_for_streams([hist], [gen], 3, 10)      # the loop's bookkeeping on the stream it emitted
    for key in ("steps", "attempts", "accepted", "emitted", "no_match"):
        assert st[key] == want[key], key
    assert gen != got or all(st[key] == st_o[key] for key in ("steps", "attempts", "accepted", "emitted", "no_match"))
    tctx.close()


def test_argument_and_capacity_errors_are_found_on_the_host():
    tctx, _ = make_pair(TARGET, 128, 1, 4, seed=2)
    dctx, _ = make_pair(SMALL, 128, 1, 3, seed=12)
    h, ld = i32(np.zeros((1, 96), dtype=np.int32)), i32([40])
    kv_t, kv_d = tctx.alloc_kv(), dctx.alloc_kv()
    kvl = i32([39])
    with pytest.raises(cs.CsError):      # k above the target's k_max
        tctx.cs_decode_loop_drafted(dctx, h, ld, kv_t, kvl, kv_d, i32([39]), 3, 10, 3, 8)
    with pytest.raises(cs.CsError):      # delta > 0 without a draft model
        tctx.cs_decode_loop_drafted(None, h, ld, kv_t, kvl, None, None, 3, 4, 3, 8)
    with pytest.raises(cs.CsError):      # the draft model's cache claims more than the history
        tctx.cs_decode_loop_drafted(dctx, h, ld, kv_t, kvl, kv_d, i32([40]), 3, 4, 3, 8)
    with pytest.raises(cs.CsError):      # history row too short for max_new more tokens
        tctx.cs_decode_loop_drafted(dctx, h, ld, kv_t, kvl, kv_d, i32([39]), 3, 4, 3, 80)
    assert int(ld[0]) == 40 and int(kvl[0]) == 39
    tctx.close(); dctx.close()
