"""Pins for acceptance, truncation and the generation loop (Sec. 3.2; App. B.2, B.3):
losslessness against plain greedy decoding, the scripted mode against a model-free
integer simulator, structural invariants, and a constructed Fig.-2-shaped example."""
import os

import numpy as np
import pytest

from oracle import copyspec_oracle as O
from paper_2502_08923_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _prefilled(cfg, w, hist, max_seq, contract=True):
    model = O.Model(cfg, w, contract=contract)
    cache = O.KVCache(cfg, 1, max_seq)
    model.prefill(hist, cache, 0)
    return model, cache


def test_accept_length_brute_force():
    rng = np.random.default_rng(0)
    for _ in range(500):
        k = int(rng.integers(0, 8))
        d = rng.integers(0, 3, size=k).tolist()
        t = rng.integers(0, 3, size=k + 1).tolist()
        want = next((i for i in range(k) if d[i] != t[i]), k)
        assert O.accept_length(d, t) == want
    assert O.accept_length([], [5]) == 0
    assert O.accept_length([1, 2, 3], [1, 2, 3, 9]) == 3
    assert O.accept_length([1, 2, 3], [9, 2, 3, 9]) == 0     # later agreement does not count


def test_argmax_ties_take_lowest_id():
    assert O.argmax_lowest(np.array([1.0, 3.0, 3.0, 2.0])) == 1
    assert O.argmax_lowest(np.array([0.0, 0.0])) == 0


def _loopy_model_case(seed):
    """A tiny random model whose greedy continuation soon falls into a cycle, so that
    real-mode copying actually gets accepted (random-init models repeat themselves)."""
    cfg = inputs.ModelConfig(n_layers=2, d_model=64, n_heads=4, n_kv_heads=2, head_dim=16,
                             d_ffn=128, vocab=64, rope_theta=10000.0, rms_eps=1e-5)
    w = inputs.make_weights(cfg, seed=seed)
    rng = np.random.default_rng(seed)
    hist = rng.integers(0, cfg.vocab, size=40).tolist()
    return cfg, w, hist


@pytest.mark.parametrize("seed", [0, 1, 2])
@pytest.mark.parametrize("policy", [O.LATEST, O.FIRST])
def test_real_mode_is_lossless(seed, policy):
    """Sec. 1 / App. B.2: a token is accepted only if it is the target's argmax, so the
    emitted sequence equals plain greedy decoding whatever is drafted."""
    cfg, w, hist = _loopy_model_case(seed)
    max_new = 96
    m1, c1 = _prefilled(cfg, w, hist, 40 + max_new + 16)
    want = O.greedy_decode(m1, c1, 0, list(hist), max_new)
    m2, c2 = _prefilled(cfg, w, hist, 40 + max_new + 16)
    h2 = list(hist)
    trace = []
    got, st = O.decode_loop(m2, c2, 0, h2, gamma=3, k=10, policy=policy, max_new=max_new,
                            trace=trace)
    assert got == want
    assert h2 == hist + want
    assert st["emitted"] == max_new == st["accepted"] + st["steps"]
    assert st["steps"] == st["attempts"] + st["no_match"]
    # the case is only meaningful if copying happened
    assert st["accepted"] > 0 and st["steps"] < max_new
    for rec in trace:
        assert 0 <= rec["tau"] <= len(rec["draft"]) <= 10
        assert len(rec["out"]) == rec["tau"] + 1
        if rec["tau"] < len(rec["draft"]) and len(rec["out"]) == rec["tau"] + 1 and rec is not trace[-1]:
            # Sec. 3.2: after a rejection the generated token differs from the draft's
            assert rec["out"][-1] != rec["draft"][rec["tau"]]
    # the KV kept after the loop equals the KV of plain decoding up to n-1 (App. B.2)
    n = len(h2)
    assert np.abs(c2.a[:, :, :, :, :n - 1] - c1.a[:, :, :, :, :n - 1]).max() < 1e-9


def test_eos_stops_and_drops_the_rest():
    cfg, w, hist = _loopy_model_case(0)
    m1, c1 = _prefilled(cfg, w, hist, 200)
    ref = O.greedy_decode(m1, c1, 0, list(hist), 64)
    eos = ref[20]
    first = ref.index(eos)
    m2, c2 = _prefilled(cfg, w, hist, 200)
    h2 = list(hist)
    got, st = O.decode_loop(m2, c2, 0, h2, 3, 10, O.LATEST, 64, eos_id=eos)
    assert got == ref[:first + 1]
    assert h2 == hist + got and st["emitted"] == len(got)


@pytest.mark.parametrize("k", [0, 1, 5, 10, 20])
@pytest.mark.parametrize("policy", [O.LATEST, O.FIRST])
def test_scripted_mode_equals_simulator_and_script(k, policy):
    cfg = inputs.ModelConfig(n_layers=1, d_model=32, n_heads=2, n_kv_heads=1, head_dim=16,
                             d_ffn=64, vocab=50, rope_theta=10000.0, rms_eps=1e-5)
    w = inputs.make_weights(cfg, seed=3)
    rng = np.random.default_rng(9)
    ctx = rng.integers(0, cfg.vocab, size=120).astype(np.int32)
    max_new = 75
    script = inputs.copy_script(rng, ctx, max_new, 0.6, 4, 25, cfg.vocab, zipf_s=None)
    model, cache = _prefilled(cfg, w, ctx.tolist(), 120 + max_new + 32)
    h = ctx.tolist()
    trace = []
    got, st = O.decode_loop(model, cache, 0, h, 3, k, policy, max_new, script=script,
                            trace=trace)
    steps, st2, h_sim = O.scripted_simulator(ctx, script, 3, k, policy, max_new)
    assert got == script.tolist()                    # emitted stream is the script itself
    assert h == h_sim
    assert st == st2
    assert [(r["n"], r["p0"], r["draft"], r["tau"], r["out"]) for r in trace] == \
           [(r["n"], r["p0"], r["draft"], r["tau"], r["out"]) for r in steps]
    assert st["emitted"] == max_new
    if k == 0:
        assert st["steps"] == max_new and st["accepted"] == 0
    if k >= 5:
        assert st["steps"] < max_new                 # planted spans do get copied


def test_verify_step_kv_length_and_outputs():
    cfg, w, hist = _loopy_model_case(1)
    model, cache = _prefilled(cfg, w, hist, 80)
    kv_len = len(hist) - 1
    rng = np.random.default_rng(0)
    for tau_want in (0, 3, 10):
        last, draft, dlen, script = inputs.verify_inputs_with_tau(rng, 1, 10, [tau_want], cfg.vocab)
        tau, out, am, new_len, logits = O.verify_step(model, cache, 0, last[0], draft[0], kv_len,
                                                      script_row=script[0])
        assert tau == tau_want and len(out) == tau + 1 and new_len == kv_len + tau + 1
        assert out == script[0][:tau + 1].tolist()
        assert logits.shape == (11, cfg.vocab) and len(am) == 11
    # real mode, empty draft: exactly one plain decode step
    tau, out, am, new_len, _ = O.verify_step(model, cache, 0, hist[-1], [], kv_len)
    assert tau == 0 and out == am and new_len == kv_len + 1


def _read_golden(name):
    rec = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, _, val = line.partition(":")
            rec[key.strip()] = val.strip()
    return rec


def test_fig2_structured_example():
    """Fig. 2 (caption): 3 matched tokens, 10 copied, a prefix accepted, one extra token."""
    g = _read_golden("fig2_structure.txt")
    words = (g["context"] + " " + g["generated"] + " " + g["target"]).split()
    vocab = {}
    for wd in words:
        vocab.setdefault(wd, len(vocab))
    enc = lambda s: [vocab[x] for x in s.split()]
    hist = enc(g["context"]) + enc(g["generated"])
    script = enc(g["target"])
    gamma, k = int(g["gamma"]), int(g["k"])
    n = len(hist)
    p0 = O.find_match(np.asarray(hist), n, gamma, O.LATEST)
    assert p0 == int(g["expected_p0"]) == O.find_match(np.asarray(hist), n, gamma, O.FIRST)
    draft = O.gather_draft(hist, n, p0, gamma, k)
    assert draft == enc(g["expected_draft"]) and len(draft) == 10
    tau = O.accept_length(draft, script)
    assert tau == int(g["expected_tau"])
    # through the loop, with a throw-away model (scripted mode ignores its argmax)
    cfg = inputs.ModelConfig(n_layers=1, d_model=32, n_heads=2, n_kv_heads=1, head_dim=16,
                             d_ffn=64, vocab=len(vocab), rope_theta=10000.0, rms_eps=1e-5)
    w = inputs.make_weights(cfg, seed=0)
    model, cache = _prefilled(cfg, w, hist, 64)
    h = list(hist)
    trace = []
    O.decode_loop(model, cache, 0, h, gamma, k, O.LATEST, len(script), script=script, trace=trace)
    assert trace[0]["out"] == enc(g["expected_emitted"]) and trace[0]["tau"] == tau
    assert trace[1]["n"] == int(g["expected_hist_len_after"])
    assert trace[1]["n"] - 1 == int(g["expected_kv_len_after"])
    assert trace[1]["p0"] == int(g["expected_next_p0"])


def test_tiny_config_loop_runs_and_is_lossless():
    """The small CPU-checkable configuration end to end (512-token context with planted
    spans, gamma=3, k=10, 64 steps) in real mode against plain greedy decoding."""
    cfg = inputs.TINY
    w = inputs.make_weights(cfg, seed=0)
    ctx, spans = inputs.tiny_context(seed=1)
    hist = ctx.tolist()
    m1, c1 = _prefilled(cfg, w, hist, 1024)
    m2, c2 = _prefilled(cfg, w, hist, 1024)
    h2 = list(hist)
    got, st = O.decode_loop(m2, c2, 0, h2, 3, 10, O.LATEST, 64)
    want = O.greedy_decode(m1, c1, 0, list(hist), 64)
    assert got == want and st["emitted"] == 64
