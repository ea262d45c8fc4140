"""Pins for the oracle's CopySpec + draft-model loop (Sec. 3.3; App. B.3 step 3): losslessness
against plain greedy decoding, the closed form for a draft model equal to the target, the
reduction to the copy-only loop, scripted-mode output, and the rolled-back draft cache."""
import numpy as np
import pytest

from oracle import copyspec_oracle as O
from paper_2502_08923_b200 import inputs

TARGET = inputs.ModelConfig(n_layers=2, d_model=64, n_heads=4, n_kv_heads=2, head_dim=16,
                            d_ffn=128, vocab=64, rope_theta=10000.0, rms_eps=1e-5)
SMALL = inputs.ModelConfig(n_layers=1, d_model=32, n_heads=2, n_kv_heads=1, head_dim=16,
                           d_ffn=64, vocab=64, rope_theta=10000.0, rms_eps=1e-5)


def _prefilled(cfg, w, hist, max_seq):
    model = O.Model(cfg, w, contract=True)
    cache = O.KVCache(cfg, 1, max_seq)
    return model, cache, model.prefill(hist, cache, 0)


@pytest.mark.parametrize("seed", [0, 1])
@pytest.mark.parametrize("delta", [3, 5])
def test_real_mode_with_a_draft_model_is_lossless(seed, delta):
    """Whatever the draft model proposes, only the target's own greedy tokens are accepted."""
    hist = np.random.default_rng(seed).integers(0, 64, size=40).tolist()
    wt, wd = inputs.make_weights(TARGET, seed=seed), inputs.make_weights(SMALL, seed=seed + 10)
    max_new, cap = 80, 40 + 80 + 16
    m, c, _ = _prefilled(TARGET, wt, hist, cap)
    want = O.greedy_decode(m, c, 0, list(hist), max_new)
    t, tc, _ = _prefilled(TARGET, wt, hist, cap)
    d, dc, d_len = _prefilled(SMALL, wd, hist, cap)
    h, trace = list(hist), []
    got, st, d_len = O.decode_loop_drafted(t, tc, d, dc, d_len, 0, h, 3, 10, delta, O.LATEST, max_new, trace=trace)
    assert got == want and h == hist + want
    assert st["steps"] == st["attempts"] + st["no_match"] and st["draft_attempts"] == st["no_match"] > 0
    assert st["emitted"] == max_new == st["steps"] + st["accepted"] + st["draft_accepted"]
    for r in trace:
        assert len(r["draft"]) == delta if r["drafted"] else len(r["draft"]) <= 10
        assert 0 <= r["tau"] <= len(r["draft"]) and r["d_len"] <= r["n"] + r["tau"]
    # target cache == plain decoding's; draft cache == a fresh pass over the accepted tokens
    n = len(h)
    assert d_len <= n - 1
    assert np.abs(tc.a[..., :n - 1, :] - c.a[..., :n - 1, :]).max() < 1e-9
    fresh = O.KVCache(SMALL, 1, cap)
    d.forward_block(h[:d_len], 0, fresh, 0)
    assert np.abs(dc.a[..., :d_len, :] - fresh.a[..., :d_len, :]).max() < 1e-9


def test_a_draft_model_equal_to_the_target_has_every_proposal_accepted():
    hist = np.random.default_rng(4).integers(0, 64, size=30).tolist()
    w = inputs.make_weights(TARGET, seed=4)
    max_new, delta, cap = 61, 4, 30 + 61 + 16
    t, tc, _ = _prefilled(TARGET, w, hist, cap)
    d, dc, d_len = _prefilled(TARGET, w, hist, cap)
    trace = []
    got, st, _ = O.decode_loop_drafted(t, tc, d, dc, d_len, 0, list(hist), 3, 10, delta, O.LATEST, max_new, trace=trace)
    assert st["draft_attempts"] > 0
    for r in trace:
        if r["drafted"] and r is not trace[-1]:
            assert r["tau"] == delta and r["out"][:delta] == r["draft"]      # delta accepted + 1 extra token
            assert r["d_len"] == r["n"] + delta - 1                           # nothing to roll back


@pytest.mark.parametrize("delta", [0, 3])
def test_scripted_mode_emits_the_script_and_delta_zero_is_the_copy_only_loop(delta):
    rng = np.random.default_rng(9)
    ctx = rng.integers(0, 64, size=100).astype(np.int32)
    max_new = 60
    script = inputs.copy_script(rng, ctx, max_new, 0.5, 4, 20, 64, zipf_s=None)
    wt, wd = inputs.make_weights(TARGET, seed=3), inputs.make_weights(SMALL, seed=5)
    cap = 100 + max_new + 32
    t, tc, _ = _prefilled(TARGET, wt, ctx.tolist(), cap)
    d, dc, d_len = _prefilled(SMALL, wd, ctx.tolist(), cap)
    h = ctx.tolist()
    got, st, d_len = O.decode_loop_drafted(t, tc, d, dc, d_len, 0, h, 3, 10, delta, O.LATEST, max_new, script=script)
    assert got == script.tolist() and st["emitted"] == max_new
    t2, tc2, _ = _prefilled(TARGET, wt, ctx.tolist(), cap)
    got2, st2 = O.decode_loop(t2, tc2, 0, ctx.tolist(), 3, 10, O.LATEST, max_new, script=script)
    if delta == 0:
        assert st["draft_attempts"] == 0 and {k: st[k] for k in st2} == st2 and d_len == 99
    else:
        # drafting never changes what a copy step does, it only shortens the no-match stretches
        assert st["steps"] <= st2["steps"] and st["draft_attempts"] > 0
        assert st["steps"] + st["accepted"] + st["draft_accepted"] == max_new
