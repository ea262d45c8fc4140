"""The seeded workload generators produce what they promise (checked with the oracle's
model-free simulator, which is pure integer logic)."""
import numpy as np
import pytest

from oracle import copyspec_oracle as O
from paper_2502_08923_b200 import inputs


@pytest.mark.parametrize("policy", [O.LATEST, O.FIRST])
def test_tau_controlled_case_gives_the_requested_accept_lengths(policy):
    rng = np.random.default_rng(0)
    taus = [int(t) for t in rng.permutation(np.repeat(np.arange(11), 10))]
    hist, script = inputs.tau_controlled_case(rng, taus, 3, 10, 4096, 128256)
    assert len(hist) == 4097 and len(script) == sum(taus) + len(taus)
    # ids are distinct except for the two tokens each path shares with its predecessor
    assert len(set(hist.tolist())) >= len(hist) - 3 - 2 * len(taus)
    steps, st, _ = O.scripted_simulator(hist, script, 3, 10, policy, len(script))
    assert [s["tau"] for s in steps] == taus
    assert st["no_match"] == 0 and st["steps"] == len(taus)


def test_tau_controlled_case_needs_room():
    with pytest.raises(ValueError):
        inputs.tau_controlled_case(np.random.default_rng(0), [5] * 400, 3, 10, 4096, 128256)


def test_shapes_of_the_named_configurations():
    c = inputs.LLAMA8B
    assert c.params_per_layer() == 218103808 and c.streamed_params() == 7504658432
    assert c.kv_bytes_per_token() == 131072
    ctx, script = inputs.long_context_case(4, context_len=3000, script_len=400)
    assert len(ctx) == 3000 and len(script) == 400
    # a good share of the script's 3-grams occur in the context (verbatim spans)
    grams = {tuple(ctx[i:i + 3]) for i in range(len(ctx) - 2)}
    hit = sum(tuple(script[i:i + 3]) in grams for i in range(len(script) - 2)) / (len(script) - 2)
    assert hit > 0.4
    h, s, off = inputs.multi_turn_case(5, history_len=2048, answer_len=256, script_len=400)
    assert len(h) == 2048 and len(s) == 400
    same = sum(int(a == b) for a, b in zip(h[off:off + 50], s[:50]))
    assert same >= 25            # the second turn starts as an edited copy of the answer
    pk = __import__("paper_2502_08923_b200.binding", fromlist=["pack_gate_up"]).pack_gate_up
    import torch
    w = torch.arange(2 * 100 * 8, dtype=torch.float32).view(200, 8)       # F = 100: ragged last block
    p = pk(w, 100)
    assert p.shape == (256, 8)
    assert torch.equal(p[0:64], w[0:64]) and torch.equal(p[64:128], w[100:164])
    assert torch.equal(p[128:164], w[64:100]) and torch.equal(p[192:228], w[164:200])
    assert p[164:192].abs().sum() == 0 and p[228:].abs().sum() == 0


# ------------------------------------------------------------------ the write-canary checker itself
def test_canary_checker_catches_stray_writes():
    """The checker of the GPU canary tests, tried on CPU tensors with planted stray writes: one
    position behind the block, one in front of it, one in another sequence, one in a guard band."""
    import pytest
    import torch
    from helpers import PATTERN, assert_only_rows_written, guarded_kv
    cfg = inputs.TINY
    B, max_seq, kv_len, rows = 2, 40, 17, 5
    buf, kv = guarded_kv(cfg, B, max_seq, kv_len, seed=1, device="cpu")
    before = kv.clone()
    kv[:, :, 0, :, kv_len:kv_len + rows, :] = 0.5                      # what a step may write
    assert_only_rows_written(buf, kv, before, [(kv_len, rows), (kv_len, 0)])
    for where in [(0, 0, 0, 0, kv_len + rows, 0), (1, 1, 0, 0, kv_len - 1, 3), (0, 1, 1, 0, kv_len, 0)]:
        bad = kv.clone()
        bad[where] = 7.0
        with pytest.raises(AssertionError):
            assert_only_rows_written(buf, bad, before, [(kv_len, rows), (kv_len, 0)])
    buf2 = buf.clone()
    buf2[5] = 0.0
    with pytest.raises(AssertionError):
        assert_only_rows_written(buf2, kv, before, [(kv_len, rows), (kv_len, 0)])
    assert float(torch.tensor(PATTERN, dtype=torch.bfloat16)) == PATTERN
