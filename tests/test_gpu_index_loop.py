"""The generation loop searching through the gamma-gram index (Sec. 3.1: every gamma-token
subsequence of the accepted sequence in a hash map, updated after each step - App. B.3 step
2(d)) instead of scanning the history: every integer the loop produces must equal the
model-free simulator's, and hence the scan's, in both match policies."""
import numpy as np
import pytest
import torch

from oracle import copyspec_oracle as O
from paper_2502_08923_b200 import binding as cs, inputs
from helpers import COUNTERS, LOGIT_TOL, counters_for_streams, greedy_margins, i32, make_pair

pytestmark = pytest.mark.gpu


def _loop(ctx, hists, lens, stride, gamma, k, max_new, policy, index, script=None, eos_id=-1):
    B = len(hists)
    h = np.zeros((B, stride), dtype=np.int32)
    for b in range(B):
        h[b, :lens[b]] = hists[b][:lens[b]]
    hd, ld = i32(h), i32(lens)
    kv = ctx.alloc_kv()
    kvl = torch.zeros(ctx.max_batch, dtype=torch.int32, device="cuda")[:B].contiguous()
    ctx.cs_prefill(hd, ld, int(max(lens)), kv, kvl)
    ctx.cs_set_match_index(index)
    try:
        st = ctx.cs_decode_loop(hd, ld, kv, kvl, gamma, k, max_new, policy=policy, eos_id=eos_id,
                                script=None if script is None else i32(script))
    finally:
        ctx.cs_set_match_index(None)
    return hd.cpu().numpy(), ld.cpu().numpy(), kvl.cpu().numpy(), st


@pytest.mark.parametrize("policy", [cs.LATEST, cs.FIRST])
@pytest.mark.parametrize("gamma", [3, 5])
def test_scripted_batch_through_the_index(policy, gamma):
    """Three sequences of different lengths over a small alphabet (many repeated grams, so first
    and latest differ and the tables see collisions), different scripts, one finishing early."""
    cfg = inputs.ModelConfig(n_layers=1, d_model=128, n_heads=4, n_kv_heads=2, head_dim=32, d_ffn=256, vocab=12,
                             rope_theta=10000.0, rms_eps=1e-5)
    B, k, stride = 3, 6, 512
    ctx, _ = make_pair(cfg, 640, B, k, seed=1)
    rng = np.random.default_rng(7 * gamma + policy)
    lens = [150, 61, 240]
    hists = [rng.integers(0, cfg.vocab, size=n).astype(np.int32) for n in lens]
    max_new = 200
    scripts = np.stack([inputs.copy_script(rng, hists[b], max_new, 0.7, 4, 25, cfg.vocab, zipf_s=None) for b in range(B)])
    index = cs.GramIndex(B, stride, gamma)
    h, n, kvl, st = _loop(ctx, hists, lens, stride, gamma, k, max_new, policy, index, script=scripts)
    assert ctx.cs_sync_status() == 0 and index.cs_gram_index_status() == 0
    tot = O.new_stats()
    for b in range(B):
        steps, so, h_sim = O.scripted_simulator(hists[b], scripts[b], gamma, k, policy, max_new)
        assert h[b, :n[b]].tolist() == h_sim, b
        assert kvl[b] == n[b] - 1 == lens[b] + max_new - 1
        for key in COUNTERS:
            tot[key] += so[key]
        for i, v in enumerate(so["tau_hist"]):
            tot["tau_hist"][i] += v
    for key in COUNTERS:
        assert st[key] == tot[key], key
    assert st["tau_hist"] == tot["tau_hist"]
    assert st["attempts"] > 20 and st["no_match"] > 0
    # and the scan gives the very same run
    h2, n2, _, st2 = _loop(ctx, hists, lens, stride, gamma, k, max_new, policy, None, script=scripts)
    assert np.array_equal(h, h2) and np.array_equal(n, n2) and st == st2
    ctx.close()


def test_real_mode_with_eos_through_the_index():
    cfg = inputs.ModelConfig(n_layers=2, d_model=128, n_heads=4, n_kv_heads=2, head_dim=32, d_ffn=256, vocab=64,
                             rope_theta=10000.0, rms_eps=1e-5)
    B, k, max_new, stride = 4, 5, 60, 128
    ctx, model = make_pair(cfg, 256, B, k, seed=2)
    rng = np.random.default_rng(2)
    lens = [40, 25, 33, 8]
    hists = [rng.integers(0, cfg.vocab, size=n).astype(np.int32) for n in lens]
    c0 = O.KVCache(cfg, 1, 256); model.prefill(hists[0].tolist(), c0, 0)
    eos = O.greedy_decode(model, c0, 0, hists[0].tolist(), max_new)[max_new // 2]
    index = cs.GramIndex(B, stride, 3)
    h, n, kvl, st = _loop(ctx, hists, lens, stride, 3, k, max_new, cs.LATEST, index, eos_id=eos)
    gens = [h[b, lens[b]:n[b]].tolist() for b in range(B)]
    for b in range(B):
        assert kvl[b] == n[b] - 1
        assert max(greedy_margins(model, cfg, hists[b], gens[b])) < LOGIT_TOL, b
        assert len(gens[b]) == max_new or gens[b][-1] == eos
    want = counters_for_streams(hists, gens, 3, k)
    for key in COUNTERS:
        assert st[key] == want[key], key
    ctx.close()


def test_an_index_sized_for_fewer_tokens_than_the_row_is_refused():
    cfg = inputs.TINY
    ctx, _ = make_pair(cfg, 256, 1, 4)
    index = cs.GramIndex(1, 100, 3)
    ctx.cs_set_match_index(index)
    hd, ld, kvl = i32(np.zeros((1, 128), dtype=np.int32)), i32([20]), i32([19])
    with pytest.raises(cs.CsError) as err:
        ctx.cs_decode_loop(hd, ld, ctx.alloc_kv(), kvl, 3, 4, 10)
    assert err.value.code == cs.CS_ERR_CAPACITY
    assert int(ld[0]) == 20 and int(kvl[0]) == 19
    ctx.cs_set_match_index(None)
    ctx.close()


def test_step_timeline_stamps():
    """cs_set_stamps: one slot per stamped launch, families in launch order, times that never
    run backwards inside a step, and no effect on what the loop computes."""
    cfg = inputs.TINY
    ctx, _ = make_pair(cfg, 1024, 1, 10)
    ctxt, _ = inputs.tiny_context(seed=1)
    max_new = 60
    script = inputs.copy_script(np.random.default_rng(5), ctxt, max_new, 0.6, 5, 30, cfg.vocab, zipf_s=None)
    h = np.zeros((1, 1024), dtype=np.int32); h[0, :512] = ctxt

    def begin(stamps):
        hd, ld, kvl = i32(h), i32([512]), torch.zeros(1, dtype=torch.int32, device="cuda")
        kv = ctx.alloc_kv()
        ctx.cs_prefill(hd, ld, 512, kv, kvl)
        ctx.cs_set_stamps(stamps)
        ctx.cs_loop_begin(hd, ld, kv, kvl, 3, 10, max_new, script=i32(script[None, :]))
        return hd, ld

    stamps = torch.zeros(256, dtype=torch.int64, device="cuda")
    hd, ld = begin(stamps)
    fams = ctx.cs_stamp_layout()
    L = cfg.n_layers
    assert fams == ["other"] * 3 + ["gemm", "attention", "merge", "gemm", "gemm", "gemm"] * L + ["lm_head", "other", "other"]
    ctx.cs_loop_steps(1)
    torch.cuda.synchronize()
    first = stamps[:len(fams)].cpu().numpy()
    assert (first > 0).all() and (np.diff(first) >= 0).all()
    assert (stamps[len(fams):] == 0).all()
    ctx.cs_loop_steps(3)
    torch.cuda.synchronize()
    later = stamps[:len(fams)].cpu().numpy()
    assert (np.diff(later) >= 0).all() and later[0] >= first[-1]
    assert 0 < (later[-1] - later[0]) < 50_000_000          # one tiny step: well under 50 ms
    with pytest.raises(cs.CsError):                         # the graph holds the slots
        ctx.cs_set_stamps(None)
    st, _ = ctx.cs_loop_poll()
    ctx.cs_loop_end()
    with_stamps = hd[0, :int(ld[0])].cpu().tolist()
    hd, ld = begin(None)
    assert ctx.cs_stamp_layout() == []
    ctx.cs_loop_steps(4)
    st2, _ = ctx.cs_loop_poll()
    ctx.cs_loop_end()
    assert hd[0, :int(ld[0])].cpu().tolist() == with_stamps and st == st2
    ctx.close()
