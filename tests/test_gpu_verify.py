"""cs_prefill / cs_verify_step / cs_kv_truncate on the GPU against the CPU oracle
(Sec. 3.2; App. B.2; App. B.3 step 2)."""
import numpy as np
import pytest
import torch

from oracle import copyspec_oracle as O
from paper_2502_08923_b200 import binding as cs, inputs
from helpers import LOGIT_TOL, argmax_consistent, i32, make_pair

pytestmark = pytest.mark.gpu


def _oracle_cache(cfg, batch, max_seq):
    return O.KVCache(cfg, batch, max_seq)


def _kv_close(kv_gpu, cache, b_gpu, b_or, n, tol=2e-2):
    got = kv_gpu[:, :, b_gpu, :, :n, :].float().cpu().numpy()
    want = cache.a[:, :, b_or, :, :n, :]
    return np.abs(got - want).max() <= tol, float(np.abs(got - want).max())


@pytest.mark.parametrize("cfg_name", ["tiny", "gqa", "gqa-tc", "gqa-mma"])
def test_prefill_and_verify_steps(cfg_name, monkeypatch):
    if cfg_name == "tiny":
        cfg = inputs.TINY
    else:   # grouped-query attention with 128-wide heads, odd sizes that leave ragged tiles
        # (the library picks the attention kernel by shape; the suffix forces one of the two
        #  for contexts created from here on, so both are checked on the same case)
        if "-" in cfg_name:
            monkeypatch.setenv("CS_ATTN_KERNEL", cfg_name.split("-")[1])
        cfg = inputs.ModelConfig(n_layers=2, d_model=320, n_heads=4, n_kv_heads=2, head_dim=128, d_ffn=1000,
                                 vocab=1000, rope_theta=500000.0, rms_eps=1e-5)
    B, k, max_seq = 3, 10, 700
    ctx, model = make_pair(cfg, max_seq, B, k, seed=0, gain_jitter=0.1)
    rng = np.random.default_rng(0)
    lens = np.array([512, 300, 77], dtype=np.int32)
    stride = 640
    hist = rng.integers(0, cfg.vocab, size=(B, stride), dtype=np.int32)
    kv = ctx.alloc_kv()
    kv_len = torch.zeros(B, dtype=torch.int32, device="cuda")
    ctx.cs_prefill(i32(hist), i32(lens), int(lens.max()), kv, kv_len)
    assert ctx.cs_sync_status() == 0
    assert kv_len.cpu().tolist() == (lens - 1).tolist()
    cache = _oracle_cache(cfg, B, max_seq)
    for b in range(B):
        model.prefill(hist[b, :lens[b]].tolist(), cache, b)
        ok, err = _kv_close(kv, cache, b, b, lens[b] - 1)
        assert ok, (b, err)

    # three verification steps with different draft lengths and accepted prefixes
    cur = (lens - 1).copy()
    for step, (dls, taus) in enumerate([([10, 4, 0], [3, 4, 0]), ([10, 10, 10], [10, 0, 7]), ([1, 0, 5], [0, 0, 5])]):
        last, draft, _, script = inputs.verify_inputs_with_tau(rng, B, k, taus, cfg.vocab)
        dl = np.array(dls, dtype=np.int32)
        logits = torch.zeros(B, k + 1, cfg.vocab, dtype=torch.float32, device="cuda")
        kvl = i32(cur)
        al, ot, am = ctx.cs_verify_step(i32(last), i32(draft), i32(dl), kv, kvl, target_script=i32(script),
                                        logits_dbg=logits)
        assert ctx.cs_sync_status() == 0
        al, ot, am, lg = al.cpu().numpy(), ot.cpu().numpy(), am.cpu().numpy(), logits.cpu().numpy()
        for b in range(B):
            tau, out, am_o, new_len, lg_o = O.verify_step(model, cache, b, last[b], draft[b, :dl[b]], int(cur[b]),
                                                          script_row=script[b])
            assert al[b] == tau == min(taus[b], dl[b])
            assert ot[b, :tau + 1].tolist() == out and (ot[b, tau + 1:] == -1).all()
            assert np.abs(lg[b, :dl[b] + 1] - lg_o).max() <= LOGIT_TOL
            assert not argmax_consistent(lg_o, am[b, :dl[b] + 1].tolist())
            assert (am[b, dl[b] + 1:] == -1).all()
            assert int(kvl[b]) == new_len
            cur[b] = new_len
            ok, err = _kv_close(kv, cache, b, b, new_len)
            assert ok, (step, b, err)
    ctx.close()


def test_real_mode_single_step_matches_oracle_argmax():
    cfg = inputs.TINY
    ctx, model = make_pair(cfg, 256, 1, 10)
    rng = np.random.default_rng(3)
    hist = rng.integers(0, cfg.vocab, size=(1, 128), dtype=np.int32)
    lens = np.array([100], dtype=np.int32)
    kv = ctx.alloc_kv()
    kv_len = torch.zeros(1, dtype=torch.int32, device="cuda")
    ctx.cs_prefill(i32(hist), i32(lens), 100, kv, kv_len)
    cache = O.KVCache(cfg, 1, 256)
    model.prefill(hist[0, :100].tolist(), cache, 0)
    draft = rng.integers(0, cfg.vocab, size=(1, 10), dtype=np.int32)
    # make the first two draft tokens what the model would say, so tau is 2 in real mode
    t0 = O.verify_step(model, O.KVCache(cfg, 1, 256, data=cache.a.copy()), 0, hist[0, 99], [], 99)[1][0]
    draft[0, 0] = t0
    t1 = O.verify_step(model, O.KVCache(cfg, 1, 256, data=cache.a.copy()), 0, hist[0, 99], [t0], 99)[1][1]
    draft[0, 1] = t1
    tau, out, am_o, new_len, lg_o = O.verify_step(model, cache, 0, hist[0, 99], draft[0], 99)
    assert tau >= 2
    al, ot, am = ctx.cs_verify_step(i32(hist[:, 99]), i32(draft), i32([10]), kv, kv_len)
    assert ctx.cs_sync_status() == 0
    assert not argmax_consistent(lg_o, am[0].cpu().tolist())
    assert int(al[0]) == tau and ot[0, :tau + 1].cpu().tolist() == out
    assert int(kv_len[0]) == new_len
    ctx.close()


def test_capacity_and_truncate_status():
    cfg = inputs.TINY
    ctx, _ = make_pair(cfg, 64, 2, 10)
    kv = ctx.alloc_kv()
    kv_len = i32([60, 10])                     # 60 + 10 + 1 > 64: sequence 0 cannot take the step
    last = i32([1, 2]); draft = i32(np.ones((2, 10))); dl = i32([10, 10])
    al, ot, am = ctx.cs_verify_step(last, draft, dl, kv, kv_len)
    assert ctx.cs_sync_status() == cs.CS_ERR_CAPACITY
    assert int(al[0]) == -1 and int(kv_len[0]) == 60 and int(al[1]) >= 0 and int(kv_len[1]) > 10
    assert ctx.cs_sync_status() == 0           # the word is cleared once read
    # truncation: shrinking is fine, growing is refused and leaves the length alone
    kv_len = i32([30, 10])
    ctx.cs_kv_truncate(kv_len, i32([12, 10]))
    assert ctx.cs_sync_status() == 0 and kv_len.cpu().tolist() == [12, 10]
    ctx.cs_kv_truncate(kv_len, i32([5, 11]))
    assert ctx.cs_sync_status() == cs.CS_ERR_ARG and kv_len.cpu().tolist() == [5, 10]
    with pytest.raises(cs.CsError):
        ctx.cs_verify_step(i32([1, 2, 3]), i32(np.ones((3, 10))), i32([1, 1, 1]), kv, i32([1, 1, 1]))  # B > max_batch
    ctx.close()


def test_truncated_rows_do_not_leak_into_the_next_step():
    """App. B.2: after a rejection the rejected rows' K/V are dead; the next step must give
    the same logits as an oracle that never saw them."""
    cfg = inputs.TINY
    ctx, model = make_pair(cfg, 128, 1, 10)
    rng = np.random.default_rng(5)
    hist = rng.integers(0, cfg.vocab, size=(1, 64), dtype=np.int32)
    kv = ctx.alloc_kv(); kv_len = torch.zeros(1, dtype=torch.int32, device="cuda")
    ctx.cs_prefill(i32(hist), i32([41]), 41, kv, kv_len)
    cache = O.KVCache(cfg, 1, 128); model.prefill(hist[0, :41].tolist(), cache, 0)
    last, draft, dl, script = inputs.verify_inputs_with_tau(rng, 1, 10, [2], cfg.vocab)
    ctx.cs_verify_step(i32(last), i32(draft), i32(dl), kv, kv_len, target_script=i32(script))
    tau, out, _, new_len, _ = O.verify_step(model, cache, 0, last[0], draft[0], 40, script_row=script[0])
    assert int(kv_len[0]) == new_len == 43
    logits = torch.zeros(1, 11, cfg.vocab, dtype=torch.float32, device="cuda")
    nxt = np.array([out[-1]], dtype=np.int32)
    ctx.cs_verify_step(i32(nxt), i32(draft), i32([0]), kv, kv_len, logits_dbg=logits)
    clean = O.KVCache(cfg, 1, 128)            # an oracle that only ever saw the accepted tokens
    seq = hist[0, :40].tolist() + [int(last[0])] + out
    model.prefill(seq, clean, 0)
    lg = model.forward_block([seq[-1]], len(seq) - 1, clean, 0)
    assert np.abs(logits[0, :1].cpu().numpy() - lg).max() <= LOGIT_TOL
    ctx.close()


@pytest.mark.parametrize("k", [50, 100])
def test_wide_block_logits(k):
    """One verification step with a 51- / 101-row block on the 128-wide-head configuration:
    102 query rows per KV head still go to the tcgen05 attention kernel, 202 to the mma.sync
    one; logits and the appended K/V rows against the oracle."""
    cfg = inputs.ModelConfig(n_layers=2, d_model=320, n_heads=4, n_kv_heads=2, head_dim=128, d_ffn=1000,
                             vocab=1000, rope_theta=500000.0, rms_eps=1e-5)
    max_seq = 512
    ctx, model = make_pair(cfg, max_seq, 1, k, seed=2, gain_jitter=0.1)
    rng = np.random.default_rng(4)
    n0 = 301
    hist = rng.integers(0, cfg.vocab, size=(1, 320), dtype=np.int32)
    kv = ctx.alloc_kv()
    kv_len = torch.zeros(1, dtype=torch.int32, device="cuda")
    ctx.cs_prefill(i32(hist), i32([n0]), n0, kv, kv_len)
    cache = O.KVCache(cfg, 1, max_seq)
    model.prefill(hist[0, :n0].tolist(), cache, 0)
    last, draft, dl, script = inputs.verify_inputs_with_tau(rng, 1, k, [k - 7], cfg.vocab)
    logits = torch.zeros(1, k + 1, cfg.vocab, dtype=torch.float32, device="cuda")
    al, ot, am = ctx.cs_verify_step(i32(last), i32(draft), i32(dl), kv, kv_len, target_script=i32(script), logits_dbg=logits)
    assert ctx.cs_sync_status() == 0
    tau, out, am_o, new_len, lg_o = O.verify_step(model, cache, 0, last[0], draft[0], n0 - 1, script_row=script[0])
    assert int(al[0]) == tau == k - 7 and ot[0, :tau + 1].cpu().tolist() == out
    assert np.abs(logits[0].cpu().numpy() - lg_o).max() <= LOGIT_TOL
    assert not argmax_consistent(lg_o, am[0].cpu().tolist())
    assert int(kv_len[0]) == new_len
    ok, err = _kv_close(kv, cache, 0, 0, new_len)
    assert ok, err
    ctx.close()
