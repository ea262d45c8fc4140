"""Numerics of the verification forward (Sec. 3.2) at the block heights and cache depths of the
long-context and multi-turn workloads: a 2-layer slice of the 8B-class shape (d 4096, 32 / 8
heads of 128, FFN 14,336; a 4,096-row head keeps the oracle quick) over synthetic caches of
30,720 and 8,192 keys, plus small-width models that put every launch variant of the tcgen05
attention kernels (up to 48, 49-96, 97-128 padded query rows, and blocks cut into row groups)
on key slices of at least five tiles per CTA; every case runs once with the kernel the library
picks for such key ranges (keys and head dims as the M dimension) and once with the other one
forced (query rows as M).  Logits, greedy tokens, acceptance and the
block's K/V rows are compared with the oracle element by element.  The second layer's K/V rows
and the logits depend on the first layer's attention output, so a wrong key tile, ring slot or
mask anywhere in the slice fails them."""
import numpy as np
import pytest
import torch

from oracle import copyspec_oracle as O
from paper_2502_08923_b200 import binding as cs, inputs
from helpers import LOGIT_TOL, argmax_consistent, i32

pytestmark = pytest.mark.gpu

GAMMA = 3
SLICE8B = inputs.ModelConfig(n_layers=2, d_model=4096, n_heads=32, n_kv_heads=8, head_dim=128, d_ffn=14336,
                             vocab=4096, rope_theta=500000.0, rms_eps=1e-5)
NARROW = inputs.ModelConfig(n_layers=2, d_model=512, n_heads=8, n_kv_heads=4, head_dim=128, d_ffn=1024,
                            vocab=1024, rope_theta=500000.0, rms_eps=1e-5)


@pytest.fixture(autouse=True, params=["default", "tc"])
def attention_kernel(request, monkeypatch):
    """Every case runs with the attention kernel the library picks for its key range (keys and head
    dims as M at these depths) and with the query-rows-as-M kernel forced."""
    if request.param != "default":
        monkeypatch.setenv("CS_ATTN_KERNEL", request.param)
    return request.param


@pytest.fixture(scope="module")
def slice8b():
    w = inputs.make_weights(SLICE8B, seed=3, gain_jitter=0.05)
    return w, inputs.weights_to(w, "cuda"), O.Model(SLICE8B, w, contract=True)


@pytest.fixture(scope="module")
def narrow():
    w = inputs.make_weights(NARROW, seed=4, gain_jitter=0.05)
    return w, inputs.weights_to(w, "cuda"), O.Model(NARROW, w, contract=True)


def oracle_block(model, cfg, kv_dev, b, kv_len, block):
    """Oracle forward of one sequence's block against the first kv_len cached positions of
    sequence b of the device cache.  Returns (logits [R][V], oracle cache)."""
    cache = O.KVCache(cfg, 1, kv_len + len(block), dtype=np.float32)
    cache.a[:, :, 0, :, :kv_len, :] = kv_dev[:, :, b, :, :kv_len, :].float().cpu().numpy()
    return model.forward_block([int(t) for t in block], kv_len, cache, 0), cache


def check_rows(cfg, model, kv_before, kv_after, b, kv_len, block, draft, gpu_logits, gpu_ids, gpu_tau):
    """One sequence of a verification step against the oracle.  `gpu_logits` may be None
    (the generation loop writes none); `gpu_tau` None skips the acceptance check."""
    lg, cache = oracle_block(model, cfg, kv_before, b, kv_len, block)
    R = len(block)
    if gpu_logits is not None:
        err = float(np.abs(gpu_logits[:R] - lg).max())
        assert err <= LOGIT_TOL, (b, err)
    ids = [int(t) for t in gpu_ids[:R]]
    assert not argmax_consistent(lg, ids), b
    assert all(int(t) == -1 for t in gpu_ids[R:]), b
    if gpu_tau is not None:
        # acceptance follows the greedy tokens; they may differ from the oracle's only inside its margin
        assert int(gpu_tau) == O.accept_length([int(t) for t in draft], ids), b
    # the block's K/V rows of both layers, within bf16 resolution of the oracle's stored rows
    new = kv_after[:, :, b, :, kv_len:kv_len + R, :].float().cpu().numpy()
    want = cache.a[:, :, 0, :, kv_len:kv_len + R, :]
    assert np.abs(new - want).max() <= 2e-2 * max(1.0, float(np.abs(want).max())), b


def run_verify(cfg, w_gpu, model, B, k, kv_lens, draft_lens, seed, max_seq=None):
    rng = np.random.default_rng(seed)
    max_seq = max_seq or (max(kv_lens) + k + 1 + 64)
    ctx = cs.Context(cfg, w_gpu, max_seq=max_seq, max_batch=B, k_max=k)
    kv = inputs.synthetic_kv(cfg, B, max_seq, max(kv_lens), seed=seed, device="cuda")
    last = rng.integers(0, cfg.vocab, size=B)
    draft = rng.integers(0, cfg.vocab, size=(B, k))
    kv_run = kv.clone()
    kvl = i32(kv_lens)
    logits = torch.full((B, k + 1, cfg.vocab), float("nan"), dtype=torch.float32, device="cuda")
    al, ot, am = ctx.cs_verify_step(i32(last), i32(draft), i32(draft_lens), kv_run, kvl, logits_dbg=logits)
    assert ctx.cs_sync_status() == 0
    al, am, lg = al.cpu().tolist(), am.cpu().numpy(), logits.cpu().numpy()
    for b in range(B):
        dl = int(draft_lens[b])
        block = [int(last[b])] + [int(t) for t in draft[b, :dl]]
        check_rows(cfg, model, kv, kv_run, b, int(kv_lens[b]), block, draft[b, :dl], lg[b], am[b], al[b])
        assert int(kvl[b]) == int(kv_lens[b]) + al[b] + 1
    ctx.close()


def planted_history(rng, n, vocab, k):
    """n random tokens whose last GAMMA tokens repeat an earlier place followed by >= k tokens."""
    h = rng.integers(0, vocab, size=n, dtype=np.int32)
    src = int(rng.integers(n // 4, n // 2))
    h[n - GAMMA:] = h[src:src + GAMMA]
    return h


def run_loop_first_step(cfg, w_gpu, model, B, k, hist_lens, seed):
    """The first step of the generation loop (real mode): its launches are the ones bench.py
    times - step graph, cached key tiles requested before the dependency wait."""
    rng = np.random.default_rng(seed)
    max_new = 2 * (k + 1)
    n_max = max(hist_lens)
    stride = (n_max + max_new + 67) // 4 * 4
    max_seq = n_max + max_new + k + 64
    ctx = cs.Context(cfg, w_gpu, max_seq=max_seq, max_batch=B, k_max=k)
    kv = inputs.synthetic_kv(cfg, B, max_seq, n_max - 1, seed=seed, device="cuda")
    h = np.zeros((B, stride), dtype=np.int32)
    for b in range(B):
        h[b, :hist_lens[b]] = planted_history(rng, hist_lens[b], cfg.vocab, k)
    hd, ld, kvl = i32(h), i32(hist_lens), i32(np.asarray(hist_lens) - 1)
    kv_run = kv.clone()
    ctx.cs_loop_begin(hd, ld, kv_run, kvl, GAMMA, k, max_new)
    ctx.cs_loop_steps(1)
    st, _ = ctx.cs_loop_poll()
    mp, dl, al, ot, am = (t.numpy() for t in ctx.cs_loop_last_step())
    ctx.cs_loop_end()
    assert st["steps"] == B and st["attempts"] == B
    for b in range(B):
        n = int(hist_lens[b])
        p0 = O.find_match(h[b], n, GAMMA, O.LATEST)
        draft = O.gather_draft(h[b], n, p0, GAMMA, k)
        assert int(mp[b]) == p0 and int(dl[b]) == len(draft) == k
        block = [int(h[b, n - 1])] + draft
        check_rows(cfg, model, kv, kv_run, b, n - 1, block, draft, None, am[b], al[b])
        tau = int(al[b])
        assert ot[b, :tau + 1].tolist() == am[b, :tau + 1].tolist() and all(ot[b, tau + 1:] == -1)
        assert int(ld[b]) == n + tau + 1 and int(kvl[b]) == n + tau
        assert hd[b, n:n + tau + 1].cpu().tolist() == ot[b, :tau + 1].tolist()
    ctx.close()


# ------------------------------------------------------------------ 8B-shape slice, deep caches
def test_long_context_batch1_k10_verify_step(slice8b):
    """30,720 cached keys, 11-row block: 44 query rows per KV head, one K/V stage, two CTAs per
    SM, six to seven key tiles per CTA."""
    _, w_gpu, model = slice8b
    run_verify(SLICE8B, w_gpu, model, 1, 10, [30720], [10], seed=11)


def test_long_context_batch1_k10_inside_the_loop(slice8b):
    _, w_gpu, model = slice8b
    run_loop_first_step(SLICE8B, w_gpu, model, 1, 10, [30721], seed=12)


def test_long_context_batch8_k20_verify_step(slice8b):
    """168-row block (84 query rows per KV head: two K/V stages, one CTA per SM, two key slices
    of about 120 tiles each), ragged cache depths and draft lengths."""
    _, w_gpu, model = slice8b
    kv_lens = [30720, 30000, 29999, 25001, 30720, 12345, 30719, 28672]
    draft_lens = [20, 20, 7, 20, 0, 20, 13, 20]
    run_verify(SLICE8B, w_gpu, model, 8, 20, kv_lens, draft_lens, seed=13)


def test_long_context_batch8_k20_inside_the_loop(slice8b):
    _, w_gpu, model = slice8b
    run_loop_first_step(SLICE8B, w_gpu, model, 8, 20, [30721, 30001, 29000, 30721, 27777, 30500, 30721, 26000], seed=14)


def test_multi_turn_batch16_k10_verify_step(slice8b):
    """176-row block over 8,192-key caches of ragged depth: about 32 key tiles per CTA."""
    _, w_gpu, model = slice8b
    rng = np.random.default_rng(15)
    kv_lens = [8192] + [int(x) for x in rng.integers(5000, 8193, size=15)]
    draft_lens = [10] * 8 + [int(x) for x in rng.integers(0, 11, size=8)]
    run_verify(SLICE8B, w_gpu, model, 16, 10, kv_lens, draft_lens, seed=15)


def test_multi_turn_batch16_k10_inside_the_loop(slice8b):
    _, w_gpu, model = slice8b
    rng = np.random.default_rng(16)
    run_loop_first_step(SLICE8B, w_gpu, model, 16, 10, [8193] + [int(x) for x in rng.integers(6000, 8194, size=15)], seed=16)


# ------------------------------------------------------------------ every attention launch variant, >= 5 tiles per CTA
@pytest.mark.parametrize("B,k,kv_max,label", [
    (16, 10, 3100, "22 query rows: one stage, two CTAs per SM, 4 key slices"),
    (7, 32, 4000, "66 query rows: two stages, one CTA per SM, 5 key slices"),
    (4, 59, 6500, "120 query rows: one stage, one CTA per SM, 9 key slices"),
    (2, 100, 6500, "202 query rows in two row groups of 102, 9 key slices"),
])
def test_attention_variants_over_many_key_tiles(narrow, B, k, kv_max, label):
    _, w_gpu, model = narrow
    rng = np.random.default_rng(B * 1000 + k)
    kv_lens = [kv_max] + [int(x) for x in rng.integers(kv_max * 7 // 10, kv_max + 1, size=B - 1)]
    draft_lens = [k] + [int(x) for x in rng.integers(0, k + 1, size=B - 1)]
    run_verify(NARROW, w_gpu, model, B, k, kv_lens, draft_lens, seed=B * 1000 + k)


@pytest.mark.parametrize("seed", [31, 32, 33])
def test_one_column_group_fully_masked(narrow, seed):
    """Short drafts in most sequences: the upper half of the query columns of their CTAs is masked
    throughout, so that half of the softmax threads finishes its tiles much sooner than the half that
    works out maxima - the two halves must still hand every tile over together."""
    _, w_gpu, model = narrow
    rng = np.random.default_rng(seed)
    kv_lens = [3100] + [int(x) for x in rng.integers(2200, 3101, size=15)]
    draft_lens = [10] + [int(x) for x in rng.integers(0, 4, size=15)]
    run_verify(NARROW, w_gpu, model, 16, 10, kv_lens, draft_lens, seed=seed)


def test_attention_variants_inside_the_loop(narrow):
    """The same variants with the step graph and the early tile requests of the loop."""
    _, w_gpu, model = narrow
    run_loop_first_step(NARROW, w_gpu, model, 16, 10, [3101] + [2500 + 37 * b for b in range(15)], seed=21)
    run_loop_first_step(NARROW, w_gpu, model, 7, 32, [4001] + [3000 + 111 * b for b in range(6)], seed=22)
