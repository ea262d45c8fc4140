"""Shared set-up of the GPU parity tests: the same seeded weights go to the CUDA library
(bf16 on the device) and to the CPU oracle."""
import numpy as np
import torch

from oracle import copyspec_oracle as O
from paper_2502_08923_b200 import binding as cs, inputs

LOGIT_TOL = 2e-2     # max |logit difference| with bf16 operands and fp32 accumulation


def make_pair(cfg, max_seq, max_batch, k_max, seed=0, gain_jitter=0.0, weights=None):
    w_cpu = weights if weights is not None else inputs.make_weights(cfg, seed=seed, gain_jitter=gain_jitter)
    w_gpu = inputs.weights_to(w_cpu, "cuda")
    ctx = cs.Context(cfg, w_gpu, max_seq=max_seq, max_batch=max_batch, k_max=k_max)
    model = O.Model(cfg, w_cpu, contract=True)
    return ctx, model


def i32(a, device="cuda"):
    return torch.as_tensor(np.ascontiguousarray(a), dtype=torch.int32).to(device)


def argmax_consistent(oracle_logits, gpu_ids, tol=LOGIT_TOL):
    """GPU argmax must equal the oracle's unless the oracle's own margin over the GPU's
    choice is below the logit tolerance."""
    bad = []
    for r, gid in enumerate(gpu_ids):
        row = oracle_logits[r]
        oid = int(np.argmax(row))
        if gid != oid and not (row[oid] - row[gid] < tol):
            bad.append((r, gid, oid, float(row[oid] - row[gid])))
    return bad


def greedy_margins(model, cfg, prompt, generated):
    """Teacher-forced check of a greedy continuation: for every generated token, how far its
    oracle logit lies below the oracle's best logit at that position (0 = the oracle's own
    choice).  A correct greedy decoder may only deviate where this margin is below the
    logit tolerance."""
    seq = [int(t) for t in prompt] + [int(t) for t in generated]
    cache = O.KVCache(cfg, 1, len(seq) + 1)
    logits = model.forward_block(seq[:-1], 0, cache, 0)
    n0 = len(prompt)
    return [float(logits[n0 - 1 + j].max() - logits[n0 - 1 + j][tok]) for j, tok in enumerate(generated)]


COUNTERS = ("steps", "attempts", "accepted", "emitted", "no_match")


def counters_for_streams(hists, streams, gamma, k, policy=O.LATEST):
    """What the loop's statistics must be, given the token stream each sequence actually
    emitted: with the targets fixed to those tokens, matches, drafts and accepted lengths are
    integer functions of history and stream, which the model-free simulator replays.  This
    checks the loop's bookkeeping on its own output whether or not a near-tie made that output
    differ from the oracle's (the tokens themselves are pinned by greedy_margins)."""
    tot = O.new_stats()
    for hist, gen in zip(hists, streams):
        if len(gen) == 0:
            continue
        _, st, h = O.scripted_simulator(hist, np.asarray(gen, dtype=np.int64), gamma, k, policy, len(gen))
        assert h == [int(t) for t in hist] + [int(t) for t in gen]
        for key in COUNTERS:
            tot[key] += st[key]
        for i, v in enumerate(st["tau_hist"]):
            tot["tau_hist"][i] += v
    return tot


# ------------------------------------------------------------------ write canaries around a KV cache
GUARD = 1 << 16     # bf16 elements on either side of the cache
PATTERN = -1232.0   # exactly representable in bf16


def guarded_kv(cfg, B, max_seq, fill_len, seed, device="cuda"):
    """(whole buffer, cache view inside it): the cache holds N(0,1) up to fill_len and a pattern behind
    it, the guard bands hold the pattern."""
    n = cfg.n_layers * 2 * B * cfg.n_kv_heads * max_seq * cfg.head_dim
    buf = torch.full((n + 2 * GUARD,), PATTERN, dtype=torch.bfloat16, device=device)
    kv = buf[GUARD:GUARD + n].view(cfg.n_layers, 2, B, cfg.n_kv_heads, max_seq, cfg.head_dim)
    kv[:, :, :, :, :fill_len, :] = inputs.synthetic_kv(cfg, B, max_seq, fill_len, seed=seed, device=device)[:, :, :, :, :fill_len, :]
    return buf, kv


def assert_only_rows_written(buf, kv, before, written):
    """`written[b]` = (first, count): the only positions of sequence b that may differ from `before`."""
    assert torch.all(buf[:GUARD] == PATTERN) and torch.all(buf[-GUARD:] == PATTERN), "guard band of the cache overwritten"
    same = (kv == before)
    for b, (first, count) in enumerate(written):
        same[:, :, b, :, first:first + count, :] = True
    bad = torch.nonzero(~same)
    assert bad.numel() == 0, f"cache written outside the block's rows, first at (layer, k/v, seq, head, pos, dim) = {bad[0].tolist()}"
    for b, (first, count) in enumerate(written):
        if count:
            rows = kv[:, :, b, :, first:first + count, :]
            assert torch.isfinite(rows.float()).all() and not torch.all(rows == PATTERN), b


