"""Seeded synthetic inputs for the copy-and-verify decode step.

This module only *draws* data: model shapes, random weights, token histories with
planted repeats, scripted continuations and synthetic KV fills.  It holds none of the
method's arithmetic (no search, no forward, no acceptance), so both the CUDA path and
the CPU oracle may be fed from it without sharing any logic.

Workload shapes follow the paper's settings: histories are prompts plus earlier turns
plus generated text (Sec. 3.1), continuations re-emit verbatim spans of the context
(extractive summaries, Sec. 4.2) or an earlier answer with edits (MT-Redundant,
Sec. 4.3).  No dataset item is reproduced; everything is drawn from seeded generators.
"""
from __future__ import annotations

from dataclasses import dataclass, asdict

import numpy as np
import torch


# --------------------------------------------------------------------------- shapes
@dataclass(frozen=True)
class ModelConfig:
    n_layers: int
    d_model: int
    n_heads: int
    n_kv_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    rope_theta: float = 10000.0
    rms_eps: float = 1e-5

    @property
    def q_dim(self) -> int:
        return self.n_heads * self.head_dim

    @property
    def kv_dim(self) -> int:
        return self.n_kv_heads * self.head_dim

    @property
    def qkv_dim(self) -> int:
        return self.q_dim + 2 * self.kv_dim

    def params_per_layer(self) -> int:
        d = self.d_model
        return d * self.qkv_dim + self.q_dim * d + 3 * d * self.d_ffn

    def streamed_params(self) -> int:
        """Weight elements one verification forward reads (layers + LM head)."""
        return self.n_layers * self.params_per_layer() + self.vocab * self.d_model

    def kv_bytes_per_token(self) -> int:
        return self.n_layers * 2 * self.kv_dim * 2

    def as_dict(self) -> dict:
        return asdict(self)


#: small decoder the CPU oracle finishes in seconds
TINY = ModelConfig(n_layers=2, d_model=256, n_heads=8, n_kv_heads=8, head_dim=32,
                   d_ffn=1024, vocab=4096, rope_theta=10000.0, rms_eps=1e-5)

#: 8B-class shape (GQA 32/8, head_dim 128, SwiGLU 14336, vocab 128256)
LLAMA8B = ModelConfig(n_layers=32, d_model=4096, n_heads=32, n_kv_heads=8, head_dim=128,
                      d_ffn=14336, vocab=128256, rope_theta=500000.0, rms_eps=1e-5)


def sliced(cfg: ModelConfig, n_layers: int) -> ModelConfig:
    """The same shape with fewer layers (bounded CPU samples of a big model)."""
    d = cfg.as_dict()
    d["n_layers"] = n_layers
    return ModelConfig(**d)


# -------------------------------------------------------------------------- weights
def make_weights(cfg: ModelConfig, seed: int = 0, device: str = "cpu",
                 gain_jitter: float = 0.0) -> dict:
    """Random-init decoder weights: fp32 N(0, 0.02) drawn from `seed`, rounded once to
    bf16; those rounded values are what every consumer sees.  Norm gains are 1.0, or
    1 + gain_jitter * N(0,1) when a test wants the gain multiply to matter.

    Layout (all row-major `[out][in]`, bf16):
      embed [V][d], lm_head [V][d], final_norm [d], and per layer
      attn_norm [d], wqkv [(H + 2 Hkv) Dh][d] (q rows, then k rows, then v rows),
      wo [d][H Dh], ffn_norm [d], w_gate_up [2 F][d] (gate rows, then up rows),
      w_down [d][F].
    """
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)

    def normal(*shape):
        w = torch.empty(*shape, dtype=torch.float32, device=device)
        w.normal_(0.0, 0.02, generator=gen)
        return w.to(torch.bfloat16)

    def gain(n):
        g = torch.ones(n, dtype=torch.float32, device=device)
        if gain_jitter:
            g += gain_jitter * torch.empty(n, dtype=torch.float32, device=device).normal_(
                0.0, 1.0, generator=gen)
        return g.to(torch.bfloat16)

    d, f = cfg.d_model, cfg.d_ffn
    w = {"embed": normal(cfg.vocab, d), "lm_head": normal(cfg.vocab, d),
         "final_norm": gain(d), "layers": []}
    for _ in range(cfg.n_layers):
        w["layers"].append({
            "attn_norm": gain(d),
            "wqkv": normal(cfg.qkv_dim, d),
            "wo": normal(d, cfg.q_dim),
            "ffn_norm": gain(d),
            "w_gate_up": normal(2 * f, d),
            "w_down": normal(d, f),
        })
    return w


def weights_to(w: dict, device: str) -> dict:
    out = {k: (v.to(device) if torch.is_tensor(v) else v) for k, v in w.items()
           if k != "layers"}
    out["layers"] = [{k: v.to(device) for k, v in lay.items()} for lay in w["layers"]]
    return out


def synthetic_kv(cfg: ModelConfig, batch: int, max_seq: int, fill_len: int, seed: int = 0,
                 device: str = "cpu") -> torch.Tensor:
    """A KV cache `[layer][K|V][B][Hkv][max_seq][Dh]` (bf16) whose first `fill_len`
    positions hold N(0,1) values standing in for an already ingested context; the rest
    is zero."""
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    kv = torch.zeros(cfg.n_layers, 2, batch, cfg.n_kv_heads, max_seq, cfg.head_dim,
                     dtype=torch.bfloat16, device=device)
    if fill_len > 0:
        for layer in range(cfg.n_layers):
            blk = torch.empty(2, batch, cfg.n_kv_heads, fill_len, cfg.head_dim,
                              dtype=torch.float32, device=device)
            blk.normal_(0.0, 1.0, generator=gen)
            kv[layer, :, :, :, :fill_len, :] = blk.to(torch.bfloat16)
    return kv


# --------------------------------------------------------------------------- tokens
def zipf_tokens(rng: np.random.Generator, n: int, vocab: int, s: float = 1.1) -> np.ndarray:
    """`n` ids with P(id = r - 1) proportional to r**-s over ranks 1..vocab
    (inverse-CDF sampling)."""
    ranks = np.arange(1, vocab + 1, dtype=np.float64)
    cdf = np.cumsum(ranks ** (-s))
    cdf /= cdf[-1]
    u = rng.random(n)
    ids = np.searchsorted(cdf, u, side="left")
    return np.minimum(ids, vocab - 1).astype(np.int32)


def plant_repeats(rng: np.random.Generator, h: np.ndarray, n_spans: int, lo: int, hi: int,
                  limit: int | None = None) -> list:
    """Copy `n_spans` spans (length uniform in [lo, hi]) of `h[:limit]` verbatim to a
    later, non-overlapping place, in place.  Sources lie in the first half, copies in
    the second half, each on its own slot, so no span overwrites another.  Returns
    `[(src, dst, length), ...]`."""
    limit = len(h) if limit is None else limit
    half = limit // 2
    slot = half // n_spans
    if slot < hi:
        raise ValueError("history too short for the requested spans")
    spans = []
    order = rng.permutation(n_spans)
    for i in range(n_spans):
        length = int(rng.integers(lo, hi + 1))
        src = i * slot + int(rng.integers(0, slot - length + 1))
        j = int(order[i])
        dst = half + j * slot + int(rng.integers(0, slot - length + 1))
        h[dst:dst + length] = h[src:src + length]
        spans.append((src, dst, length))
    return spans


def tiny_context(seed: int = 1, n: int = 512, vocab: int = 4096, n_spans: int = 4,
                 span: int = 40) -> tuple:
    """512 uniform random ids with 4 verbatim 40-token spans repeated once later."""
    rng = np.random.default_rng(seed)
    h = rng.integers(0, vocab, size=n, dtype=np.int32)
    spans = plant_repeats(rng, h, n_spans, span, span)
    return h, spans


def copy_script(rng: np.random.Generator, context: np.ndarray, length: int,
                copy_frac: float, span_lo: int, span_hi: int, vocab: int,
                zipf_s: float | None = 1.1) -> np.ndarray:
    """A scripted continuation of `length` tokens of which about `copy_frac` are
    verbatim spans (length uniform in [span_lo, span_hi]) lifted from random offsets
    of `context`; the rest are fresh tokens (Zipf, or uniform when zipf_s is None)."""
    out = []
    total = 0
    copied = 0
    while total < length:
        want_copy = copied < copy_frac * (total + 1)
        if want_copy:
            ln = int(rng.integers(span_lo, span_hi + 1))
            ln = min(ln, len(context) - 1)
            off = int(rng.integers(0, len(context) - ln))
            seg = context[off:off + ln]
            copied += ln
        else:
            mean_fresh = max(1.0, 0.5 * (span_lo + span_hi) * (1 - copy_frac) / max(copy_frac, 1e-6))
            ln = max(1, int(rng.integers(1, int(2 * mean_fresh) + 1)))
            if zipf_s is None:
                seg = rng.integers(0, vocab, size=ln, dtype=np.int32)
            else:
                seg = zipf_tokens(rng, ln, vocab, zipf_s)
        out.append(np.asarray(seg, dtype=np.int32))
        total += ln
    return np.concatenate(out)[:length].astype(np.int32)


def match_search_histories(batch: int = 64, n: int = 32768, vocab: int = 128256,
                           seed: int = 2, n_spans: int = 16, span_lo: int = 64,
                           span_hi: int = 512, gamma_max: int = 5) -> tuple:
    """Histories for the search-only workload.  Ids are Zipf(1.1) over `vocab - 1`
    ranks (the last id is reserved); each history has `n_spans` planted repeats.  The
    tail differs by `b % 4`: 0 and 1 end a few tokens (>= gamma_max) into a replay of
    a planted span, 2 ends in plain Zipf text (chance matches on frequent ids), 3 ends
    with the reserved id (no match possible).  Returns `(hist [B][n] int32,
    kinds [B], spans per history)`."""
    hist = np.empty((batch, n), dtype=np.int32)
    kinds = np.empty(batch, dtype=np.int32)
    all_spans = []
    for b in range(batch):
        rng = np.random.default_rng(seed + b)
        h = zipf_tokens(rng, n, vocab - 1, 1.1)
        tail_room = 64
        spans = plant_repeats(rng, h, n_spans, span_lo, span_hi, limit=n - tail_room)
        kind = b % 4
        if kind in (0, 1):
            src, _, length = spans[int(rng.integers(0, n_spans))]
            t = gamma_max + int(rng.integers(0, 20))
            t = min(t, length - 1, tail_room)
            h[n - t:] = h[src:src + t]
        elif kind == 3:
            h[n - 1] = vocab - 1
        hist[b] = h
        kinds[b] = kind
        all_spans.append(spans)
    return hist, kinds, all_spans


def long_context_case(seed: int, context_len: int = 30720, script_len: int = 2048,
                      vocab: int = 128256, copy_frac: float = 0.6, span_lo: int = 20,
                      span_hi: int = 200) -> tuple:
    """Long Zipf context plus a scripted continuation, 60 % of which is verbatim spans
    of 20-200 tokens lifted from the context."""
    rng = np.random.default_rng(seed)
    ctx = zipf_tokens(rng, context_len, vocab, 1.1)
    script = copy_script(rng, ctx, script_len, copy_frac, span_lo, span_hi, vocab)
    return ctx, script


def multi_turn_case(seed: int, history_len: int = 8192, answer_len: int = 1024,
                    script_len: int = 2048, vocab: int = 128256, sub_rate: float = 0.05,
                    ins_rate: float = 0.03) -> tuple:
    """An 8,192-token history holding a 1,024-token first-turn answer (not at the
    tail), and a scripted second turn that re-emits that answer with 5 % token
    substitutions and 3 % single-token insertions, then fresh text."""
    rng = np.random.default_rng(seed)
    h = zipf_tokens(rng, history_len, vocab, 1.1)
    off = int(rng.integers(history_len // 4, history_len - answer_len - 64))
    answer = h[off:off + answer_len]
    out = []
    for tok in answer:
        if rng.random() < ins_rate:
            out.append(int(zipf_tokens(rng, 1, vocab, 1.1)[0]))
        if rng.random() < sub_rate:
            out.append(int(zipf_tokens(rng, 1, vocab, 1.1)[0]))
        else:
            out.append(int(tok))
    out = np.asarray(out, dtype=np.int32)
    if len(out) < script_len:
        out = np.concatenate([out, zipf_tokens(rng, script_len - len(out), vocab, 1.1)])
    return h, out[:script_len].astype(np.int32), off


def verify_inputs_with_tau(rng: np.random.Generator, batch: int, k: int, taus, vocab: int) -> tuple:
    """Draft blocks and target scripts for one stand-alone verification step such that
    sequence b's longest agreeing prefix is exactly `taus[b]`: the first taus[b] draft
    tokens equal the script, the next one differs.  Returns `(last_tok [B], draft
    [B][k], draft_len [B], script [B][k+1])`, all int32."""
    taus = np.asarray(taus, dtype=np.int64).reshape(batch)
    script = rng.integers(0, vocab, size=(batch, k + 1), dtype=np.int32)
    draft = script[:, :k].copy()
    for b in range(batch):
        t = int(taus[b])
        if t < k:
            draft[b, t] = (script[b, t] + 1 + int(rng.integers(0, vocab - 1))) % vocab
            draft[b, t + 1:] = rng.integers(0, vocab, size=k - t - 1, dtype=np.int32)
    last_tok = rng.integers(0, vocab, size=batch, dtype=np.int32)
    draft_len = np.full(batch, k, dtype=np.int32)
    return last_tok, draft.astype(np.int32), draft_len, script


def tau_controlled_case(rng: np.random.Generator, taus, gamma: int = 3, k: int = 10,
                        context_len: int = 4096, vocab: int = 128256) -> tuple:
    """A history and a scripted continuation on which every decode step finds a match and
    accepts exactly `taus[i]` draft tokens at step i (0 <= taus[i] <= k).

    The context holds one "path" of distinct tokens per step.  A path starts with the two
    tokens that end the previous step's accepted run, so when the script leaves the path
    being copied (rejecting draft token taus[i]) the extra token it emits completes the
    opening gamma-gram of the next path, which is the only earlier occurrence of the new
    suffix.  taus[i] == k means the whole draft is accepted and the same path goes on.
    All tokens are distinct ids, so no chance matches occur.  Returns `(hist, script)`:
    hist has `context_len + 1` tokens (so the KV cache holds `context_len` positions
    before the first step), script has sum(taus) + len(taus) tokens.  Only gamma == 3."""
    assert gamma == 3
    taus = [int(t) for t in taus]
    ids = rng.permutation(vocab).astype(np.int32)
    nxt = [0]

    def fresh(n):
        out = ids[nxt[0]:nxt[0] + n].tolist()
        nxt[0] += n
        if nxt[0] > vocab:
            raise ValueError("vocabulary too small for this many steps")
        return out

    paths = [fresh(3)]
    script = []
    tail = list(paths[0][:3])          # last tokens of history + script so far
    cur, pos = 0, 3
    for tau in taus:
        need = pos + 2 * k + 2 - len(paths[cur])
        if need > 0:
            paths[cur].extend(fresh(need))
        if tau >= k:
            seg = paths[cur][pos:pos + k + 1]
            script.extend(seg)
            tail = (tail + seg)[-3:]
            pos += k + 1
        else:
            seg = paths[cur][pos:pos + tau]
            script.extend(seg)
            tail = (tail + seg)[-3:]
            new = [tail[-2], tail[-1]] + fresh(1)
            script.append(new[2])
            tail = (tail + [new[2]])[-3:]
            paths.append(new)
            cur, pos = len(paths) - 1, 3
    need = pos + 2 * k + 2 - len(paths[cur])
    if need > 0:
        paths[cur].extend(fresh(need))
    body = [t for p in paths for t in p]
    room = context_len + 1 - 3 - len(body)
    if room < 0:
        raise ValueError(f"context_len {context_len} too small: the paths need {len(body) + 2} tokens")
    hist = fresh(room) + body + list(paths[0][:3])
    return np.asarray(hist, dtype=np.int32), np.asarray(script, dtype=np.int32)
