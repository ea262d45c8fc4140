"""CPU oracle for the CopySpec copy-and-verify decode step (arXiv 2502.08923).

TEST INFRASTRUCTURE ONLY.  This file is a plain, slow restatement of what the method
computes, written from the paper's definitions in numpy (fp64 unless stated).  It is
used by the tests, by the smoke check and by the benchmark's CPU-baseline leg; the CUDA
library never calls it, and it shares no code with the CUDA sources.

Notation (paper main text / App. B): gamma = length of the search key, k = number of
copied draft tokens (|S_copyspec|, "chunk size m"), tau = accepted draft tokens per
attempt ("accepted count"), n = current accepted length ("t"), p0 = 0-indexed start of
the matched gamma-gram (App. B uses 1-indexed p).

Readings taken where the paper is silent or at odds with itself:
  * several matches: LATEST (largest p0) by default; FIRST (smallest p0, the paper's
    footnote in Sec. 3.2 and App. B.3 step 1(c)) is the other policy.
  * non-overlap (App. B.3 step 1(c)): p + gamma - 1 < t - gamma + 1, i.e. p0 <= n - 2 gamma.
  * fewer than k tokens after the match: the draft is clipped, never read past n.
  * a match is exact token equality (the "rolling hash" of Sec. 2.1 is only a lookup
    device; collisions never count as matches).
  * every verification emits tau accepted tokens plus one guaranteed token (Sec. 3.2).
  * argmax ties go to the lowest token id.
  * the model (not given by the paper): pre-norm decoder, RMSNorm, rotate-half RoPE,
    grouped-query attention scaled by 1/sqrt(Dh), SwiGLU FFN, untied LM head, no biases.

Precision contract (`contract=True`): what "bf16 weights, bf16 KV cache, fp32 accumulation"
fixes - the weights are bf16 values (given as such) and new K/V rows are rounded to
nearest-even bf16 when they are stored in the cache.  Nothing else is rounded: activations,
the residual stream, norms, RoPE, softmax and all accumulation are wide (fp64 here; the
CUDA path carries activations as two bf16 terms, i.e. fp32-equivalent operands, and
accumulates in fp32).  `contract=False` stores K/V unrounded too: the plain fp64 definition.

Pins (tests/test_oracle_*.py): brute-force enumeration of all matches; closed forms
(constant, increasing and periodic histories); the paper's hash-map dictionary method
re-implemented separately; a Hugging Face Llama forward (library routine) for the
whole transformer; cache-vs-recompute and block-vs-single-row invariants; RoPE
relative-position property; real-mode output == plain greedy decoding; scripted-mode
output == the script and == a model-free integer simulator; the draft-model fallback of
Sec. 3.3 (decode_loop_drafted) by losslessness, by the closed form "a draft model equal to
the target has every proposal accepted", by delta = 0 reducing to decode_loop and by its
rolled-back cache equalling a fresh forward over the accepted tokens; a constructed example with
the structure of Fig. 2 (gamma=3, 10 copied tokens, accepted prefix + 1 extra token).
The paper's tables (tokens/s, tau, % copied) depend on trained weights and datasets:
parity with them is unpinned.
"""
from __future__ import annotations

import numpy as np

LATEST = 0
FIRST = 1


# ------------------------------------------------------------------ match and draft
def all_matches_bruteforce(h, n, gamma):
    """Every p0 with h[p0:p0+gamma] == h[n-gamma:n] and p0 <= n - 2*gamma, by direct
    enumeration in pure Python (Sec. 3.1; App. B.3 step 1(a)-(c))."""
    out = []
    if gamma < 1 or n < 2 * gamma:
        return out
    for p0 in range(0, n - 2 * gamma + 1):
        ok = True
        for j in range(gamma):
            if int(h[p0 + j]) != int(h[n - gamma + j]):
                ok = False
                break
        if ok:
            out.append(p0)
    return out


def find_match(h, n, gamma, policy=LATEST):
    """Start p0 of the chosen earlier occurrence of the last gamma tokens of h[0:n], or
    -1 (Sec. 3.1; App. B.1 "Match location p"; App. B.3 step 1).  Naive scan over all
    candidate positions, one vectorised comparison per key token."""
    if gamma < 1 or n < 2 * gamma:
        return -1
    h = np.asarray(h)
    n_cand = n - 2 * gamma + 1
    hit = np.ones(n_cand, dtype=bool)
    for j in range(gamma):
        hit &= h[j:j + n_cand] == h[n - gamma + j]
    idx = np.flatnonzero(hit)
    if idx.size == 0:
        return -1
    return int(idx[-1]) if policy == LATEST else int(idx[0])


def gather_draft(h, n, p0, gamma, k):
    """S_copyspec: the (at most k) tokens that followed the match (Sec. 3.2; App. B.1
    "Chunk size m"; App. B.3 step 1(d))."""
    if p0 < 0:
        return []
    start = p0 + gamma
    ln = min(k, n - start)
    return [int(t) for t in h[start:start + ln]]


class GammaGramDict:
    """The paper's own search structure (Sec. 3.1): a hash map from every gamma-token
    subsequence of the accepted sequence to the positions where it starts; O(gamma)
    work per appended token and per lookup, independent of the context size."""

    def __init__(self, gamma):
        self.gamma = gamma
        self.seq = []
        self.table = {}

    def append(self, tok):
        self.seq.append(int(tok))
        g = self.gamma
        if len(self.seq) >= g:
            key = tuple(self.seq[-g:])
            self.table.setdefault(key, []).append(len(self.seq) - g)

    def extend(self, toks):
        for t in toks:
            self.append(t)

    def lookup(self, policy=LATEST):
        g, n = self.gamma, len(self.seq)
        if n < 2 * g:
            return -1
        cands = [p for p in self.table.get(tuple(self.seq[-g:]), []) if p <= n - 2 * g]
        if not cands:
            return -1
        return cands[-1] if policy == LATEST else cands[0]


# --------------------------------------------------------------------- acceptance
def accept_length(draft, target):
    """tau: length of the longest prefix of the draft that equals the target's tokens
    (Sec. 3.2; App. B.2; App. B.3 step 2(a)).  target has len(draft)+1 entries."""
    tau = 0
    for i, d in enumerate(draft):
        if int(d) == int(target[i]):
            tau += 1
        else:
            break
    return tau


def argmax_lowest(row):
    """Greedy choice at temperature 0 (App. B.2), lowest id on ties."""
    return int(np.argmax(row))  # numpy returns the first maximum


# -------------------------------------------------------------------------- model
def round_bf16(x):
    """Round to the nearest bf16 value, ties to even; returned as float64."""
    a = np.ascontiguousarray(np.asarray(x, dtype=np.float32))
    u = a.view(np.uint32).astype(np.uint64)
    r = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return r.astype(np.uint32).view(np.float32).astype(np.float64)


def _np64(t):
    if isinstance(t, np.ndarray):
        return t.astype(np.float64)
    return t.detach().float().cpu().numpy().astype(np.float64)  # torch tensor


def rmsnorm(x, g, eps):
    """x * rsqrt(mean(x^2) + eps) * g, row-wise."""
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * g


def rope(x, pos, theta):
    """Rotate-half rotary embedding.  x: [R][heads][Dh], pos: [R] absolute positions.
    Pair (i, i + Dh/2) is rotated by the angle pos * theta**(-2 i / Dh)."""
    dh = x.shape[-1]
    half = dh // 2
    inv = theta ** (-np.arange(half, dtype=np.float64) * 2.0 / dh)
    ang = np.asarray(pos, dtype=np.float64)[:, None] * inv[None, :]
    c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    a, b = x[..., :half], x[..., half:]
    return np.concatenate([a * c - b * s, b * c + a * s], axis=-1)


def silu(x):
    return x / (1.0 + np.exp(-x))


class KVCache:
    """Per layer K and V for each sequence, [L][2][B][Hkv][max_seq][Dh]; only the
    first kv_len[b] positions of sequence b are meaningful (App. B.2)."""

    def __init__(self, cfg, batch, max_seq, data=None, dtype=np.float64):
        shape = (cfg.n_layers, 2, batch, cfg.n_kv_heads, max_seq, cfg.head_dim)
        if data is None:
            self.a = np.zeros(shape, dtype=dtype)
        else:
            arr = data if isinstance(data, np.ndarray) else data.detach().float().cpu().numpy()
            self.a = arr.astype(dtype).reshape(shape)
        self.max_seq = max_seq


class Model:
    """Decoder-only target model evaluated block-wise against a KV cache."""

    def __init__(self, cfg, weights, contract=True, cache_weights=True):
        self.cfg = cfg
        self.w = weights
        self.contract = contract
        self._cache = {} if cache_weights else None

    # weights are converted to fp64 on use (and kept, for small models)
    def _w(self, layer, name):
        key = (layer, name)
        if self._cache is not None and key in self._cache:
            return self._cache[key]
        t = self.w[name] if layer is None else self.w["layers"][layer][name]
        a = _np64(t)
        if self._cache is not None:
            self._cache[key] = a
        return a

    def _store(self, x):
        return round_bf16(x) if self.contract else x

    def _mm(self, x, layer, name):
        """x [R][in] times W[out][in]^T (W holds bf16 values)."""
        return x @ self._w(layer, name).T

    def embed(self, tokens):
        return self._w(None, "embed")[np.asarray(tokens, dtype=np.int64)]

    def forward_block(self, tokens, pos0, cache, b, return_hidden=False):
        """One forward over `tokens` placed at absolute positions pos0, pos0+1, ...
        of sequence b, whose cache holds positions [0, pos0).  Appends the block's K
        and V rows to the cache at pos0.. and returns logits [R][V] (Sec. 3.2: the
        speculative tokens are appended to the context and evaluated in one pass)."""
        cfg = self.cfg
        R = len(tokens)
        H, Hkv, Dh = cfg.n_heads, cfg.n_kv_heads, cfg.head_dim
        G = H // Hkv
        pos = np.arange(pos0, pos0 + R)
        scale = 1.0 / np.sqrt(Dh)
        x = self.embed(tokens)
        for l in range(cfg.n_layers):
            xn = rmsnorm(x, self._w(l, "attn_norm"), cfg.rms_eps)
            qkv = self._mm(xn, l, "wqkv")
            q = qkv[:, :H * Dh].reshape(R, H, Dh)
            kk = qkv[:, H * Dh:(H + Hkv) * Dh].reshape(R, Hkv, Dh)
            vv = qkv[:, (H + Hkv) * Dh:].reshape(R, Hkv, Dh)
            q = rope(q, pos, cfg.rope_theta)
            kk = self._store(rope(kk, pos, cfg.rope_theta))
            vv = self._store(vv)
            cache.a[l, 0, b, :, pos0:pos0 + R, :] = kk.transpose(1, 0, 2)
            cache.a[l, 1, b, :, pos0:pos0 + R, :] = vv.transpose(1, 0, 2)
            Lk = pos0 + R
            o = np.zeros((R, H, Dh))
            causal = np.arange(Lk)[None, :] <= pos[:, None]          # [R][Lk]
            for hd in range(H):
                K = cache.a[l, 0, b, hd // G, :Lk, :].astype(np.float64)
                V = cache.a[l, 1, b, hd // G, :Lk, :].astype(np.float64)
                s = (q[:, hd, :] @ K.T) * scale
                s = np.where(causal, s, -np.inf)
                s = s - s.max(axis=-1, keepdims=True)
                p = np.exp(s)
                p = p / p.sum(axis=-1, keepdims=True)
                o[:, hd, :] = p @ V
            x = x + self._mm(o.reshape(R, H * Dh), l, "wo")
            xn = rmsnorm(x, self._w(l, "ffn_norm"), cfg.rms_eps)
            gu = self._mm(xn, l, "w_gate_up")
            act = silu(gu[:, :cfg.d_ffn]) * gu[:, cfg.d_ffn:]
            x = x + self._mm(act, l, "w_down")
        xn = rmsnorm(x, self._w(None, "final_norm"), cfg.rms_eps)
        logits = self._mm(xn, None, "lm_head")
        if return_hidden:
            return logits, x
        return logits

    def prefill(self, tokens, cache, b, chunk=64):
        """Fill the cache with tokens[0:len-1] (the last accepted token's K/V are
        computed by the next step)."""
        n = len(tokens) - 1
        for s in range(0, n, chunk):
            self.forward_block(tokens[s:min(n, s + chunk)], s, cache, b)
        return n


# ----------------------------------------------------------------- one verify step
def verify_step(model, cache, b, last_tok, draft, kv_len, script_row=None):
    """App. B.3 step 2 with the extra guaranteed token of Sec. 3.2.  Evaluates the
    block [last_tok, draft...] at positions kv_len.., takes the greedy token per row,
    and accepts the longest agreeing prefix.  In scripted mode the target tokens are
    script_row[0..len(draft)] instead of the argmax (the logits are still computed).
    Returns (tau, out_tokens[tau+1], argmax_ids[len(draft)+1], new_kv_len, logits)."""
    block = [int(last_tok)] + [int(t) for t in draft]
    logits = model.forward_block(block, kv_len, cache, b)
    am = [argmax_lowest(logits[r]) for r in range(len(block))]
    target = am if script_row is None else [int(t) for t in script_row[:len(block)]]
    tau = accept_length(draft, target)
    out = target[:tau + 1]
    return tau, out, am, kv_len + tau + 1, logits


def new_stats(k_max=64):
    return {"steps": 0, "attempts": 0, "accepted": 0, "emitted": 0, "no_match": 0,
            "tau_hist": [0] * (k_max + 1)}


# ------------------------------------------------------------------ generation loop
def decode_loop(model, cache, b, hist, gamma, k, policy, max_new, eos_id=-1, script=None,
                trace=None):
    """App. B.3 steps 1, 2, 4 repeated: search, copy, verify, truncate, append, until
    max_new tokens are emitted (the last block is clipped) or, in real mode, EOS is
    emitted (tokens after it are dropped).  `hist` (list) is extended in place; the
    cache must hold positions [0, len(hist)-1).  Returns (emitted tokens, stats)."""
    hist_list = hist
    emitted = []
    st = new_stats()
    done = False
    while len(emitted) < max_new and not done:
        n = len(hist_list)
        e = len(emitted)
        p0 = find_match(np.asarray(hist_list, dtype=np.int64), n, gamma, policy)
        draft = gather_draft(hist_list, n, p0, gamma, k)
        kv_len = n - 1
        block = [hist_list[-1]] + draft
        logits = model.forward_block(block, kv_len, cache, b)
        am = [argmax_lowest(logits[r]) for r in range(len(block))]
        if script is None:
            target = am
        else:
            # rows past the end of the script have no target: they cannot be accepted
            target = [int(script[e + r]) if e + r < max_new else -1 for r in range(len(block))]
        tau = accept_length(draft, target)
        out = target[:tau + 1]
        out = out[:max_new - e]
        if script is None and eos_id >= 0 and eos_id in out:
            out = out[:out.index(eos_id) + 1]
            done = True
        c = len(out)
        hist_list.extend(out)
        emitted.extend(out)
        st["steps"] += 1
        st["emitted"] += c
        if p0 >= 0:
            st["attempts"] += 1
            st["accepted"] += c - 1
            st["tau_hist"][min(c - 1, len(st["tau_hist"]) - 1)] += 1   # the last bin also takes longer prefixes
        else:
            st["no_match"] += 1
        if trace is not None:
            trace.append({"n": n, "p0": p0, "draft": draft, "argmax": am, "tau": c - 1,
                          "out": list(out)})
    return emitted, st


def decode_loop_drafted(target, t_cache, drafter, d_cache, d_len, b, hist, gamma, k, delta, policy,
                        max_new, eos_id=-1, script=None, trace=None):
    """CopySpec merged with vanilla speculative decoding (Sec. 3.3; App. B.3 steps 1-4).
    Every step first looks for a match of the last gamma tokens; with a match the k copied
    tokens are the draft (step 2).  Without one the smaller draft model proposes delta tokens
    one at a time at temperature 0 (step 3(a)); the target verifies them in one block exactly
    like a copied draft (step 3(b)), and the draft model's cache is rolled back to the accepted
    prefix together with the target's (step 3(c)).
    `d_cache` holds the draft model's K/V for positions [0, d_len) of `hist`, d_len <= len(hist)-1;
    copy steps leave it alone, so before it drafts the draft model first runs over the tokens
    it has not seen.  Readings: the draft model is greedy like the target (the paper evaluates
    at temperature 0); a drafted block earns the extra guaranteed token too (Sec. 3.2).
    Returns (emitted tokens, stats, d_len); stats as in decode_loop (attempts / accepted /
    tau_hist count copy attempts only) plus draft_attempts and draft_accepted."""
    emitted = []
    st = new_stats()
    st["draft_attempts"] = 0
    st["draft_accepted"] = 0
    done = False
    while len(emitted) < max_new and not done:
        n = len(hist)
        e = len(emitted)
        p0 = find_match(np.asarray(hist, dtype=np.int64), n, gamma, policy)
        drafted = p0 < 0 and delta > 0
        if drafted:
            lg = drafter.forward_block(hist[d_len:n], d_len, d_cache, b)     # catch up; last row predicts position n
            d_len = n
            draft = [argmax_lowest(lg[-1])]
            while len(draft) < delta:
                lg = drafter.forward_block([draft[-1]], d_len, d_cache, b)
                d_len += 1
                draft.append(argmax_lowest(lg[0]))
        else:
            draft = gather_draft(hist, n, p0, gamma, k)
        block = [hist[-1]] + draft
        logits = target.forward_block(block, n - 1, t_cache, b)
        am = [argmax_lowest(logits[r]) for r in range(len(block))]
        if script is None:
            tgt = am
        else:
            tgt = [int(script[e + r]) if e + r < max_new else -1 for r in range(len(block))]
        tau = accept_length(draft, tgt)
        out = tgt[:tau + 1][:max_new - e]
        if script is None and eos_id >= 0 and eos_id in out:
            out = out[:out.index(eos_id) + 1]
            done = True
        c = len(out)
        hist.extend(out)
        emitted.extend(out)
        if drafted:
            # positions n .. n+c-2 hold draft tokens that were accepted; the rest is rolled back
            d_len = min(d_len, n + c - 1)
        st["steps"] += 1
        st["emitted"] += c
        if p0 >= 0:
            st["attempts"] += 1
            st["accepted"] += c - 1
            st["tau_hist"][min(c - 1, len(st["tau_hist"]) - 1)] += 1
        else:
            st["no_match"] += 1
            if drafted:
                st["draft_attempts"] += 1
                st["draft_accepted"] += c - 1
        if trace is not None:
            trace.append({"n": n, "p0": p0, "drafted": drafted, "draft": list(draft), "argmax": am,
                          "tau": c - 1, "out": list(out), "d_len": d_len})
    return emitted, st, d_len


def greedy_decode(model, cache, b, hist, max_new, eos_id=-1):
    """Plain one-token-at-a-time greedy decoding with the same model: what the copy
    path must reproduce token for token (Sec. 1; App. B.2)."""
    emitted = []
    while len(emitted) < max_new:
        n = len(hist)
        logits = model.forward_block([hist[-1]], n - 1, cache, b)
        t = argmax_lowest(logits[0])
        hist.append(t)
        emitted.append(t)
        if eos_id >= 0 and t == eos_id:
            break
    return emitted


def scripted_simulator(hist, script, gamma, k, policy, max_new):
    """Model-free replay of the loop in scripted mode, integers only: which match is
    found, what is drafted, how much is accepted, at every step."""
    h = [int(t) for t in hist]
    e = 0
    steps = []
    st = new_stats()
    while e < max_new:
        n = len(h)
        cands = all_matches_bruteforce(h, n, gamma)
        p0 = -1 if not cands else (cands[-1] if policy == LATEST else cands[0])
        draft = [] if p0 < 0 else h[p0 + gamma:min(n, p0 + gamma + k)]
        tau = 0
        while tau < len(draft) and e + tau < max_new and draft[tau] == int(script[e + tau]):
            tau += 1
        c = min(tau + 1, max_new - e)
        out = [int(t) for t in script[e:e + c]]
        h.extend(out)
        e += c
        st["steps"] += 1
        st["emitted"] += c
        if p0 >= 0:
            st["attempts"] += 1
            st["accepted"] += c - 1
            st["tau_hist"][min(c - 1, len(st["tau_hist"]) - 1)] += 1   # the last bin also takes longer prefixes
        else:
            st["no_match"] += 1
        steps.append({"n": n, "p0": p0, "draft": draft, "tau": c - 1, "out": out})
    return steps, st, h
