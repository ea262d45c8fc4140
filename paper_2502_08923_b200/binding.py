"""ctypes binding of libcopyspec.so: same names as the C ABI (include/copyspec.h),
argument marshalling only.  PyTorch provides device memory and the current stream; every
step of the path runs in the library's CUDA kernels.  There is no CPU fallback: if the
library cannot be loaded, every call raises."""
from __future__ import annotations

import ctypes as C
import os

import torch

from . import build as _build

CS_OK = 0
CS_ERR_ARG, CS_ERR_SHAPE, CS_ERR_CAPACITY, CS_ERR_CUDA, CS_ERR_TIMEOUT, CS_ERR_UNSUPPORTED = -1, -2, -3, -4, -5, -6
CS_ERR_LIMIT = -7
LATEST, FIRST = 0, 1
STAMP_FAMILIES = ("gemm", "attention", "lm_head", "merge", "other")
TAU_HIST = 65

_STATUS = {0: "CS_OK", -1: "CS_ERR_ARG", -2: "CS_ERR_SHAPE", -3: "CS_ERR_CAPACITY", -4: "CS_ERR_CUDA",
           -5: "CS_ERR_TIMEOUT", -6: "CS_ERR_UNSUPPORTED", -7: "CS_ERR_LIMIT"}


class CsError(RuntimeError):
    def __init__(self, code, where, detail=""):
        self.code = code
        super().__init__(f"{where}: {_STATUS.get(code, code)} {detail}".strip())


class CsModelConfig(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_heads", "n_kv_heads", "head_dim",
                                         "d_ffn", "vocab", "max_seq", "max_batch", "k_max")] + \
               [("rope_theta", C.c_float), ("rms_eps", C.c_float)]


class CsWeights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("lm_head", C.c_void_p), ("final_norm", C.c_void_p)] + \
               [(n, C.POINTER(C.c_void_p)) for n in ("attn_norm", "wqkv", "wo", "ffn_norm", "w_gate_up", "w_down")]


class CsStats(C.Structure):
    _fields_ = [(n, C.c_uint64) for n in ("steps", "attempts", "accepted", "emitted", "no_match")] + \
               [("tau_hist", C.c_uint64 * TAU_HIST)]

    def as_dict(self):
        return {"steps": self.steps, "attempts": self.attempts, "accepted": self.accepted,
                "emitted": self.emitted, "no_match": self.no_match, "tau_hist": list(self.tau_hist)}


WORKSPACE_GUARD, GUARD_BYTE = 4096, 0xA5   # guard bands around a Context's workspace
EXPORTS = ("cs_workspace_bytes", "cs_create", "cs_destroy", "cs_last_error", "cs_sync_status",
           "cs_find_match", "cs_verify_step", "cs_kv_truncate", "cs_decode_loop", "cs_decode_loop_drafted", "cs_step_host",
           "cs_prefill", "cs_linear", "cs_step_host_reset", "cs_debug_drop_tile",
           "cs_loop_begin", "cs_loop_steps", "cs_loop_poll", "cs_loop_end", "cs_loop_last_step", "cs_set_stamps", "cs_stamp_layout", "cs_set_match_index",
           "cs_loop_launches_per_step", "cs_lm_head", "cs_lm_head_static", "cs_gram_index_bytes",
           "cs_gram_index_reset", "cs_gram_index_update", "cs_find_match_indexed", "cs_gram_index_status")

_lib = None


def lib_path() -> str:
    return _build.LIB


def load(build_if_missing: bool = True) -> C.CDLL:
    """Load libcopyspec.so (building it with nvcc first when it is missing or stale)."""
    global _lib
    if _lib is not None:
        return _lib
    if build_if_missing:
        _build.build()
    if not os.path.exists(_build.LIB):
        raise RuntimeError("libcopyspec.so is not built: run `python -m paper_2502_08923_b200.build`")
    lib = C.CDLL(_build.LIB)
    vp, ip, i = C.c_void_p, C.c_void_p, C.c_int
    lib.cs_workspace_bytes.restype = C.c_size_t
    lib.cs_workspace_bytes.argtypes = [C.POINTER(CsModelConfig)]
    lib.cs_create.restype = i
    lib.cs_create.argtypes = [C.POINTER(C.c_void_p), C.POINTER(CsModelConfig), C.POINTER(CsWeights), vp, C.c_size_t]
    lib.cs_destroy.restype = None
    lib.cs_destroy.argtypes = [vp]
    lib.cs_last_error.restype = C.c_char_p
    lib.cs_last_error.argtypes = [vp]
    lib.cs_sync_status.restype = i
    lib.cs_sync_status.argtypes = [vp, vp]
    lib.cs_find_match.restype = i
    lib.cs_find_match.argtypes = [ip, ip, i, i, i, i, i, ip, ip, ip, vp]
    lib.cs_verify_step.restype = i
    lib.cs_verify_step.argtypes = [vp, ip, ip, ip, i, i, vp, ip, ip, ip, ip, ip, vp, vp]
    lib.cs_kv_truncate.restype = i
    lib.cs_kv_truncate.argtypes = [vp, ip, ip, i, vp]
    lib.cs_decode_loop.restype = i
    lib.cs_decode_loop.argtypes = [vp, ip, ip, i, i, vp, ip, i, i, i, i, i, ip, C.POINTER(CsStats), vp]
    lib.cs_step_host.restype = i
    lib.cs_step_host.argtypes = [vp, ip, ip, i, i, ip, ip, vp, ip, i, i, i, ip, ip, ip, vp]
    lib.cs_decode_loop_drafted.restype = i
    lib.cs_decode_loop_drafted.argtypes = [vp, vp, ip, ip, i, vp, ip, vp, ip, i, i, i, i, i, i, ip,
                                           C.POINTER(CsStats), C.POINTER(C.c_uint64), vp]
    lib.cs_loop_begin.restype = i
    lib.cs_loop_begin.argtypes = [vp, ip, ip, i, i, vp, ip, i, i, i, i, i, ip, vp]
    lib.cs_loop_steps.restype = i
    lib.cs_loop_steps.argtypes = [vp, i, vp]
    lib.cs_loop_poll.restype = i
    lib.cs_loop_poll.argtypes = [vp, C.POINTER(CsStats), C.POINTER(C.c_int), vp]
    lib.cs_loop_launches_per_step.restype = i
    lib.cs_loop_launches_per_step.argtypes = [vp]
    lib.cs_loop_last_step.restype = i
    lib.cs_loop_last_step.argtypes = [vp, ip, ip, ip, ip, ip, vp]
    lib.cs_loop_end.restype = None
    lib.cs_loop_end.argtypes = [vp]
    lib.cs_set_match_index.restype = i
    lib.cs_set_match_index.argtypes = [vp, vp, i]
    lib.cs_set_stamps.restype = i
    lib.cs_set_stamps.argtypes = [vp, vp, i]
    lib.cs_stamp_layout.restype = i
    lib.cs_stamp_layout.argtypes = [vp, C.POINTER(C.c_int), i]
    lib.cs_prefill.restype = i
    lib.cs_prefill.argtypes = [vp, ip, ip, i, i, i, vp, ip, vp]
    lib.cs_lm_head.restype = i
    lib.cs_lm_head.argtypes = [vp, vp, i, ip, vp, vp]
    lib.cs_lm_head_static.restype = i
    lib.cs_lm_head_static.argtypes = [vp, vp, i, i, i, ip, vp]
    lib.cs_step_host_reset.restype = None
    lib.cs_step_host_reset.argtypes = [vp]
    lib.cs_debug_drop_tile.restype = i
    lib.cs_debug_drop_tile.argtypes = [vp, i]
    lib.cs_linear.restype = i
    lib.cs_linear.argtypes = [vp, vp, vp, i, i, i, vp, vp]
    _lib = lib
    return lib


def _ptr(t):
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor")
    return C.c_void_p(t.data_ptr())


def _host_i32(t, name):
    if t is None:
        return None
    if t.is_cuda or not t.is_contiguous() or t.dtype != torch.int32:
        raise ValueError(f"{name} must be a contiguous int32 host tensor")
    return C.c_void_p(t.data_ptr())


def _i32(t, name):
    if t is not None and t.dtype != torch.int32:
        raise ValueError(f"{name} must be int32")
    return _ptr(t)


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def cs_find_match(hist, hist_len, gamma, k, policy=LATEST, out=None):
    """Suffix-match search and draft gather.  hist [B][stride] int32, hist_len [B] int32 (CUDA).
    Returns (match_pos [B], draft [B][k], draft_len [B]); `out` may supply those tensors."""
    lib = load()
    B, stride = hist.shape
    if out is None:
        out = (torch.empty(B, dtype=torch.int32, device=hist.device),
               torch.empty(B, max(k, 1), dtype=torch.int32, device=hist.device)[:, :k].contiguous(),
               torch.empty(B, dtype=torch.int32, device=hist.device))
    mp, dr, dl = out
    rc = lib.cs_find_match(_i32(hist, "hist"), _i32(hist_len, "hist_len"), B, stride, gamma, k, policy,
                           _i32(mp, "match_pos"), C.c_void_p(dr.data_ptr()) if k > 0 else None,
                           _i32(dl, "draft_len"), _stream())
    if rc != CS_OK:
        raise CsError(rc, "cs_find_match")
    return mp, dr, dl


class GramIndex:
    """Device-resident gamma-gram index (argument marshalling only).  One per batch of sequences."""

    def __init__(self, B, capacity_tokens, gamma, device="cuda"):
        self.lib = load()
        self.B, self.cap, self.gamma = B, capacity_tokens, gamma
        self.lib.cs_gram_index_bytes.restype = C.c_size_t
        nbytes = self.lib.cs_gram_index_bytes(B, capacity_tokens)
        self.buf = torch.empty(nbytes, dtype=torch.uint8, device=device)
        self.cs_gram_index_reset()

    def _p(self):
        return C.c_void_p(self.buf.data_ptr())

    def cs_gram_index_reset(self):
        rc = self.lib.cs_gram_index_reset(self._p(), self.B, self.cap, _stream())
        if rc != CS_OK:
            raise CsError(rc, "cs_gram_index_reset")

    def cs_gram_index_update(self, hist, hist_len):
        B, stride = hist.shape
        rc = self.lib.cs_gram_index_update(self._p(), B, self.cap, _i32(hist, "hist"), _i32(hist_len, "hist_len"), stride,
                                           self.gamma, _stream())
        if rc != CS_OK:
            raise CsError(rc, "cs_gram_index_update")

    def cs_find_match_indexed(self, hist, hist_len, k, policy=LATEST, out=None):
        B, stride = hist.shape
        if out is None:
            out = (torch.empty(B, dtype=torch.int32, device=hist.device),
                   torch.empty(B, max(k, 1), dtype=torch.int32, device=hist.device)[:, :k].contiguous(),
                   torch.empty(B, dtype=torch.int32, device=hist.device))
        mp, dr, dl = out
        rc = self.lib.cs_find_match_indexed(self._p(), B, self.cap, _i32(hist, "hist"), _i32(hist_len, "hist_len"), stride,
                                            self.gamma, k, policy, _i32(mp, "match_pos"),
                                            C.c_void_p(dr.data_ptr()) if k > 0 else None, _i32(dl, "draft_len"), _stream())
        if rc != CS_OK:
            raise CsError(rc, "cs_find_match_indexed")
        return mp, dr, dl

    def cs_gram_index_status(self):
        return self.lib.cs_gram_index_status(self._p(), self.B, self.cap, _stream())


def pack_gate_up(w_gate_up, d_ffn):
    """Re-lay the [2F][d] (gate rows, then up rows) matrix into the layout the library reads:
    blocks of 128 rows, each holding 64 gate rows followed by the 64 matching up rows (rows
    past F are zero), so that one GEMM tile sees both halves of SwiGLU."""
    d = w_gate_up.shape[1]
    nb = -(-d_ffn // 64)
    out = torch.zeros(nb, 2, 64, d, dtype=w_gate_up.dtype, device=w_gate_up.device)
    pad = torch.zeros(nb * 64, d, dtype=w_gate_up.dtype, device=w_gate_up.device)
    pad[:d_ffn] = w_gate_up[:d_ffn]
    out[:, 0] = pad.view(nb, 64, d)
    pad.zero_()
    pad[:d_ffn] = w_gate_up[d_ffn:]
    out[:, 1] = pad.view(nb, 64, d)
    return out.view(nb * 128, d).contiguous()


def cs_lm_head_static(X, W, ids, rows=None):
    """Greedy token ids of bf16 rows X under the LM head W, written into the caller's `ids`.
    For callers that may not allocate: needs no Context and no workspace, and this wrapper
    itself allocates nothing - X, W and ids are all the caller's tensors.  Limits: rows <= 64,
    vocab <= 131072 (CsError with CS_ERR_LIMIT beyond).  Calls share one fixed scratch array
    inside the library, so keep them on one stream."""
    lib = load()
    rows = X.shape[0] if rows is None else rows
    vocab, d = W.shape
    rc = lib.cs_lm_head_static(_ptr(X), _ptr(W), rows, vocab, d, _i32(ids, "ids"), _stream())
    if rc != CS_OK:
        raise CsError(rc, "cs_lm_head_static")
    return ids


class Context:
    """Owns the device workspace and the cs_ctx handle for one model.  `weights` uses the
    plain layouts of `inputs.make_weights`; the gate/up matrix is re-laid here once."""

    def __init__(self, cfg, weights, max_seq, max_batch, k_max):
        lib = load()
        self.lib = lib
        self.cfg = cfg
        self.max_seq, self.max_batch, self.k_max = max_seq, max_batch, k_max
        self.c_cfg = CsModelConfig(cfg.n_layers, cfg.d_model, cfg.n_heads, cfg.n_kv_heads, cfg.head_dim,
                                   cfg.d_ffn, cfg.vocab, max_seq, max_batch, k_max, cfg.rope_theta, cfg.rms_eps)
        nbytes = lib.cs_workspace_bytes(C.byref(self.c_cfg))
        if nbytes == 0:
            raise CsError(CS_ERR_SHAPE, "cs_workspace_bytes", "unsupported configuration")
        self.workspace_bytes = nbytes
        # the workspace sits between two guard bands of a fixed byte pattern (workspace_guards_intact)
        raw = torch.empty(nbytes + 1024 + 2 * WORKSPACE_GUARD, dtype=torch.uint8, device="cuda")
        off = WORKSPACE_GUARD + (-(raw.data_ptr() + WORKSPACE_GUARD)) % 1024
        raw[:off].fill_(GUARD_BYTE)
        raw[off + nbytes:].fill_(GUARD_BYTE)
        self._raw, self._ws_off = raw, off
        self.weights = weights          # keeps the tensors alive
        L = cfg.n_layers
        self._arrs = {}
        self._packed = []
        cw = CsWeights()
        for name in ("embed", "lm_head", "final_norm"):
            t = weights[name]
            assert t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous()
            setattr(cw, name, t.data_ptr())
        for name in ("attn_norm", "wqkv", "wo", "ffn_norm", "w_gate_up", "w_down"):
            arr = (C.c_void_p * L)()
            for l in range(L):
                t = weights["layers"][l][name]
                if name == "w_gate_up":
                    t = pack_gate_up(t, cfg.d_ffn)
                    self._packed.append(t)
                assert t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous()
                arr[l] = t.data_ptr()
            self._arrs[name] = arr
            setattr(cw, name, C.cast(arr, C.POINTER(C.c_void_p)))
        self.handle = C.c_void_p()
        rc = lib.cs_create(C.byref(self.handle), C.byref(self.c_cfg), C.byref(cw),
                           C.c_void_p(raw.data_ptr() + off), nbytes)
        if rc != CS_OK:
            raise CsError(rc, "cs_create")

    def workspace_guards_intact(self) -> bool:
        """True while nothing has written into the guard bands on either side of the workspace
        (synchronises the device)."""
        torch.cuda.synchronize()
        lo, hi = self._raw[:self._ws_off], self._raw[self._ws_off + self.workspace_bytes:]
        return bool((lo == GUARD_BYTE).all().item() and (hi == GUARD_BYTE).all().item())

    def close(self):
        if getattr(self, "handle", None):
            self.lib.cs_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, rc, where):
        if rc != CS_OK:
            msg = self.lib.cs_last_error(self.handle)
            raise CsError(rc, where, msg.decode() if msg else "")

    def alloc_kv(self):
        c = self.cfg
        return torch.zeros(c.n_layers, 2, self.max_batch, c.n_kv_heads, self.max_seq, c.head_dim,
                           dtype=torch.bfloat16, device="cuda")

    def cs_sync_status(self):
        return self.lib.cs_sync_status(self.handle, _stream())

    def cs_verify_step(self, last_tok, draft, draft_len, kv_cache, kv_len, target_script=None, out=None,
                       logits_dbg=None):
        """One verification forward + acceptance.  Returns (accept_len [B], out_tokens [B][k+1],
        argmax_ids [B][k+1]); kv_len is advanced in place."""
        B = last_tok.shape[0]
        k = draft.shape[1] if draft is not None and draft.dim() == 2 else 0
        dev = last_tok.device
        if out is None:
            out = (torch.empty(B, dtype=torch.int32, device=dev),
                   torch.empty(B, k + 1, dtype=torch.int32, device=dev),
                   torch.empty(B, k + 1, dtype=torch.int32, device=dev))
        al, ot, am = out
        rc = self.lib.cs_verify_step(self.handle, _i32(last_tok, "last_tok"),
                                     C.c_void_p(draft.data_ptr()) if k > 0 else None,
                                     _i32(draft_len, "draft_len"), B, k, _ptr(kv_cache), _i32(kv_len, "kv_len"),
                                     _i32(target_script, "target_script"), _i32(al, "accept_len"),
                                     _i32(ot, "out_tokens"), _i32(am, "argmax_ids"), _ptr(logits_dbg), _stream())
        self._check(rc, "cs_verify_step")
        return al, ot, am

    def cs_step_host(self, hist_host, hist_len_host, hist_dev, hist_len_dev, kv_cache, kv_len, gamma, k,
                     accept_len_host, out_tokens_host, policy=LATEST, script_host=None):
        """One step from host (CPU, ideally pinned) int32 tensors; hist_host / hist_len_host advance in
        place, accept_len_host [B] and out_tokens_host [B][k+1] receive the step's result."""
        B, stride = hist_host.shape
        rc = self.lib.cs_step_host(self.handle, _host_i32(hist_host, "hist_host"), _host_i32(hist_len_host, "hist_len_host"),
                                   B, stride, _i32(hist_dev, "hist_dev"), _i32(hist_len_dev, "hist_len_dev"),
                                   _ptr(kv_cache), _i32(kv_len, "kv_len"), gamma, k, policy,
                                   _host_i32(script_host, "script_host"), _host_i32(accept_len_host, "accept_len_host"),
                                   _host_i32(out_tokens_host, "out_tokens_host"), _stream())
        self._check(rc, "cs_step_host")

    def cs_step_host_reset(self):
        self.lib.cs_step_host_reset(self.handle)

    def cs_debug_drop_tile(self, k_block):
        self._check(self.lib.cs_debug_drop_tile(self.handle, k_block), "cs_debug_drop_tile")

    def cs_kv_truncate(self, kv_len, new_len):
        rc = self.lib.cs_kv_truncate(self.handle, _i32(kv_len, "kv_len"), _i32(new_len, "new_len"),
                                     kv_len.shape[0], _stream())
        self._check(rc, "cs_kv_truncate")

    def cs_prefill(self, hist, hist_len, max_len, kv_cache, kv_len):
        B, stride = hist.shape
        rc = self.lib.cs_prefill(self.handle, _i32(hist, "hist"), _i32(hist_len, "hist_len"), B, stride,
                                 int(max_len), _ptr(kv_cache), _i32(kv_len, "kv_len"), _stream())
        self._check(rc, "cs_prefill")

    def cs_decode_loop(self, hist, hist_len, kv_cache, kv_len, gamma, k, max_new, policy=LATEST, eos_id=-1,
                       script=None):
        """The generation loop; returns the statistics as a dict.  hist/hist_len/kv_len advance in place."""
        B, stride = hist.shape
        st = CsStats()
        rc = self.lib.cs_decode_loop(self.handle, _i32(hist, "hist"), _i32(hist_len, "hist_len"), B, stride,
                                     _ptr(kv_cache), _i32(kv_len, "kv_len"), gamma, k, policy, max_new, eos_id,
                                     _i32(script, "script"), C.byref(st), _stream())
        self._check(rc, "cs_decode_loop")
        return st.as_dict()

    def cs_decode_loop_drafted(self, drafter, hist, hist_len, kv_cache, kv_len, kv_drafter, kv_len_drafter, gamma, k,
                               delta, max_new, policy=LATEST, eos_id=-1, script=None):
        """The loop merged with a draft model (`self` is the target, `drafter` another Context or
        None when delta is 0), one sequence: hist [1][stride].  Returns the statistics as a dict
        with draft_attempts and draft_accepted added."""
        B, stride = hist.shape
        if B != 1:
            raise ValueError("cs_decode_loop_drafted takes one sequence")
        st = CsStats()
        ds = (C.c_uint64 * 2)()
        rc = self.lib.cs_decode_loop_drafted(self.handle, drafter.handle if drafter is not None else None,
                                             _i32(hist, "hist"), _i32(hist_len, "hist_len"), stride, _ptr(kv_cache),
                                             _i32(kv_len, "kv_len"), _ptr(kv_drafter) if kv_drafter is not None else None,
                                             _i32(kv_len_drafter, "kv_len_drafter"), gamma, k, delta, policy, max_new,
                                             eos_id, _i32(script, "script"), C.byref(st), ds, _stream())
        self._check(rc, "cs_decode_loop_drafted")
        out = st.as_dict()
        out["draft_attempts"], out["draft_accepted"] = int(ds[0]), int(ds[1])
        return out

    def cs_loop_begin(self, hist, hist_len, kv_cache, kv_len, gamma, k, max_new, policy=LATEST, eos_id=-1,
                      script=None):
        B, stride = hist.shape
        self._loop_refs = (hist, hist_len, kv_cache, kv_len, script)     # keep the buffers alive
        self._loop_shape = (B, k)
        rc = self.lib.cs_loop_begin(self.handle, _i32(hist, "hist"), _i32(hist_len, "hist_len"), B, stride,
                                    _ptr(kv_cache), _i32(kv_len, "kv_len"), gamma, k, policy, max_new, eos_id,
                                    _i32(script, "script"), _stream())
        self._check(rc, "cs_loop_begin")

    def cs_loop_steps(self, n_steps):
        self._check(self.lib.cs_loop_steps(self.handle, n_steps, _stream()), "cs_loop_steps")

    def cs_loop_poll(self):
        """Waits for the stream; returns (statistics dict, number of finished sequences)."""
        st, done = CsStats(), C.c_int(0)
        self._check(self.lib.cs_loop_poll(self.handle, C.byref(st), C.byref(done), _stream()), "cs_loop_poll")
        return st.as_dict(), done.value

    def cs_loop_last_step(self):
        """The most recent step's (match_pos [B], draft_len [B], accept_len [B], out_tokens [B][k+1],
        argmax_ids [B][k+1]) as int32 host tensors."""
        B, k = self._loop_shape
        mp, dl, al = (torch.empty(B, dtype=torch.int32) for _ in range(3))
        ot, am = (torch.empty(B, k + 1, dtype=torch.int32) for _ in range(2))
        rc = self.lib.cs_loop_last_step(self.handle, *(C.c_void_p(t.data_ptr()) for t in (mp, dl, al, ot, am)), _stream())
        self._check(rc, "cs_loop_last_step")
        return mp, dl, al, ot, am

    def cs_loop_launches_per_step(self):
        return self.lib.cs_loop_launches_per_step(self.handle)

    def cs_loop_end(self):
        self.lib.cs_loop_end(self.handle)
        self._loop_refs = None

    def cs_set_match_index(self, index):
        """The loop searches through `index` (a GramIndex sized for the loop's batch and stride) or,
        with None, scans."""
        self._match_index = index
        if index is None:
            rc = self.lib.cs_set_match_index(self.handle, None, 0)
        else:
            rc = self.lib.cs_set_match_index(self.handle, index._p(), index.cap)
        self._check(rc, "cs_set_match_index")

    def cs_set_stamps(self, stamps):
        """Step timeline on (`stamps`: zeroed int64 CUDA tensor, one slot per stamped launch) or off (None)."""
        self._stamps = stamps
        n = 0 if stamps is None else stamps.numel()
        self._check(self.lib.cs_set_stamps(self.handle, _ptr(stamps), n), "cs_set_stamps")

    def cs_stamp_layout(self):
        """Kernel family of every slot one step uses (see STAMP_FAMILIES)."""
        fam = (C.c_int * 4096)()
        n = self.lib.cs_stamp_layout(self.handle, fam, 4096)
        return [STAMP_FAMILIES[f] for f in list(fam)[:n]]

    def cs_lm_head(self, X, rows=None, logits_dbg=None):
        """Greedy token ids of bf16 rows X[rows][d_model] under the model's LM head."""
        rows = X.shape[0] if rows is None else rows
        ids = torch.empty(rows, dtype=torch.int32, device=X.device)
        rc = self.lib.cs_lm_head(self.handle, _ptr(X), rows, _i32(ids, "ids"), _ptr(logits_dbg), _stream())
        self._check(rc, "cs_lm_head")
        return ids

    def cs_linear(self, X, W, rows=None):
        """Y[rows][N] fp32 = X[rows][K] bf16 @ W[N][K]^T bf16 through the tensor-core GEMM."""
        rows = X.shape[0] if rows is None else rows
        N, K = W.shape
        Y = torch.empty(rows, N, dtype=torch.float32, device=X.device)
        rc = self.lib.cs_linear(self.handle, _ptr(X), _ptr(W), rows, N, K, _ptr(Y), _stream())
        self._check(rc, "cs_linear")
        return Y
