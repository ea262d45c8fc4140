"""Host-side checks that need no GPU: the library builds for sm_100a, loads, exports every
symbol the header declares, and rejects bad arguments before touching a device."""
import ctypes as C
import os
import re

import pytest

from paper_2502_08923_b200 import binding as cs, inputs

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "copyspec.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(cs_[a-z_0-9]+)\s*\(", text)))


def test_header_symbols_are_exported():
    lib = cs.load()
    names = _declared()
    assert {"cs_find_match", "cs_verify_step", "cs_kv_truncate", "cs_decode_loop"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n
    assert set(cs.EXPORTS) == set(names)


def _cfg(cfg, max_seq=1024, max_batch=1, k_max=10):
    return cs.CsModelConfig(cfg.n_layers, cfg.d_model, cfg.n_heads, cfg.n_kv_heads, cfg.head_dim, cfg.d_ffn,
                            cfg.vocab, max_seq, max_batch, k_max, cfg.rope_theta, cfg.rms_eps)


def test_workspace_bytes_is_host_arithmetic():
    lib = cs.load()
    small = lib.cs_workspace_bytes(C.byref(_cfg(inputs.TINY)))
    big = lib.cs_workspace_bytes(C.byref(_cfg(inputs.LLAMA8B, 32768 + 2048 + 32, 8, 20)))
    assert 0 < small < big < 2 << 30
    assert lib.cs_workspace_bytes(None) == 0
    bad = _cfg(inputs.TINY); bad.head_dim = 48
    assert lib.cs_workspace_bytes(C.byref(bad)) == 0
    bad = _cfg(inputs.TINY, max_batch=32, k_max=10)         # 352 rows > 256
    assert lib.cs_workspace_bytes(C.byref(bad)) == 0
    bad = _cfg(inputs.TINY); bad.n_kv_heads = 3
    assert lib.cs_workspace_bytes(C.byref(bad)) == 0


def test_find_match_argument_errors_need_no_device():
    lib = cs.load()
    assert lib.cs_find_match(None, None, 0, 0, 3, 10, 0, None, None, None, None) == cs.CS_OK       # B == 0
    assert lib.cs_find_match(None, None, 1, 8, 0, 10, 0, None, None, None, None) == cs.CS_ERR_ARG  # gamma < 1
    assert lib.cs_find_match(None, None, 1, 8, 9, 10, 0, None, None, None, None) == cs.CS_ERR_ARG  # gamma > 8
    assert lib.cs_find_match(None, None, 1, 8, 3, -1, 0, None, None, None, None) == cs.CS_ERR_ARG
    assert lib.cs_find_match(None, None, 1, 8, 3, 10, 7, None, None, None, None) == cs.CS_ERR_ARG  # policy
    assert lib.cs_find_match(None, None, 1, 8, 3, 10, 0, None, None, None, None) == cs.CS_ERR_ARG  # NULL


def test_context_calls_reject_null():
    lib = cs.load()
    assert lib.cs_verify_step(None, None, None, None, 1, 1, None, None, None, None, None, None, None, None) == cs.CS_ERR_ARG
    assert lib.cs_kv_truncate(None, None, None, 1, None) == cs.CS_ERR_ARG
    assert lib.cs_decode_loop(None, None, None, 1, 1, None, None, 3, 10, 0, 1, -1, None, None, None) == cs.CS_ERR_ARG
    assert lib.cs_decode_loop_drafted(None, None, None, None, 8, None, None, None, None, 3, 10, 3, 0, 1, -1, None, None,
                                      None, None) == cs.CS_ERR_ARG
    assert lib.cs_step_host(None, None, None, 1, 8, None, None, None, None, 3, 1, 0, None, None, None, None) == cs.CS_ERR_ARG
    assert lib.cs_prefill(None, None, None, 1, 1, 1, None, None, None) == cs.CS_ERR_ARG
    assert lib.cs_sync_status(None, None) == cs.CS_ERR_ARG
    h = C.c_void_p()
    assert lib.cs_create(C.byref(h), None, None, None, 0) == cs.CS_ERR_ARG
    assert lib.cs_last_error(None) == b"cs_create: NULL argument"     # cs_create leaves its text with the thread
    bad = _cfg(inputs.TINY); bad.head_dim = 48
    assert lib.cs_create(C.byref(h), C.byref(bad), C.byref(cs.CsWeights()), C.c_void_p(1024), 0) == cs.CS_ERR_SHAPE
    assert b"configuration" in lib.cs_last_error(None)
    assert lib.cs_loop_last_step(None, None, None, None, None, None, None) == cs.CS_ERR_ARG
    assert lib.cs_debug_drop_tile(None, 0) == cs.CS_ERR_ARG
    lib.cs_step_host_reset(None)
    lib.cs_destroy(None)
