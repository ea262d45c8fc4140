"""cs_lm_head_static: the LM-head argmax for callers that cannot allocate device memory.

Some users of this library run where cudaMalloc is not available to them - inside another
framework's allocator or stream callback, as a plug-in that receives input and output buffers
but no allocator, or with the device memory already fully committed - so they cannot provide
the workspace that cs_create needs.  cs_lm_head_static takes only inputs and outputs and keeps
its intermediate per-tile maxima in a fixed array inside the library.  These tests check it
against cs_lm_head (the workspace-based entry point) on two calls in a row, because the fixed
array is shared between calls and keeps the previous call's contents.

This file is named so that pytest collects it last."""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2502_08923_b200 import binding as cs, inputs


def test_sizes_beyond_the_fixed_maximum_are_refused():
    """Checked on the host before any CUDA call, so this needs no GPU."""
    lib = cs.load()
    one = C.c_void_p(16)      # never dereferenced: the size check comes first
    assert lib.cs_lm_head_static(one, one, 65, 4096, 256, one, None) == cs.CS_ERR_LIMIT        # rows > 64
    assert lib.cs_lm_head_static(one, one, 11, 131073, 256, one, None) == cs.CS_ERR_LIMIT      # vocab > 131072
    assert lib.cs_lm_head_static(None, one, 11, 4096, 256, one, None) == cs.CS_ERR_ARG
    assert lib.cs_lm_head_static(one, one, 11, 4096, 252, one, None) == cs.CS_ERR_ARG          # d_model % 8


@pytest.mark.gpu
def test_static_variant_matches_workspace_variant_twice_in_a_row():
    cfg = inputs.ModelConfig(n_layers=1, d_model=256, n_heads=8, n_kv_heads=8, head_dim=32, d_ffn=512,
                             vocab=5000, rope_theta=10000.0, rms_eps=1e-5)       # 39 full tiles + a ragged one
    w = inputs.weights_to(inputs.make_weights(cfg, seed=3), "cuda")
    ctx = cs.Context(cfg, w, max_seq=64, max_batch=4, k_max=10)
    g = torch.Generator().manual_seed(0)
    # the second call has fewer rows and different data: stale pairs of the first call must not leak
    for rows in (40, 11):
        X = torch.zeros((rows + 15) // 16 * 16, cfg.d_model, dtype=torch.bfloat16, device="cuda")
        X[:rows] = torch.randn(rows, cfg.d_model, generator=g).to(torch.bfloat16).cuda()
        want = ctx.cs_lm_head(X, rows=rows)
        assert ctx.cs_sync_status() == 0
        ids = torch.full((rows,), -7, dtype=torch.int32, device="cuda")
        cs.cs_lm_head_static(X, w["lm_head"], ids, rows=rows)
        torch.cuda.synchronize()
        # same kernel, same operands: the integer outputs must agree exactly
        assert ids.cpu().tolist() == want.cpu().tolist()
        ref = X[:rows].double().cpu().numpy() @ w["lm_head"].double().cpu().numpy().T
        assert np.all(ref.max(axis=1) - ref[np.arange(rows), ids.cpu().numpy()] < 1e-4)
    with pytest.raises(cs.CsError) as e:
        cs.cs_lm_head_static(torch.zeros(80, cfg.d_model, dtype=torch.bfloat16, device="cuda"), w["lm_head"],
                             torch.zeros(65, dtype=torch.int32, device="cuda"), rows=65)
    assert e.value.code == cs.CS_ERR_LIMIT
    ctx.close()
