"""Pins for the oracle's transformer forward.  The paper names model families only, so
the forward is pinned to a library implementation of that family (Hugging Face Llama,
fp64 on CPU) and to invariants that any causal cached forward must satisfy."""
import numpy as np
import pytest
import torch

from oracle import copyspec_oracle as O
from paper_2502_08923_b200 import inputs


def _small_cfg(n_kv_heads):
    return inputs.ModelConfig(n_layers=2, d_model=64, n_heads=4, n_kv_heads=n_kv_heads,
                              head_dim=16, d_ffn=128, vocab=97, rope_theta=10000.0,
                              rms_eps=1e-5)


def _hf_llama(cfg, w):
    from transformers import LlamaConfig, LlamaForCausalLM
    hc = LlamaConfig(hidden_size=cfg.d_model, intermediate_size=cfg.d_ffn,
                     num_hidden_layers=cfg.n_layers, num_attention_heads=cfg.n_heads,
                     num_key_value_heads=cfg.n_kv_heads, head_dim=cfg.head_dim,
                     vocab_size=cfg.vocab, rms_norm_eps=cfg.rms_eps,
                     rope_parameters={"rope_theta": cfg.rope_theta, "rope_type": "default"},
                     tie_word_embeddings=False, attention_bias=False, mlp_bias=False,
                     max_position_embeddings=2048, attn_implementation="eager")
    m = LlamaForCausalLM(hc).double().eval()
    sd = {"model.embed_tokens.weight": w["embed"], "lm_head.weight": w["lm_head"],
          "model.norm.weight": w["final_norm"]}
    qd, kd = cfg.q_dim, cfg.kv_dim
    for i, lay in enumerate(w["layers"]):
        p = f"model.layers.{i}."
        sd[p + "self_attn.q_proj.weight"] = lay["wqkv"][:qd]
        sd[p + "self_attn.k_proj.weight"] = lay["wqkv"][qd:qd + kd]
        sd[p + "self_attn.v_proj.weight"] = lay["wqkv"][qd + kd:]
        sd[p + "self_attn.o_proj.weight"] = lay["wo"]
        sd[p + "mlp.gate_proj.weight"] = lay["w_gate_up"][:cfg.d_ffn]
        sd[p + "mlp.up_proj.weight"] = lay["w_gate_up"][cfg.d_ffn:]
        sd[p + "mlp.down_proj.weight"] = lay["w_down"]
        sd[p + "input_layernorm.weight"] = lay["attn_norm"]
        sd[p + "post_attention_layernorm.weight"] = lay["ffn_norm"]
    missing = m.load_state_dict({k: v.double() for k, v in sd.items()}, strict=False)
    assert not [k for k in missing.missing_keys if "rotary" not in k]
    assert not missing.unexpected_keys
    return m


@pytest.mark.parametrize("n_kv_heads", [4, 2, 1])
def test_forward_matches_library_llama(n_kv_heads):
    cfg = _small_cfg(n_kv_heads)
    w = inputs.make_weights(cfg, seed=11, gain_jitter=0.2)
    toks = np.random.default_rng(0).integers(0, cfg.vocab, size=37).tolist()
    hf = _hf_llama(cfg, w)
    with torch.no_grad():
        want = hf(torch.tensor([toks])).logits[0].numpy()
    model = O.Model(cfg, w, contract=False)
    cache = O.KVCache(cfg, 1, 64)
    # feed as three blocks of different sizes through the cache
    got = np.concatenate([model.forward_block(toks[0:20], 0, cache, 0),
                          model.forward_block(toks[20:21], 20, cache, 0),
                          model.forward_block(toks[21:37], 21, cache, 0)])
    assert got.shape == want.shape
    scale = np.abs(want).max()
    # the library computes its rotary tables in fp32, hence 1e-6 rather than 1e-12
    assert np.abs(got - want).max() <= 1e-6 * max(1.0, scale)
    # a transposed operand, a wrong RoPE pairing or a dropped residual is O(1) here
    assert np.abs(want).max() > 1e-3


def test_tiny_config_matches_library_llama():
    cfg = inputs.TINY
    w = inputs.make_weights(cfg, seed=0)
    toks = np.random.default_rng(2).integers(0, cfg.vocab, size=24).tolist()
    hf = _hf_llama(cfg, w)
    with torch.no_grad():
        want = hf(torch.tensor([toks])).logits[0].numpy()
    model = O.Model(cfg, w, contract=False)
    cache = O.KVCache(cfg, 1, 32)
    got = model.forward_block(toks, 0, cache, 0)
    assert np.abs(got - want).max() <= 1e-6


def test_block_equals_row_by_row_and_recompute():
    cfg = _small_cfg(2)
    w = inputs.make_weights(cfg, seed=5, gain_jitter=0.1)
    toks = np.random.default_rng(1).integers(0, cfg.vocab, size=30).tolist()
    for contract in (False, True):
        model = O.Model(cfg, w, contract=contract)
        c1, c2, c3 = (O.KVCache(cfg, 1, 40) for _ in range(3))
        full = model.forward_block(toks, 0, c1, 0)                      # no cache at all
        model.forward_block(toks[:19], 0, c2, 0)
        block = model.forward_block(toks[19:], 19, c2, 0)               # cached block
        model.forward_block(toks[:19], 0, c3, 0)
        rows = np.concatenate([model.forward_block(toks[i:i + 1], i, c3, 0)
                               for i in range(19, 30)])                 # one row at a time
        assert np.abs(block - full[19:]).max() < 1e-10
        assert np.abs(rows - full[19:]).max() < 1e-10
        assert np.abs(c2.a - c1.a).max() < 1e-12 and np.abs(c3.a - c1.a).max() < 1e-12


def test_stale_cache_rows_beyond_kv_len_are_ignored():
    """App. B.2: after truncation the entries past the accepted length are dead."""
    cfg = _small_cfg(2)
    w = inputs.make_weights(cfg, seed=5)
    model = O.Model(cfg, w, contract=True)
    toks = np.random.default_rng(4).integers(0, cfg.vocab, size=12).tolist()
    clean, dirty = O.KVCache(cfg, 1, 32), O.KVCache(cfg, 1, 32)
    dirty.a[...] = 123.0
    a = model.forward_block(toks, 0, clean, 0)
    b = model.forward_block(toks, 0, dirty, 0)
    assert np.array_equal(a, b)


def test_rope_relative_position_property():
    rng = np.random.default_rng(0)
    q = rng.standard_normal((1, 1, 32))
    k = rng.standard_normal((1, 1, 32))
    def dot(pq, pk):
        return float((O.rope(q, [pq], 10000.0) * O.rope(k, [pk], 10000.0)).sum())
    assert abs(dot(5, 2) - dot(105, 102)) < 1e-9
    assert abs(dot(7, 7) - float((q * k).sum())) < 1e-9
    assert abs(dot(9, 2) - dot(5, 2)) > 1e-3            # it does depend on the offset
    # rotation preserves norms; position 0 is the identity
    assert abs(np.linalg.norm(O.rope(q, [77], 5e5)) - np.linalg.norm(q)) < 1e-12
    assert np.array_equal(O.rope(q, [0], 5e5), q)
    # first pair (i = 0, i + Dh/2) rotates by exactly pos radians
    e = np.zeros((1, 1, 32)); e[0, 0, 0] = 1.0
    r = O.rope(e, [3], 10000.0)
    assert abs(r[0, 0, 0] - np.cos(3.0)) < 1e-15 and abs(r[0, 0, 16] - np.sin(3.0)) < 1e-15


def test_rmsnorm_closed_form():
    x = np.full((2, 8), 3.0)
    g = np.arange(1, 9, dtype=np.float64)
    y = O.rmsnorm(x, g, 0.0)
    assert np.allclose(y, np.tile(g, (2, 1)))             # constant vector -> unit entries
    y = O.rmsnorm(x, g, 7.0)
    assert np.allclose(y, np.tile(g, (2, 1)) * 3.0 / 4.0)  # sqrt(9 + 7) = 4


def test_round_bf16_against_torch():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.standard_normal(10000) * 10 ** rng.uniform(-6, 6, 10000),
                        [0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895314e38]])
    want = torch.tensor(x, dtype=torch.float32).to(torch.bfloat16).double().numpy()
    assert np.array_equal(O.round_bf16(x), want)


def test_contract_rounding_is_small_but_present():
    cfg = inputs.TINY
    w = inputs.make_weights(cfg, seed=0)
    toks = np.random.default_rng(2).integers(0, cfg.vocab, size=16).tolist()
    a = O.Model(cfg, w, contract=False).forward_block(toks, 0, O.KVCache(cfg, 1, 16), 0)
    b = O.Model(cfg, w, contract=True).forward_block(toks, 0, O.KVCache(cfg, 1, 16), 0)
    d = np.abs(a - b).max()
    assert 0 < d < 2e-2
