"""Pins for the forward oracle: an independent library Llama, closed forms, special cases."""
import numpy as np
import pytest
import torch

from oracle import transformer as tf
from paper_2402_13720_b200 import synth

TINY = synth.ModelDesc(2, 64, 4, 2, 16, 96, 100, 64, "f32", rope_theta=10000.0, rms_eps=1e-5)


def _hf_model(m, w):
    from transformers import LlamaConfig, LlamaForCausalLM
    cfg = LlamaConfig(vocab_size=m.vocab, hidden_size=m.d_model, intermediate_size=m.d_ffn,
                      num_hidden_layers=m.n_layers, num_attention_heads=m.n_heads,
                      num_key_value_heads=m.n_kv_heads, head_dim=m.head_dim, rms_norm_eps=m.rms_eps,
                      rope_theta=m.rope_theta, attention_bias=False, mlp_bias=False, tie_word_embeddings=False,
                      max_position_embeddings=m.max_seq, attn_implementation="eager")
    hf = LlamaForCausalLM(cfg).double().eval()
    sd = {"model.embed_tokens.weight": w["embed"], "model.norm.weight": w["final_norm"], "lm_head.weight": w["lm_head"]}
    names = {"attn_norm": "input_layernorm", "wq": "self_attn.q_proj", "wk": "self_attn.k_proj",
             "wv": "self_attn.v_proj", "wo": "self_attn.o_proj", "ffn_norm": "post_attention_layernorm",
             "w_gate": "mlp.gate_proj", "w_up": "mlp.up_proj", "w_down": "mlp.down_proj"}
    for l, lw in enumerate(w["layers"]):
        for k, v in lw.items():
            sd[f"model.layers.{l}.{names[k]}.weight"] = v
    missing = hf.load_state_dict({k: v.double() for k, v in sd.items()}, strict=False)
    assert not [k for k in missing.missing_keys if "rotary" not in k]
    return hf


@pytest.mark.parametrize("seed", [0, 1])
def test_forward_equals_library_llama(seed):
    """Whole forward (RMSNorm, half-split RoPE, GQA, SwiGLU, head) against the library the paper ran on.
    The library keeps its rotary cos/sin table in float32 whatever the model dtype, which bounds the
    agreement at about 1e-7; every planted mistake below moves the logits by more than 1e-4."""
    w = synth.model_weights(TINY, seed)
    hf = _hf_model(TINY, w)
    toks = synth.prompt(seed, TINY.vocab, 24, 0.3, 4, 8)
    with torch.no_grad():
        ref = hf(torch.tensor(toks[None].astype(np.int64))).logits[0].numpy()
    W = tf.Weights(TINY, w)
    got = tf.forward(W, tf.KVCache(TINY), toks, list(range(24)), tf.causal_visible(0, 24))
    assert np.abs(got - ref).max() < 5e-7
    # and in two pieces through the cache (prefix 15, then a 9-row causal block)
    c = tf.KVCache(TINY)
    tf.forward(W, c, toks[:15], list(range(15)), tf.causal_visible(0, 15))
    c.length = 15
    got2 = tf.forward(W, c, toks[15:], list(range(15, 24)), tf.causal_visible(15, 9))
    assert np.abs(got2 - ref[15:]).max() < 5e-7
    assert np.abs(got2 - got[15:]).max() < 1e-13


def test_attention_equals_library_sdpa():
    rng = np.random.default_rng(0)
    q, k, v = rng.standard_normal((5, 4, 8)), rng.standard_normal((9, 2, 8)), rng.standard_normal((9, 2, 8))
    vis = rng.random((5, 9)) < 0.6
    vis[:, 0] = True
    got = tf.masked_attention(q, k, v, vis)
    tq = torch.tensor(q).permute(1, 0, 2)[None]
    tk = torch.tensor(k).permute(1, 0, 2).repeat_interleave(2, dim=0)[None]
    tv = torch.tensor(v).permute(1, 0, 2).repeat_interleave(2, dim=0)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, attn_mask=torch.tensor(vis)[None, None])
    assert np.abs(got - ref[0].permute(1, 0, 2).numpy()).max() < 1e-12


def test_single_visible_key_returns_its_value():
    rng = np.random.default_rng(1)
    q, k, v = rng.standard_normal((3, 2, 4)), rng.standard_normal((6, 2, 4)), rng.standard_normal((6, 2, 4))
    vis = np.zeros((3, 6), dtype=bool)
    vis[0, 4] = vis[1, 0] = vis[2, 5] = True
    out = tf.masked_attention(q, k, v, vis)
    for r, s in ((0, 4), (1, 0), (2, 5)):
        assert np.array_equal(out[r], v[s])


def test_equal_scores_give_mean_of_visible_values():
    rng = np.random.default_rng(2)
    v = rng.standard_normal((7, 1, 4))
    vis = np.array([[True, True, False, True, False, False, True]])
    out = tf.masked_attention(np.zeros((1, 1, 4)), rng.standard_normal((7, 1, 4)), v, vis)
    assert np.allclose(out[0, 0], v[[0, 1, 3, 6], 0].mean(axis=0), atol=1e-15)


def test_gqa_head_mapping():
    """Query heads 0,1 read kv head 0; heads 2,3 read kv head 1."""
    rng = np.random.default_rng(3)
    q = rng.standard_normal((2, 4, 4))
    k, v = rng.standard_normal((5, 2, 4)), rng.standard_normal((5, 2, 4))
    vis = np.ones((2, 5), dtype=bool)
    out = tf.masked_attention(q, k, v, vis)
    for a in range(4):
        solo = tf.masked_attention(q[:, a:a + 1], k[:, a // 2:a // 2 + 1], v[:, a // 2:a // 2 + 1], vis)
        assert np.array_equal(out[:, a], solo[:, 0])


def test_rope_closed_forms():
    rng = np.random.default_rng(4)
    x = rng.standard_normal((3, 2, 8))
    assert np.array_equal(tf.rope(x, [0, 0, 0], 10000.0), x)                      # position 0 is the identity
    y = tf.rope(x, [5, 17, 40], 10000.0)
    assert np.allclose(np.linalg.norm(y, axis=-1), np.linalg.norm(x, axis=-1))    # a rotation
    # pair (i, i + h/2) turns by pos * theta^(-2i/h): check the fastest and the slowest pair by hand
    e = np.zeros((1, 1, 8)); e[0, 0, 0] = 1.0
    r = tf.rope(e, [3], 10000.0)[0, 0]
    assert np.allclose([r[0], r[4]], [np.cos(3.0), np.sin(3.0)]) and np.allclose(np.delete(r, [0, 4]), 0)
    e = np.zeros((1, 1, 8)); e[0, 0, 7] = 1.0
    r = tf.rope(e, [3], 10000.0)[0, 0]
    a = 3.0 * 10000.0 ** (-6.0 / 8.0)
    assert np.allclose([r[3], r[7]], [-np.sin(a), np.cos(a)])
    # scores depend on the position difference only
    q, k = rng.standard_normal((1, 1, 8)), rng.standard_normal((1, 1, 8))
    s1 = (tf.rope(q, [9], 100.0) * tf.rope(k, [4], 100.0)).sum()
    s2 = (tf.rope(q, [30], 100.0) * tf.rope(k, [25], 100.0)).sum()
    assert abs(s1 - s2) < 1e-12


def test_rmsnorm_closed_forms():
    x = np.array([[3.0, -4.0, 0.0, 0.0]])
    out = tf.rmsnorm(x, np.array([1.0, 2.0, 1.0, 1.0]), 0.0)
    assert np.allclose(out, [[3 / 2.5, -8 / 2.5, 0, 0]])                           # rms = sqrt(25/4)
    rng = np.random.default_rng(5)
    y = tf.rmsnorm(rng.standard_normal((4, 32)), np.ones(32), 0.0)
    assert np.allclose((y * y).mean(axis=-1), 1.0)


def test_argmax_ties_take_smallest_id():
    assert list(tf.argmax_rows(np.array([[1.0, 5.0, 5.0, 2.0], [7.0, 7.0, 7.0, 7.0]]))) == [1, 0]


def test_planted_mistakes_are_caught(monkeypatch):
    """A wrong RoPE sign and a dropped norm gain each break the library pin."""
    w = synth.model_weights(TINY, 0)
    hf = _hf_model(TINY, w)
    toks = synth.prompt(0, TINY.vocab, 12, 0.0, 4, 8)
    with torch.no_grad():
        ref = hf(torch.tensor(toks[None].astype(np.int64))).logits[0].numpy()
    W = tf.Weights(TINY, w)

    def run():
        return np.abs(tf.forward(W, tf.KVCache(TINY), toks, list(range(12)), tf.causal_visible(0, 12)) - ref).max()

    assert run() < 5e-7
    good_rope, good_norm = tf.rope, tf.rmsnorm
    monkeypatch.setattr(tf, "rope", lambda x, p, t: good_rope(x, [-q for q in p], t))
    assert run() > 1e-4
    monkeypatch.setattr(tf, "rope", good_rope)
    monkeypatch.setattr(tf, "rmsnorm", lambda x, g, e: good_norm(x, np.ones_like(g), e))
    assert run() > 1e-4
    monkeypatch.setattr(tf, "rmsnorm", good_norm)
    assert run() < 5e-7
