"""Pins for the oracle's transformer (oracle/transformer.c).

The paper fixes no model numerics, so the block forward is pinned against
things other than itself: an independent library implementation of the same
architectures (Hugging Face LlamaForCausalLM / Qwen3ForCausalLM in fp64,
loaded with the same synthetic weights), a hand-computed one-layer case,
and structural identities (per-path reruns, rotary relative-shift, GQA ==
MHA with repeated KV heads).
"""
import math

import numpy as np
import pytest
import torch

import synth
from oracle import esp

SMALL = synth.TINY.replace(name="pin", n_layers=2, d_model=64, n_q_heads=4, n_kv_heads=2, head_dim=32, d_ffn=96,
                           vocab=300, tied=False, rope_base=5000.0)


def _hf_model(shape, w):
    from transformers import LlamaConfig, LlamaForCausalLM, Qwen3Config, Qwen3ForCausalLM
    kw = dict(vocab_size=shape.vocab, hidden_size=shape.d_model, intermediate_size=shape.d_ffn,
              num_hidden_layers=shape.n_layers, num_attention_heads=shape.n_q_heads,
              num_key_value_heads=shape.n_kv_heads, head_dim=shape.head_dim, rms_norm_eps=shape.rms_eps,
              rope_parameters={"rope_type": "default", "rope_theta": shape.rope_base},
              tie_word_embeddings=shape.tied, attention_bias=False, max_position_embeddings=1024)
    if shape.qk_norm:
        m = Qwen3ForCausalLM(Qwen3Config(use_sliding_window=False, **kw))
    else:
        m = LlamaForCausalLM(LlamaConfig(mlp_bias=False, **kw))
    sd = {"model.embed_tokens.weight": w["embed"], "model.norm.weight": w["final_norm"], "lm_head.weight": w["lm_head"]}
    names = {"wq": "self_attn.q_proj", "wk": "self_attn.k_proj", "wv": "self_attn.v_proj", "wo": "self_attn.o_proj",
             "w_gate": "mlp.gate_proj", "w_up": "mlp.up_proj", "w_down": "mlp.down_proj",
             "norm_attn": "input_layernorm", "norm_ffn": "post_attention_layernorm"}
    if shape.qk_norm:
        names.update({"q_norm": "self_attn.q_norm", "k_norm": "self_attn.k_norm"})
    for l in range(shape.n_layers):
        for k, v in names.items():
            sd[f"model.layers.{l}.{v}.weight"] = w[k][l]
    sd = {k: v.double() for k, v in sd.items()}
    m = m.double().eval()
    missing, unexpected = m.load_state_dict(sd, strict=False)
    assert not unexpected and all("rotary" in k or "inv_freq" in k for k in missing), (missing, unexpected)
    return m


@pytest.mark.parametrize("qk_norm,tied", [(False, False), (True, False), (False, True)])
def test_block_forward_matches_library_decoder(qk_norm, tied):
    shape = SMALL.replace(qk_norm=qk_norm, tied=tied, rms_eps=1e-6 if qk_norm else 1e-5)
    w = synth.make_weights(shape, seed=3, gain_jitter=True, std=0.15)
    toks = synth.make_prompt(shape.vocab, 23, seed=1)
    hf = _hf_model(shape, w)
    with torch.no_grad():
        ref = hf(torch.tensor(toks[None].astype(np.int64))).logits[0].numpy()
    model = esp.OracleModel(shape, w)
    kc, vc = model.new_cache(64)
    # first 9 tokens in one causal block, then the rest as a second block against the cache
    t0 = 9
    E = np.stack([model.embed(int(t)) for t in toks])
    lg0, kb, vb, _ = model.block_forward(kc, vc, 0, E[:t0], np.arange(t0), np.tril(np.ones((t0, t0), np.uint8)))
    kc[:, :t0], vc[:, :t0] = kb, vb
    n1 = len(toks) - t0
    lg1, _, _, _ = model.block_forward(kc, vc, t0, E[t0:], t0 + np.arange(n1), np.tril(np.ones((n1, n1), np.uint8)))
    got = np.concatenate([lg0, lg1])
    scale = np.abs(ref).max()
    assert scale > 0.5  # the test model is not degenerate
    assert np.abs(got - ref).max() <= 2e-5 * scale


def test_one_layer_hand_computed():
    """d=4, one head of size 4, identity-like weights: every number below is worked out by hand."""
    shape = synth.TINY.replace(n_layers=1, d_model=4, n_q_heads=1, n_kv_heads=1, head_dim=4, d_ffn=4, vocab=4,
                               tied=False, rms_eps=0.0, rope_base=10000.0)
    I = np.eye(4, dtype=np.float32)
    Z = np.zeros((4, 4), np.float32)
    w = {"embed": I.copy(), "lm_head": I.copy(), "final_norm": np.ones(4, np.float32),
         "wq": [Z.copy()], "wk": [Z.copy()], "wv": [I.copy()], "wo": [I.copy()],
         "w_gate": [Z.copy()], "w_up": [I.copy()], "w_down": [I.copy()],
         "norm_attn": [np.ones(4, np.float32)], "norm_ffn": [np.ones(4, np.float32)],
         "q_norm": [np.ones(4, np.float32)], "k_norm": [np.ones(4, np.float32)]}
    model = esp.OracleModel(shape, w)
    kc, vc = model.new_cache(4)
    x = np.stack([model.embed(0), model.embed(1)])
    lg, kb, vb, hid = model.block_forward(kc, vc, 0, x, np.arange(2), np.tril(np.ones((2, 2), np.uint8)), need_hidden=True)
    # RMSNorm of a unit basis vector in d=4 with eps=0 scales it by 2; q = k = 0 so attention is a plain
    # average of the visible values; gate = 0 so silu(0) * up = 0 and the FFN adds nothing.
    # row 0: v0 = 2 e0; h = e0 + 2 e0 = 3 e0.          final norm: 3 e0 / sqrt(9/4) = 2 e0
    # row 1: mean(v0, v1) = e0 + e1; h = e0 + 2 e1.     final norm: (e0 + 2 e1) / sqrt(5/4)
    np.testing.assert_allclose(vb[0, :, 0], 2 * I[:2], atol=1e-6)
    np.testing.assert_allclose(lg[0], [2, 0, 0, 0], atol=1e-6)
    r = 1 / math.sqrt(5 / 4)
    np.testing.assert_allclose(lg[1], [r, 2 * r, 0, 0], atol=1e-6)
    # the FFN alone: gate = identity makes the second sub-block add silu(n) * n with n the normed input
    w["w_gate"] = [I.copy()]
    model = esp.OracleModel(shape, w)
    _, _, _, hid = model.block_forward(kc, vc, 0, x[:1], np.arange(1), np.ones((1, 1), np.uint8), need_hidden=True)
    silu2 = 2 / (1 + math.exp(-2.0))
    h0 = 3 + silu2 * 2
    np.testing.assert_allclose(hid[0], [2.0, 0, 0, 0], atol=1e-6)  # final norm of h0 * e0 is again 2 e0
    assert h0 > 3


def _random_block(shape, seed, n_nodes=9, k=2, L=7):
    w = synth.make_weights(shape, seed=seed, gain_jitter=True, std=0.15)
    model = esp.OracleModel(shape, w)
    parents = synth.random_tree_parents(n_nodes, 3, seed)
    depths = np.zeros(n_nodes, np.int32)
    for i in range(1, n_nodes):
        depths[i] = depths[parents[i]] + 1
    toks = synth.make_prompt(shape.vocab, n_nodes, seed + 5)
    tree = esp.Tree(toks, parents, depths, np.zeros(n_nodes, np.float32))
    spec = esp.SpecCfg(n_probes=k, n_anchor=0)
    blk = esp.layout_block(tree, spec)
    ctx = synth.make_prompt(shape.vocab, L, seed + 9)
    kc, vc = model.new_cache(64)
    E = np.stack([model.embed(int(t)) for t in ctx])
    _, kb, vb, _ = model.block_forward(kc, vc, 0, E, np.arange(L), np.tril(np.ones((L, L), np.uint8)))
    kc[:, :L], vc[:, :L] = kb, vb
    mvec = esp.mask_init_mean(E)
    return model, tree, blk, kc, vc, L, mvec


def test_tree_block_equals_per_path_reruns():
    """Figure 1 (right) / Figure 3: each row sees only its own past, so running the whole tree in one block
    must give, for every row, exactly what an ordinary causal run of that row's root-to-self path gives."""
    shape = SMALL.replace(qk_norm=True)
    model, tree, blk, kc, vc, L, mvec = _random_block(shape, seed=11)
    x = np.stack([model.embed(int(t)) if t >= 0 else mvec for t in blk.row_token])
    lg, kb, vb, _ = model.block_forward(kc, vc, L, x, L + blk.row_pos_off, blk.vis)
    for r in range(blk.m):
        chain = [i for i in range(blk.m) if blk.vis[r, i]]
        assert chain[-1] == r
        assert list(blk.row_pos_off[chain]) == list(range(len(chain)))  # a path occupies consecutive positions
        n = len(chain)
        lg_p, kb_p, _, _ = model.block_forward(kc, vc, L, x[chain], L + np.arange(n), np.tril(np.ones((n, n), np.uint8)))
        assert np.array_equal(lg_p[-1], lg[r])
        assert np.array_equal(kb_p[:, -1], kb[:, r])


def test_rope_relative_shift_invariance():
    """Rotary embedding makes attention depend on relative positions only: shifting every position of an
    uncached sequence by a constant leaves the logits unchanged (up to fp32 rounding of the angles)."""
    shape = SMALL
    w = synth.make_weights(shape, seed=5, std=0.15)
    model = esp.OracleModel(shape, w)
    toks = synth.make_prompt(shape.vocab, 12, 2)
    E = np.stack([model.embed(int(t)) for t in toks])
    kc, vc = model.new_cache(8)
    tri = np.tril(np.ones((12, 12), np.uint8))
    a, _, _, _ = model.block_forward(kc, vc, 0, E, np.arange(12), tri)
    b, _, _, _ = model.block_forward(kc, vc, 0, E, 37 + np.arange(12), tri)
    assert np.abs(a - b).max() <= 1e-4 * np.abs(a).max()
    # ...and it does depend on relative position: reversing the order of positions changes the result
    c, _, _, _ = model.block_forward(kc, vc, 0, E, np.arange(12)[::-1].copy(), tri)
    assert np.abs(a - c).max() > 1e-3 * np.abs(a).max()


def test_gqa_equals_mha_with_repeated_kv_heads():
    shape = SMALL
    w = synth.make_weights(shape, seed=6, std=0.15)
    g = shape.n_q_heads // shape.n_kv_heads
    h = shape.head_dim
    w2 = dict(w)
    rep = lambda t: t.view(shape.n_kv_heads, 1, h, -1).expand(-1, g, -1, -1).reshape(shape.n_q_heads * h, -1).contiguous()
    w2["wk"] = [rep(t) for t in w["wk"]]
    w2["wv"] = [rep(t) for t in w["wv"]]
    toks = synth.make_prompt(shape.vocab, 10, 3)
    outs = []
    for sh, ww in ((shape, w), (shape.replace(n_kv_heads=shape.n_q_heads), w2)):
        model = esp.OracleModel(sh, ww)
        E = np.stack([model.embed(int(t)) for t in toks])
        kc, vc = model.new_cache(4)
        outs.append(model.block_forward(kc, vc, 0, E, np.arange(10), np.tril(np.ones((10, 10), np.uint8)))[0])
    assert np.array_equal(outs[0], outs[1])


def test_bf16_weights_are_widened_exactly():
    shape = SMALL.replace(dtype="bf16")
    w = synth.make_weights(shape, seed=7, std=0.15)
    wf = {k: ([t.float() for t in v] if isinstance(v, list) else v.float()) for k, v in w.items()}
    toks = synth.make_prompt(shape.vocab, 8, 4)
    outs = []
    for sh, ww in ((shape, w), (shape.replace(dtype="fp32"), wf)):
        model = esp.OracleModel(sh, ww)
        E = np.stack([model.embed(int(t)) for t in toks])
        kc, vc = model.new_cache(4)
        outs.append(model.block_forward(kc, vc, 0, E, np.arange(8), np.tril(np.ones((8, 8), np.uint8)))[0])
    assert np.array_equal(outs[0], outs[1])


def test_tree_attention_operator_against_softmax_definition():
    """The stand-alone operator against softmax(q K^T / sqrt(h)) V written with library matmuls in fp64."""
    rng = np.random.default_rng(0)
    M, L, Hq, Hkv, h = 7, 19, 4, 2, 16
    q = rng.standard_normal((M, Hq, h)).astype(np.float32)
    kc, vc = (rng.standard_normal((L, Hkv, h)).astype(np.float32) for _ in range(2))
    kb, vb = (rng.standard_normal((M, Hkv, h)).astype(np.float32) for _ in range(2))
    parents = synth.random_tree_parents(M, 3, 1)
    vis = np.zeros((M, M), np.uint8)
    for i in range(M):
        a = i
        while a >= 0:
            vis[i, a] = 1
            a = parents[a]
    out = esp.tree_attention(q, kc, vc, kb, vb, vis)
    K = np.concatenate([kc, kb]).astype(np.float64)
    V = np.concatenate([vc, vb]).astype(np.float64)
    allow = np.concatenate([np.ones((M, L), bool), vis.astype(bool)], axis=1)
    for hh in range(Hq):
        s = q[:, hh].astype(np.float64) @ K[:, hh // 2].T / math.sqrt(h)
        s[~allow] = -np.inf
        p = torch.softmax(torch.from_numpy(s), dim=-1).numpy()
        np.testing.assert_allclose(out[:, hh], p @ V[:, hh // 2], rtol=0, atol=2e-6)


def test_linear_operator_against_library_matmul():
    """The stand-alone matrix product against numpy's fp64 matmul, fp32 and bf16 weights, ragged sizes; a
    transposed operand or a dropped k term would show as an O(1) error."""
    rng = np.random.default_rng(3)
    for M, K, N in ((1, 8, 5), (7, 72, 131), (80, 200, 9)):
        x = rng.standard_normal((M, K)).astype(np.float32)
        w = torch.from_numpy(rng.standard_normal((N, K)).astype(np.float32))
        ref = x.astype(np.float64) @ w.double().numpy().T
        assert np.abs(esp.linear(x, w) - ref).max() <= 1e-5 * np.abs(ref).max()
        wb = w.bfloat16()
        refb = x.astype(np.float64) @ wb.double().numpy().T
        assert np.abs(esp.linear(x, wb) - refb).max() <= 1e-5 * np.abs(refb).max()
