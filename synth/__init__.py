"""Seeded synthetic inputs: model shapes, random-init weights, prompts, random draft trees.

This module only *draws inputs*.  It holds none of the method's arithmetic
(no attention, no tree construction, no masks) and is the one module that
both the CPU oracle's tests and the CUDA library's tests/bench may share.

Recipe (stands in for the trained LLaMA3 / Qwen3 checkpoints and the
SpecBench prompts the paper measures on, which are not available here):
every matrix is iid N(0, 0.02^2) drawn in fp32 from a seeded torch
generator (rounded to bf16 for bf16 models), RMSNorm gains are 1 (or
1 + 0.1*N(0,1) when ``gain_jitter`` is set, so tests can see a dropped gain),
prompts are token ids uniform in [0, vocab).
"""
from __future__ import annotations

import dataclasses
from typing import Dict, List, Optional

import numpy as np
import torch


@dataclasses.dataclass(frozen=True)
class ModelShape:
    name: str
    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    dtype: str  # "fp32" | "bf16"
    tied: bool
    qk_norm: bool
    rope_base: float
    rms_eps: float

    def replace(self, **kw) -> "ModelShape":
        return dataclasses.replace(self, **kw)

    def n_params_streamed(self) -> int:
        """Parameters every decode step must read: all layer matrices + LM head."""
        d, F = self.d_model, self.d_ffn
        dq, dkv = self.n_q_heads * self.head_dim, self.n_kv_heads * self.head_dim
        per_layer = d * dq + 2 * d * dkv + dq * d + 3 * d * F
        return self.n_layers * per_layer + self.vocab * d


TINY = ModelShape("tiny-llama-fp32", 2, 256, 4, 2, 64, 688, 4096, "fp32", True, False, 10000.0, 1e-5)
LLAMA3_8B = ModelShape("llama3-8b-shape", 32, 4096, 32, 8, 128, 14336, 128256, "bf16", False, False, 500000.0, 1e-5)
QWEN3_8B = ModelShape("qwen3-8b-shape", 36, 4096, 32, 8, 128, 12288, 151936, "bf16", False, True, 1000000.0, 1e-6)

LAYER_MATS = ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down")


def _mat_shape(s: ModelShape, name: str):
    d, F = s.d_model, s.d_ffn
    dq, dkv = s.n_q_heads * s.head_dim, s.n_kv_heads * s.head_dim
    return {"wq": (dq, d), "wk": (dkv, d), "wv": (dkv, d), "wo": (d, dq),
            "w_gate": (F, d), "w_up": (F, d), "w_down": (d, F)}[name]


def make_weights(shape: ModelShape, seed: int = 0, device: str = "cpu", gain_jitter: bool = False,
                 std: float = 0.02) -> Dict[str, object]:
    """Random-init weights as torch tensors on ``device`` in the model dtype.

    Returns {"embed": [V,d], "lm_head": [V,d] (the embed tensor itself when tied),
    "final_norm": [d], and per-layer lists "wq","wk","wv","wo","w_gate","w_up",
    "w_down","norm_attn","norm_ffn","q_norm","k_norm"}.  All linear weights
    are stored [out_features, in_features], row-major.
    """
    dt = torch.float32 if shape.dtype == "fp32" else torch.bfloat16
    g = torch.Generator(device=device)
    g.manual_seed(seed)

    def mat(r, c):
        return (torch.randn(r, c, generator=g, device=device, dtype=torch.float32) * std).to(dt).contiguous()

    def gain(n):
        if gain_jitter:
            return (1.0 + 0.1 * torch.randn(n, generator=g, device=device, dtype=torch.float32)).to(dt).contiguous()
        return torch.ones(n, device=device, dtype=dt)

    w: Dict[str, object] = {}
    w["embed"] = mat(shape.vocab, shape.d_model)
    w["lm_head"] = w["embed"] if shape.tied else mat(shape.vocab, shape.d_model)
    w["final_norm"] = gain(shape.d_model)
    for k in LAYER_MATS + ("norm_attn", "norm_ffn", "q_norm", "k_norm"):
        w[k] = []
    for _ in range(shape.n_layers):
        for k in LAYER_MATS:
            w[k].append(mat(*_mat_shape(shape, k)))
        w["norm_attn"].append(gain(shape.d_model))
        w["norm_ffn"].append(gain(shape.d_model))
        w["q_norm"].append(gain(shape.head_dim))
        w["k_norm"].append(gain(shape.head_dim))
    return w


def weights_to_host(w: Dict[str, object]) -> Dict[str, object]:
    """Copy a weight dict to CPU tensors (same dtype, same values); tied tensors stay tied."""
    out: Dict[str, object] = {}
    for k, v in w.items():
        if isinstance(v, list):
            out[k] = [t.cpu() for t in v]
        else:
            out[k] = v.cpu()
    if w["lm_head"] is w["embed"]:
        out["lm_head"] = out["embed"]
    return out


def make_prompt(vocab: int, n: int, seed: int = 0) -> np.ndarray:
    """``n`` token ids uniform in [0, vocab) (int32)."""
    rng = np.random.default_rng(seed + 1000003)
    return rng.integers(0, vocab, size=n, dtype=np.int64).astype(np.int32)


def random_tree_parents(n_nodes: int, max_depth: int, seed: int = 0) -> np.ndarray:
    """Parent index per node of a random rooted tree in breadth-first order.

    Node 0 is the root (parent -1).  A parent is drawn uniformly among the
    nodes that keep the child's depth <= ``max_depth`` and keep depths
    non-decreasing along the node order, so every parent index is smaller
    than its child's and nodes are sorted by depth.
    """
    rng = np.random.default_rng(seed + 7919)
    # choose per-depth node counts first so that rows stay sorted by depth
    depth = np.zeros(n_nodes, dtype=np.int32)
    parents = np.full(n_nodes, -1, dtype=np.int32)
    if n_nodes > 1:
        cuts = np.sort(rng.integers(1, n_nodes, size=max_depth - 1)) if max_depth > 1 else np.array([], dtype=np.int64)
        bounds = [1] + [int(c) for c in cuts] + [n_nodes]
        d = 1
        for a, b in zip(bounds[:-1], bounds[1:]):
            depth[a:b] = d
            if b > a:
                d += 1
        # re-number depths so they are consecutive (empty levels collapse)
        for i in range(1, n_nodes):
            cands = np.nonzero(depth[:i] == depth[i] - 1)[0]
            parents[i] = int(cands[rng.integers(0, len(cands))])
    return parents


def random_qkv(shape_q, shape_kv_cache, shape_kv_block, seed: int = 0, device: str = "cpu", dtype=torch.bfloat16):
    """N(0,1) tensors for the stand-alone tree-attention workload."""
    g = torch.Generator(device=device)
    g.manual_seed(seed + 424243)
    mk = lambda s: torch.randn(*s, generator=g, device=device, dtype=torch.float32).to(dtype).contiguous()
    return mk(shape_q), mk(shape_kv_cache), mk(shape_kv_cache), mk(shape_kv_block), mk(shape_kv_block)
