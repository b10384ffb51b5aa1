"""CPU oracle, part 2: the ESP decode-and-verify procedure, step by step.

TEST INFRASTRUCTURE ONLY.  Plain Python/numpy written from the paper; it
shares no code with the CUDA library and is imported only by tests, the
smoke check and the benchmark's CPU-baseline leg.

Notation follows the paper: k mask tokens ("probes"), Top-K candidates per
probe, budget B = number of tree nodes including the last accepted token
(the root), lambda the mask-update rate.  Positions are 0-based; L is the
number of cached positions and the root sits, uncached, at position L.

Where the paper is silent or inconsistent the reading taken here is stated in
the docstring of the function concerned.
"""
from __future__ import annotations

import ctypes
import dataclasses
from typing import List, Optional, Sequence, Tuple

import numpy as np

from . import build as _build

_F32 = np.float32


# --------------------------------------------------------------------------- C binding
class _Cfg(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("n_layers", "d_model", "n_q_heads", "n_kv_heads", "head_dim", "d_ffn", "vocab", "wdtype", "qk_norm")] + \
               [("rope_base", ctypes.c_float), ("rms_eps", ctypes.c_float)]


_PP = ctypes.POINTER(ctypes.c_void_p)


class _Weights(ctypes.Structure):
    _fields_ = [("embed", ctypes.c_void_p), ("lm_head", ctypes.c_void_p), ("final_norm", ctypes.c_void_p)] + \
               [(n, _PP) for n in ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down", "norm_attn", "norm_ffn",
                                   "q_norm", "k_norm")]


_lib = None


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(_build.build())
        _lib.orc_block_forward.restype = ctypes.c_int
        _lib.orc_tree_attention.restype = ctypes.c_int
        _lib.orc_linear.restype = ctypes.c_int
        _lib.orc_num_threads.restype = ctypes.c_int
        _lib.orc_det_logf.restype = ctypes.c_float
        _lib.orc_det_logf.argtypes = [ctypes.c_float]
        _lib.orc_gumbel_from_bits.restype = ctypes.c_float
        _lib.orc_gumbel_from_bits.argtypes = [ctypes.c_uint32]
        _lib.orc_uniform_from_bits.restype = ctypes.c_float
        _lib.orc_uniform_from_bits.argtypes = [ctypes.c_uint32]
    return _lib


def num_threads() -> int:
    return int(_load().orc_num_threads())


def _ptr(t) -> int:
    if hasattr(t, "data_ptr"):
        assert t.is_contiguous() and t.device.type == "cpu"
        return t.data_ptr()
    assert t.flags["C_CONTIGUOUS"]
    return t.ctypes.data


def _np(a, dt):
    return np.ascontiguousarray(a, dtype=dt)


class OracleModel:
    """The frozen model f_theta (Section 2): shape + weights, evaluated by ``transformer.c``.

    ``shape`` is any object with fields n_layers, d_model, n_q_heads,
    n_kv_heads, head_dim, d_ffn, vocab, dtype ("fp32"|"bf16"), qk_norm,
    rope_base, rms_eps.  ``weights`` maps names to CPU tensors/arrays holding
    fp32 values or bf16 bit patterns ([out, in] row-major; per-layer lists).
    """

    def __init__(self, shape, weights):
        self.shape = shape
        self.w = weights  # keep alive
        self.d = shape.d_model
        self.V = shape.vocab
        self.n_layers = shape.n_layers
        self.dkv = shape.n_kv_heads * shape.head_dim
        self.cfg = _Cfg(shape.n_layers, shape.d_model, shape.n_q_heads, shape.n_kv_heads, shape.head_dim,
                        shape.d_ffn, shape.vocab, 0 if shape.dtype == "fp32" else 1, int(bool(shape.qk_norm)),
                        float(shape.rope_base), float(shape.rms_eps))
        cw = _Weights()
        cw.embed, cw.lm_head, cw.final_norm = _ptr(weights["embed"]), _ptr(weights["lm_head"]), _ptr(weights["final_norm"])
        self._arrays = []
        for n in ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down", "norm_attn", "norm_ffn", "q_norm", "k_norm"):
            arr = (ctypes.c_void_p * shape.n_layers)(*[_ptr(t) for t in weights[n]])
            self._arrays.append(arr)
            setattr(cw, n, ctypes.cast(arr, _PP))
        self.cw = cw

    def embed(self, token: int) -> np.ndarray:
        """e = E[token] (Section 3.1), widened to fp32."""
        out = np.empty(self.d, dtype=_F32)
        _load().orc_embed_row(ctypes.byref(self.cfg), ctypes.c_void_p(self.cw.embed), ctypes.c_int32(int(token)),
                              ctypes.c_void_p(out.ctypes.data))
        return out

    def new_cache(self, cap: int):
        shp = (self.n_layers, cap, self.shape.n_kv_heads, self.shape.head_dim)
        return np.zeros(shp, dtype=_F32), np.zeros(shp, dtype=_F32)

    def block_forward(self, kc, vc, L, x, pos, vis, want=None, need_hidden=False):
        """Run the block; returns (logits [M,V] (rows not wanted are NaN), kblk, vblk [n_l,M,Hkv,h], hidden|None)."""
        M = x.shape[0]
        x = _np(x, _F32)
        pos = _np(pos, np.int32)
        vis = _np(vis, np.uint8)
        assert vis.shape == (M, M) and all(vis[i, i] for i in range(M))
        want = np.ones(M, np.uint8) if want is None else _np(want, np.uint8)
        cap = kc.shape[1]
        kb = np.zeros((self.n_layers, M, self.shape.n_kv_heads, self.shape.head_dim), dtype=_F32)
        vb = np.zeros_like(kb)
        logits = np.full((M, self.V), np.nan, dtype=_F32)
        hidden = np.zeros((M, self.d), dtype=_F32) if need_hidden else None
        rc = _load().orc_block_forward(
            ctypes.byref(self.cfg), ctypes.byref(self.cw), ctypes.c_void_p(kc.ctypes.data),
            ctypes.c_void_p(vc.ctypes.data), ctypes.c_int64(cap), ctypes.c_int32(int(L)), ctypes.c_int32(M),
            ctypes.c_void_p(x.ctypes.data), ctypes.c_void_p(pos.ctypes.data), ctypes.c_void_p(vis.ctypes.data),
            ctypes.c_void_p(kb.ctypes.data), ctypes.c_void_p(vb.ctypes.data), ctypes.c_void_p(want.ctypes.data),
            ctypes.c_void_p(logits.ctypes.data), ctypes.c_void_p(hidden.ctypes.data if need_hidden else None))
        if rc != 0:
            raise RuntimeError("orc_block_forward failed")
        return logits, kb, vb, hidden


def tree_attention(q, kc, vc, kb, vb, vis):
    """Tree-masked GQA attention alone: q [M,Hq,h], cache [L,Hkv,h], block [M,Hkv,h], vis [M,M] -> [M,Hq,h]."""
    q, kc, vc, kb, vb = (_np(a, _F32) for a in (q, kc, vc, kb, vb))
    vis = _np(vis, np.uint8)
    M, Hq, h = q.shape
    L, Hkv = kc.shape[0], kb.shape[1]
    out = np.zeros_like(q)
    rc = _load().orc_tree_attention(ctypes.c_int32(M), ctypes.c_int32(L), ctypes.c_int32(Hq), ctypes.c_int32(Hkv),
                                    ctypes.c_int32(h), *(ctypes.c_void_p(a.ctypes.data) for a in (q, kc, vc, kb, vb, vis, out)))
    if rc != 0:
        raise RuntimeError("orc_tree_attention failed")
    return out


def linear(x, w) -> np.ndarray:
    """y = x W^T with the oracle's matrix product (fp32 running sums over k): x [M,K] fp32, w [N,K] fp32 or bf16."""
    x = _np(x, _F32)
    M, K = x.shape
    N = w.shape[0]
    is_bf16 = hasattr(w, "dtype") and str(w.dtype).endswith("bfloat16")
    y = np.zeros((M, N), dtype=_F32)
    rc = _load().orc_linear(ctypes.c_int32(M), ctypes.c_int32(K), ctypes.c_int32(N), ctypes.c_void_p(x.ctypes.data),
                            ctypes.c_void_p(_ptr(w)), ctypes.c_int32(1 if is_bf16 else 0), ctypes.c_void_p(y.ctypes.data))
    if rc != 0:
        raise RuntimeError("orc_linear failed")
    return y


# --------------------------------------------------------------------------- ESP pieces
@dataclasses.dataclass
class SpecCfg:
    """Speculation hyper-parameters (Section 4 "Block Complexity", "Mask token design").

    n_probes      k, mask tokens per anchored node
    topk          K, candidates taken per probe (Algorithm 1 takes B-i; pool = min(K, B-i))
    max_nodes     B, tree nodes including the root
    expand_width  W: how many nodes per depth get children. 1 = the Top-1
                  expansion of Section 3.4 / Appendix D; 0 = every node, as
                  Algorithm 1's loop is printed
    n_anchor      how many nodes (in tree order, root first) carry a probe
                  chain; 0 = every node (the paper: BC = (k+1)*N rows)
    prune_parent  drop a candidate equal to its parent's token (Section 3.5)
    prune_root    also drop a candidate equal to the last generated token
    ema_per_token mask update once per emitted token (else once per step)
    lam           lambda of the mask update, 0.1 in the paper
    """
    n_probes: int = 2
    topk: int = 4
    max_nodes: int = 20
    expand_width: int = 1
    n_anchor: int = 0
    prune_parent: bool = True
    prune_root: bool = False
    ema_per_token: bool = True
    lam: float = 0.1
    static_widths: Tuple[int, ...] = ()   # fixed branch widths [K_1..K_k] (Section 4.2); empty = dynamic tree
    mask_init: str = "mean"               # "mean" (Eq. mask_init_mean) | "last_k" | "given" (Section 4, mask designs)
    temperature: float = 0.0              # 0 = greedy matching; > 0 = sample matching at that temperature (Section 4)
    seed: int = 0                         # 64-bit seed of the sampling noise

    @property
    def k_prime(self) -> int:
        """Entries kept per probe so the list refills to K after pruning ("next best candidate")."""
        k = max(self.static_widths) if self.static_widths else self.topk
        return k + int(self.prune_parent) + int(self.prune_root)


def mask_init_mean(E_rows: np.ndarray) -> np.ndarray:
    """Eq. (mask_init_mean): m = (1/t) sum_j e_j, the same vector for all k masks.  fp32 running sum in j order."""
    acc = np.zeros(E_rows.shape[1], dtype=_F32)
    for j in range(E_rows.shape[0]):
        acc = (acc + E_rows[j].astype(_F32)).astype(_F32)
    return (acc / _F32(E_rows.shape[0])).astype(_F32)


def mask_init_last_k(E_rows: np.ndarray, k: int) -> np.ndarray:
    """"Last K (hard init)" of Section 4: the k masks take the embeddings of the last k prompt tokens.  The
    paper's index expression (e_{t-k-i}) does not address the last k tokens it names; the words are followed:
    mask i (1-based) = embedding of prompt token t-k+i, i.e. the last k tokens in prompt order (a prompt
    shorter than k repeats its first token)."""
    t = E_rows.shape[0]
    return np.stack([E_rows[max(t - k + i, 0)].astype(_F32) for i in range(k)])


def mask_update(m: np.ndarray, e: np.ndarray, lam: float) -> np.ndarray:
    """Eq. (mask_update_mean): m <- m + lambda (e - m), fp32."""
    return (m + _F32(lam) * (e.astype(_F32) - m)).astype(_F32)


def topk_desc(logits: np.ndarray, kp: int) -> Tuple[np.ndarray, np.ndarray]:
    """argtopK (Section 3.2): the kp largest logits, ordered by value descending then token id ascending.

    Written as the definition: a full sort of the vocabulary.
    """
    ids = np.arange(logits.shape[0])
    order = np.lexsort((ids, -logits.astype(np.float64)))[:kp]
    return order.astype(np.int32), logits[order].astype(_F32)


def philox4x32_10(ctr: Sequence[int], key: Sequence[int]) -> List[int]:
    """One Philox4x32-10 block (Salmon et al., SC'11): 4 counter words, 2 key words -> 4 output words."""
    c = (ctypes.c_uint32 * 4)(*[int(x) & 0xffffffff for x in ctr])
    k = (ctypes.c_uint32 * 2)(*[int(x) & 0xffffffff for x in key])
    o = (ctypes.c_uint32 * 4)()
    _load().orc_philox4x32_10(c, k, o)
    return [int(x) for x in o]


def gumbel_noise(seed: int, position: int, n_vocab: int) -> np.ndarray:
    """g(seed, position, v) for every token v: standard Gumbel noise, a pure function of its arguments."""
    out = np.empty(n_vocab, dtype=_F32)
    _load().orc_gumbel_noise(ctypes.c_uint32(seed & 0xffffffff), ctypes.c_uint32((seed >> 32) & 0xffffffff),
                             ctypes.c_uint32(position), ctypes.c_int32(n_vocab), ctypes.c_void_p(out.ctypes.data))
    return out


def sample_scores(logits: np.ndarray, position: int, temperature: float, seed: int) -> np.ndarray:
    """logits / T + g in fp32: one rounded multiply by fl(1/T), one rounded add."""
    inv_t = _F32(1.0) / _F32(temperature)
    return (np.asarray(logits, dtype=_F32) * inv_t).astype(_F32) + gumbel_noise(seed, position, len(logits))


def next_token(logits: np.ndarray, position: int, spec: "SpecCfg") -> int:
    """The base model's token for absolute position `position` given the logits of the row before it:
    the arg-max (temperature 0, Section 2 first equation) or the Gumbel-max draw from softmax(logits / T)
    (Section 4 "sample matching"); ties go to the lower token id."""
    if spec.temperature > 0.0:
        return int(topk_desc(sample_scores(logits, position, spec.temperature, spec.seed), 1)[0][0])
    return int(topk_desc(logits, 1)[0][0])


def log_sum_exp(logits: np.ndarray) -> np.float32:
    """lse = max + log(sum exp(x - max)) in fp32 (softmax at temperature 1 over the full vocabulary)."""
    mx = _F32(np.max(logits))
    s = np.sum(np.exp((logits - mx).astype(_F32)).astype(_F32), dtype=_F32)
    return _F32(mx + np.log(s, dtype=_F32))


@dataclasses.dataclass
class Tree:
    tokens: np.ndarray   # [N] int32, node 0 = root
    parents: np.ndarray  # [N] int32, -1 for the root; parents[i] < i
    depths: np.ndarray   # [N] int32
    logp: np.ndarray     # [N] fp32 cumulative log-probability (root 0)

    @property
    def n(self) -> int:
        return int(self.tokens.shape[0])


def root_only(token: int) -> Tree:
    return Tree(np.array([token], np.int32), np.array([-1], np.int32), np.zeros(1, np.int32), np.zeros(1, _F32))


def build_tree(root_token: int, cand_ids: Sequence[np.ndarray], cand_logits: Sequence[np.ndarray],
               lses: Sequence[float], spec: SpecCfg) -> Tree:
    """Dynamic token tree (Algorithm 1, Section 3.4) with the pruner (Section 3.5).

    cand_ids[i-1], cand_logits[i-1] : the Top-K' list of the probe that predicts
    depth i (value descending, id ascending); lses[i-1] its log-sum-exp.

    Reading of Algorithm 1 (its printed form removes the chosen nodes from the
    set the final selection is taken from, and asks for logits "given the path
    of n" that do not exist before verification): every child at depth i is
    scored with the same probe-i distribution (Appendix D, "weak conditional
    dependence"), P(c) = P(parent) * p_i(token) (kept as a sum of fp32
    log-probabilities, logit - lse, no renormalisation after pruning); the
    nodes that get children at depth i are the top-min(W, B-i) depth-i nodes
    (W = 1 is the paper's Top-1 expansion, W = 0 expands all); each expanded
    parent draws the first min(K, B-i) entries of the list after the pruner
    dropped tokens equal to the parent's token (and to the root's, if
    prune_root); the tree is the root plus the B-1 best created nodes by
    (cumulative log-probability descending, depth ascending, creation order
    ascending).  Because log-probabilities are <= 0 a parent never ranks after
    its child, so the selection is closed under taking ancestors.  Rows are
    then ordered by depth, ties by selection rank (breadth-first order).
    """
    B, K, W = spec.max_nodes, spec.topk, spec.expand_width
    D = len(cand_ids)
    tok: List[int] = [int(root_token)]
    par: List[int] = [-1]
    dep: List[int] = [0]
    lp: List[np.float32] = [_F32(0.0)]
    expanded = [0]
    for i in range(1, D + 1):
        ids, lg, lse = cand_ids[i - 1], cand_logits[i - 1], _F32(lses[i - 1])
        pool = min(K, B - i)
        created = []
        if pool > 0:
            for p in expanded:
                taken = 0
                for j in range(len(ids)):
                    t = int(ids[j])
                    if spec.prune_parent and t == tok[p]:
                        continue
                    if spec.prune_root and t == tok[0]:
                        continue
                    if taken == pool:
                        break
                    logp_t = _F32(_F32(lg[j]) - lse)
                    tok.append(t)
                    par.append(p)
                    dep.append(i)
                    lp.append(_F32(lp[p] + logp_t))
                    created.append(len(tok) - 1)
                    taken += 1
        width = B - i if W == 0 else min(W, B - i)
        created.sort(key=lambda c: (-float(lp[c]), c))
        expanded = created[:max(width, 0)]
    cands = list(range(1, len(tok)))
    cands.sort(key=lambda c: (-float(lp[c]), dep[c], c))
    chosen = cands[:B - 1]
    rank = {c: r for r, c in enumerate(chosen)}
    order = [0] + sorted(chosen, key=lambda c: (dep[c], rank[c]))
    new_index = {c: r for r, c in enumerate(order)}
    return Tree(np.array([tok[c] for c in order], np.int32),
                np.array([-1 if par[c] < 0 else new_index[par[c]] for c in order], np.int32),
                np.array([dep[c] for c in order], np.int32),
                np.array([lp[c] for c in order], _F32))


def build_static_tree(root_token: int, cand_ids: Sequence[np.ndarray], widths: Sequence[int], spec: SpecCfg) -> Tree:
    """Static tree with fixed branch widths [K_1..K_k] (Section 4.2): the Top-1 node of depth i-1 gets the
    first K_i pruned candidates of probe i."""
    tok, par, dep = [int(root_token)], [-1], [0]
    parent = 0
    for i, Ki in enumerate(widths, start=1):
        if i > len(cand_ids):
            break
        first = None
        taken = 0
        for t in cand_ids[i - 1]:
            t = int(t)
            if spec.prune_parent and t == tok[parent]:
                continue
            if spec.prune_root and t == tok[0]:
                continue
            if taken == Ki:
                break
            tok.append(t); par.append(parent); dep.append(i)
            if first is None:
                first = len(tok) - 1
            taken += 1
        if first is None:
            break
        parent = first
    n = len(tok)
    return Tree(np.array(tok, np.int32), np.array(par, np.int32), np.array(dep, np.int32), np.zeros(n, _F32))


@dataclasses.dataclass
class Block:
    """Row layout of one forward pass (Figure 3): tree nodes first, all mask rows at the end."""
    n_nodes: int
    row_token: np.ndarray    # [M] token id, -1 for mask rows
    row_pos_off: np.ndarray  # [M] position minus L
    vis: np.ndarray          # [M,M] uint8
    anchors: List[int]       # anchored node indices, in order
    probe_row: dict          # (anchor node, j in 1..k) -> row index

    @property
    def m(self) -> int:
        return int(self.row_token.shape[0])


def anchor_set(tree: Tree, spec: SpecCfg) -> List[int]:
    n = tree.n if spec.n_anchor == 0 else min(spec.n_anchor, tree.n)
    return list(range(n)) if spec.n_probes > 0 else []


def layout_block(tree: Tree, spec: SpecCfg) -> Block:
    """Rows, position offsets and the tree attention mask (Figures 1, 3; Appendices D, E).

    A node at depth t sits at position L + t and sees its ancestors and
    itself.  Probe j (1-based) of anchored node u sits at pos(u) + j and sees
    u's ancestors-or-self plus probes 1..j of the same chain -- nothing of any
    other chain, sibling or descendant.  Paper mode (every node anchored)
    gives (k+1) * N rows, the block complexity of Section 3.3.
    """
    N, k = tree.n, spec.n_probes
    anchors = anchor_set(tree, spec)
    M = N + k * len(anchors)
    row_token = np.full(M, -1, np.int32)
    row_pos = np.zeros(M, np.int32)
    vis = np.zeros((M, M), np.uint8)
    row_token[:N] = tree.tokens
    row_pos[:N] = tree.depths
    for i in range(N):
        a = i
        while a >= 0:
            vis[i, a] = 1
            a = int(tree.parents[a])
    probe_row = {}
    r = N
    for u in anchors:
        for j in range(1, k + 1):
            probe_row[(u, j)] = r
            row_pos[r] = tree.depths[u] + j
            vis[r, :N] = vis[u, :N]
            for jj in range(1, j + 1):
                vis[r, probe_row[(u, jj)]] = 1
            r += 1
    return Block(N, row_token, row_pos, vis, anchors, probe_row)


def verify_walk(tree: Tree, next_token_of_node: Sequence[int]) -> Tuple[List[int], List[int]]:
    """Lossless verification (Section 2 "Verification", Section 3.3): starting at the root, emit the model's
    own next token at the current node; move to the child carrying exactly that token if there is one,
    else stop.  Returns (accepted node path p_0..p_a with p_0 = root, emitted tokens y_1..y_{a+1}); the
    last emitted token is the bonus token."""
    path, out = [0], []
    cur = 0
    while True:
        y = int(next_token_of_node[cur])
        out.append(y)
        nxt = -1
        for c in range(tree.n):
            if int(tree.parents[c]) == cur and int(tree.tokens[c]) == y:
                nxt = c
                break
        if nxt < 0:
            break
        cur = nxt
        path.append(cur)
    return path, out


def acceptance_length(n_emitted: int, n_steps: int) -> float:
    """tau (Section 4 "Performance Metric"): tokens emitted per model call, bonus token included."""
    return n_emitted / n_steps


def call_reduction_percent(tau: float) -> float:
    """Reduction in model forward calls (Appendix G.1): model calls are proportional to 1/tau."""
    return 100.0 * (1.0 - 1.0 / tau)


def draft_source(tree: Tree, blk: Block, path: Sequence[int], spec: SpecCfg) -> Tuple[int, int, List[int]]:
    """Which mask rows of the block just verified feed which depth of the next tree (Section 2: mask i
    elicits the token i+1 positions ahead; Appendix E position ids).

    u* is the deepest anchored node on the accepted path p_0..p_a.  Its probe j sits at pos(u*) + j and
    predicts the token at pos(u*) + j + 1.  The next root sits at L + a + 1, so depth i of the next tree
    is the token at L + a + 1 + i: it needs probe j = delta + i with delta = a - depth(u*).  Returns
    (u*, delta, rows) with rows[i-1] the block row that proposes depth i, i = 1..k-delta.
    """
    a = len(path) - 1
    ustar = max(p for p in path if p in blk.anchors)
    delta = a - int(tree.depths[ustar])
    rows = [blk.probe_row[(ustar, j)] for j in range(delta + 1, spec.n_probes + 1)]
    return ustar, delta, rows


def next_tree(root_token: int, cand_ids, cand_logits, lses, spec: SpecCfg) -> Tree:
    """The tree the next step verifies: Algorithm 1, or the fixed-width tree when spec.static_widths is set."""
    if spec.static_widths:
        return build_static_tree(root_token, cand_ids, spec.static_widths, spec)
    return build_tree(root_token, cand_ids, cand_logits, lses, spec)


def block_complexity(k: int, widths: Sequence[int]) -> int:
    """BC = (k+1) (1 + sum_i K_i) (Section 3.3)."""
    return (k + 1) * (1 + int(sum(widths)))


# --------------------------------------------------------------------------- the decoder
class EspOracle:
    """ESP generation with one model (Sections 2-3), and plain greedy decoding for comparison."""

    def __init__(self, model: OracleModel, spec: SpecCfg, cap: int):
        self.model, self.spec = model, spec
        self.kc, self.vc = model.new_cache(cap)
        self.L = 0
        self.m: Optional[np.ndarray] = None      # [max(k,1)][d]: one vector per mask position, all updated alike
        self.given_mask: Optional[np.ndarray] = None
        self.tree: Optional[Tree] = None
        self.emitted: List[int] = []
        self.steps = 0
        self.accept_hist: List[int] = []
        self.log: List[dict] = []       # per-step records for parity checks
        self.keep_logits = False

    # -- helpers
    def _rows_x(self, blk: Block) -> np.ndarray:
        x = np.empty((blk.m, self.model.d), dtype=_F32)
        probe_of_row = {row: j for (_, j), row in blk.probe_row.items()}
        for r in range(blk.m):
            x[r] = self.model.embed(int(blk.row_token[r])) if blk.row_token[r] >= 0 else self.m[probe_of_row[r] - 1]
        return x

    def set_mask(self, m: np.ndarray):
        """Mask vectors given from outside ("Sample" and mu + n*sigma initialisations): [k][d], used by prefill."""
        self.given_mask = np.array(m, dtype=_F32).reshape(max(self.spec.n_probes, 1), self.model.d)

    def _emit(self, y: int):
        self.emitted.append(int(y))
        if self.spec.ema_per_token and self.m is not None:
            self.m = mask_update(self.m, self.model.embed(int(y)), self.spec.lam)

    def _probe_lists(self, logits, rows):
        ids, vals, lses = [], [], []
        for r in rows:
            i, v = topk_desc(logits[r], self.spec.k_prime)
            ids.append(i); vals.append(v); lses.append(log_sum_exp(logits[r]))
        return ids, vals, lses

    # -- prefill (Figure 1 middle; Section 3.3 "During prefill, ESP performs only generation")
    def prefill(self, prompt: Sequence[int]):
        """Prompt rows at positions 0..t-1 followed by k mask rows at t..t+k-1 under a causal mask.

        The mask vector is the mean of the prompt embeddings.  The last prompt
        row yields the first generated token; mask row j yields the candidates
        for depth j of the first tree.  Only the prompt rows enter the cache.
        """
        sp, t, k = self.spec, len(prompt), self.spec.n_probes
        E = np.stack([self.model.embed(int(x)) for x in prompt])
        if sp.mask_init == "last_k" and k:
            self.m = mask_init_last_k(E, k)
        elif sp.mask_init == "given":
            self.m = self.given_mask.copy()
        else:
            self.m = np.tile(mask_init_mean(E), (max(k, 1), 1))
        M = t + k
        x = np.concatenate([E, self.m[:k]], axis=0) if k else E
        vis = np.tril(np.ones((M, M), np.uint8))
        want = np.zeros(M, np.uint8)
        want[t - 1:] = 1
        logits, kb, vb, _ = self.model.block_forward(self.kc, self.vc, 0, x, np.arange(M), vis, want)
        self.kc[:, :t] = kb[:, :t]
        self.vc[:, :t] = vb[:, :t]
        self.L = t
        y = next_token(logits[t - 1], t, sp)
        self._emit(y)
        if not sp.ema_per_token:
            self.m = mask_update(self.m, self.model.embed(y), sp.lam)
        ids, vals, lses = self._probe_lists(logits, range(t, t + k))
        self.tree = next_tree(y, ids, vals, lses, sp) if k else root_only(y)
        rec = {"kind": "prefill", "first": y, "L_after": t, "probe_pos": list(range(t, t + k))}
        if self.keep_logits:
            rec["logits"] = logits[t - 1:].copy()
        self.log.append(rec)
        return y

    # -- one decode-and-verify step (Figure 1 right)
    def step(self, forced_tree: Optional[Tree] = None) -> List[int]:
        sp, k = self.spec, self.spec.n_probes
        tree = forced_tree if forced_tree is not None else self.tree
        blk = layout_block(tree, sp)
        x = self._rows_x(blk)
        pos = self.L + blk.row_pos_off
        logits, kb, vb, _ = self.model.block_forward(self.kc, self.vc, self.L, x, pos, blk.vis)
        # node r sits at position pos[r]; its logits decide the token at pos[r] + 1
        nxt = [next_token(logits[r], int(pos[r]) + 1, sp) for r in range(blk.n_nodes)]
        path, out = verify_walk(tree, nxt)
        a = len(path) - 1
        # the accepted nodes' keys/values become cache entries (Appendix E: the cache grows by the
        # number of generated tokens); mask rows and rejected nodes are never cached
        for j, p in enumerate(path):
            self.kc[:, self.L + j] = kb[:, p]
            self.vc[:, self.L + j] = vb[:, p]
        self.L += a + 1
        for y in out:
            self._emit(y)
        if not sp.ema_per_token:
            self.m = mask_update(self.m, self.model.embed(out[-1]), sp.lam)
        # next proposals come from the mask chain of the deepest anchored node on the accepted path
        ids = vals = lses = ()
        rows: List[int] = []
        if k:
            _, _, rows = draft_source(tree, blk, path, sp)
            ids, vals, lses = self._probe_lists(logits, rows)
        rec = {"kind": "step", "tree": tree, "block": blk, "next_of_node": nxt, "path": path, "emitted": out,
               "cand_ids": ids, "cand_vals": vals, "lses": lses, "L_after": self.L,
               "probe_pos": [int(pos[r]) for r in rows]}
        if self.keep_logits:
            rec["logits"] = logits
        self.log.append(rec)
        self.tree = next_tree(out[-1], ids, vals, lses, sp) if k else root_only(out[-1])
        self.steps += 1
        self.accept_hist.append(a)
        return out

    def generate(self, prompt: Sequence[int], max_new: int) -> List[int]:
        """Emit exactly max_new tokens (the last step's surplus is cut)."""
        self.prefill(prompt)
        while len(self.emitted) < max_new:
            self.step()
        return self.emitted[:max_new]

    @property
    def tau(self) -> float:
        """Emitted tokens per decode step; the prefill's token and call are excluded from both counts."""
        return acceptance_length(len(self.emitted) - 1, self.steps) if self.steps else float("nan")


def greedy_generate(model: OracleModel, prompt: Sequence[int], max_new: int, cap: int, return_logits=False,
                    spec: Optional[SpecCfg] = None):
    """Plain autoregressive decoding, one token per model call (Section 2, first equation): greedy, or sampled
    with spec.temperature / spec.seed when a spec with temperature > 0 is given."""
    spec = spec if spec is not None else SpecCfg()
    kc, vc = model.new_cache(cap)
    t = len(prompt)
    E = np.stack([model.embed(int(x)) for x in prompt])
    want = np.zeros(t, np.uint8)
    want[t - 1] = 1
    logits, kb, vb, _ = model.block_forward(kc, vc, 0, E, np.arange(t), np.tril(np.ones((t, t), np.uint8)), want)
    kc[:, :t], vc[:, :t] = kb, vb
    L = t
    out = [next_token(logits[t - 1], t, spec)]
    all_logits = [logits[t - 1].copy()]
    while len(out) < max_new:
        x = model.embed(out[-1])[None]
        logits, kb, vb, _ = model.block_forward(kc, vc, L, x, np.array([L]), np.ones((1, 1), np.uint8))
        kc[:, L], vc[:, L] = kb[:, 0], vb[:, 0]
        L += 1
        out.append(next_token(logits[0], L, spec))
        all_logits.append(logits[0].copy())
    return (out, np.stack(all_logits)) if return_logits else out
