"""Pins for the oracle's ESP logic (oracle/esp.py) against what the paper and the mathematics fix."""
import itertools
import math
import os

import numpy as np
import pytest

import synth
from oracle import esp

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    out = []
    for line in open(os.path.join(GOLD, name)):
        line = line.strip()
        if line and not line.startswith("#"):
            out.append(line.split())
    return out


# ---------------------------------------------------------------- metric definitions
def test_tau_and_call_reduction_match_the_papers_tables():
    for model, bc, tau, red in _rows("paper_tau_vs_call_reduction.txt"):
        assert abs(esp.call_reduction_percent(float(tau)) - float(red)) <= 0.006, (model, bc)
    # tau counts the bonus token: 10 model calls that emitted 17 tokens
    assert esp.acceptance_length(17, 10) == pytest.approx(1.7)


def test_block_complexity_worked_sizes():
    for k, bc, nodes, widths in _rows("paper_block_sizes.txt"):
        k, bc, nodes = int(k), int(bc), int(nodes)
        widths = [int(x) for x in widths.split(",")]
        assert esp.block_complexity(k, widths) == bc
        assert 1 + sum(widths) == nodes == bc // (k + 1)
    assert esp.block_complexity(3, [7, 5, 3]) == 64  # the paper's "BC=60" three-mask setting


# ---------------------------------------------------------------- mask token
def test_mask_init_is_prompt_mean_and_ema_closed_form():
    rng = np.random.default_rng(0)
    E = rng.standard_normal((13, 32)).astype(np.float32)
    m0 = esp.mask_init_mean(E)
    np.testing.assert_allclose(m0, E.astype(np.float64).mean(0), atol=1e-6)
    lam = 0.1
    es = rng.standard_normal((9, 32)).astype(np.float32)
    m = m0
    for e in es:
        m = esp.mask_update(m, e, lam)
    n = len(es)
    closed = (1 - lam) ** n * m0.astype(np.float64) + lam * sum((1 - lam) ** (n - 1 - i) * es[i].astype(np.float64) for i in range(n))
    np.testing.assert_allclose(m, closed, atol=1e-5)
    # lambda = 1 replaces the mask by the newest embedding, lambda = 0 freezes it
    assert np.array_equal(esp.mask_update(m0, es[0], 1.0), (m0 + (es[0] - m0)).astype(np.float32))
    assert np.array_equal(esp.mask_update(m0, es[0], 0.0), m0)


# ---------------------------------------------------------------- Top-K
def test_topk_equals_repeated_argmax_with_id_tiebreak():
    rng = np.random.default_rng(1)
    x = rng.integers(-5, 6, size=200).astype(np.float32)  # many exact ties
    ids, vals = esp.topk_desc(x, 17)
    y = x.copy().astype(np.float64)
    for j in range(17):
        best = int(np.argmax(y))  # numpy's argmax returns the lowest index among equals
        assert ids[j] == best and vals[j] == x[best]
        y[best] = -np.inf
    assert esp.log_sum_exp(x) == pytest.approx(math.log(np.exp(x.astype(np.float64)).sum()), abs=1e-5)


# ---------------------------------------------------------------- tree construction
def _lists(rng, k, kp, vocab=50):
    ids, vals, lses = [], [], []
    for _ in range(k):
        logits = rng.standard_normal(vocab).astype(np.float32) * 2
        i, v = esp.topk_desc(logits, kp)
        ids.append(i); vals.append(v); lses.append(esp.log_sum_exp(logits))
    return ids, vals, lses


def _paths(tree):
    out = set()
    for i in range(1, tree.n):
        p, a = [], i
        while a > 0:
            p.append(int(tree.tokens[a]))
            a = int(tree.parents[a])
        out.add(tuple(reversed(p)))
    return out


def _check_tree_invariants(tree, spec):
    assert tree.n <= spec.max_nodes and tree.parents[0] == -1 and tree.depths[0] == 0
    for i in range(1, tree.n):
        p = int(tree.parents[i])
        assert 0 <= p < i                                  # breadth-first order, ancestor-closed
        assert tree.depths[i] == tree.depths[p] + 1
        assert tree.depths[i] >= tree.depths[i - 1]
        assert tree.logp[i] <= tree.logp[p]                # "each child inherits the probability of its parent"
        if spec.prune_parent:
            assert tree.tokens[i] != tree.tokens[p]        # Section 3.5
        sib = [int(tree.tokens[j]) for j in range(1, tree.n) if tree.parents[j] == p]
        assert len(sib) == len(set(sib))


@pytest.mark.parametrize("k,K,B", [(2, 3, 6), (3, 3, 9), (3, 4, 14), (2, 5, 30)])
def test_dynamic_tree_all_expanded_equals_brute_force(k, K, B):
    """W = 0 (Algorithm 1's loop as printed): the tree must be the B-1 most probable prefixes of the full
    product tree, scored by the product of per-depth probabilities."""
    rng = np.random.default_rng(k * 100 + K * 10 + B)
    spec = esp.SpecCfg(n_probes=k, topk=K, max_nodes=B, expand_width=0, prune_parent=True)
    root = 7
    ids, vals, lses = _lists(rng, k, spec.k_prime)
    ids[0][1] = root  # make the pruner bite at depth 1
    tree = esp.build_tree(root, ids, vals, lses, spec)
    _check_tree_invariants(tree, spec)
    # brute force: enumerate every node of the full product tree
    nodes = {}

    def grow(path, parent_tok, score, depth):
        if depth == k:
            return
        pool = [(int(t), float(v) - float(lses[depth])) for t, v in zip(ids[depth], vals[depth]) if int(t) != parent_tok]
        for t, lp in pool[:min(K, B - depth - 1)]:
            nodes[path + (t,)] = score + lp
            grow(path + (t,), t, score + lp, depth + 1)

    grow((), root, 0.0, 0)
    best = sorted(nodes.items(), key=lambda kv: -kv[1])[:B - 1]
    assert _paths(tree) == {p for p, _ in best}
    assert tree.n == min(B, 1 + len(nodes))


def test_dynamic_tree_top1_expansion_is_a_merge_of_the_k_lists():
    """W = 1 (Section 3.4, Appendix D): all depth-i nodes hang under the Top-1 node of depth i-1, so the tree
    is the B-1 best entries of the k pruned lists, list i shifted by the chain's cumulative log-probability."""
    rng = np.random.default_rng(5)
    k, K, B = 3, 6, 12
    spec = esp.SpecCfg(n_probes=k, topk=K, max_nodes=B, expand_width=1)
    root = 3
    ids, vals, lses = _lists(rng, k, spec.k_prime)
    tree = esp.build_tree(root, ids, vals, lses, spec)
    _check_tree_invariants(tree, spec)
    merged, offset, parent_tok, chain = [], 0.0, root, ()
    for i in range(k):
        pool = [(int(t), float(v) - float(lses[i])) for t, v in zip(ids[i], vals[i]) if int(t) != parent_tok][:min(K, B - i - 1)]
        for t, lp in pool:
            merged.append((chain + (t,), offset + lp))
        chain, offset, parent_tok = chain + (pool[0][0],), offset + pool[0][1], pool[0][0]
    best = sorted(merged, key=lambda kv: -kv[1])[:B - 1]
    assert _paths(tree) == {p for p, _ in best}
    widths = [int((tree.depths == i).sum()) for i in range(1, k + 1)]
    assert sum(widths) == B - 1                       # sum_i K_i = B - 1: the budget is used up


def test_appendix_d_example_bc30_two_masks():
    """Appendix D, Figure 5: BC = 30 with two masks gives a 10-node tree drawn from the Top-9 of the first
    mask and the Top-8 of the second (Algorithm 1: top-(B-i)); the printed outcome keeps 7 and 2."""
    B, k = 30 // 3, 2
    spec = esp.SpecCfg(n_probes=k, topk=B, max_nodes=B, expand_width=1, prune_parent=False)
    p1 = [0.4, 0.1, 0.09, 0.08, 0.07, 0.06, 0.05, 0.02, 0.01, 0.005, 0.004]
    p2 = [0.5, 0.19, 0.04, 0.03, 0.02, 0.01, 0.009, 0.008, 0.007, 0.006, 0.005]
    ids = [np.arange(100, 111, dtype=np.int32), np.arange(200, 211, dtype=np.int32)]
    vals = [np.log(np.array(p, np.float32)) for p in (p1, p2)]
    tree = esp.build_tree(1, ids, vals, [0.0, 0.0], spec)
    assert tree.n == 10
    assert [int((tree.depths == i).sum()) for i in (1, 2)] == [7, 2]
    assert set(tree.tokens[tree.depths == 1]) == set(range(100, 107))
    assert list(tree.tokens[tree.depths == 2]) == [200, 201] and all(tree.tokens[tree.parents[tree.depths == 2]] == 100)
    np.testing.assert_allclose(np.exp(tree.logp[tree.depths == 2]), [0.2, 0.076], rtol=1e-5)
    # pools: at most B-1 = 9 candidates can come from the first mask and B-2 = 8 from the second
    flat = esp.build_tree(1, ids, [np.zeros(11, np.float32), vals[1] - 50], [0.0, 0.0], spec)
    assert int((flat.depths == 1).sum()) == 9
    deep = esp.build_tree(1, ids, [vals[0], np.zeros(11, np.float32)], [0.0, 0.0], spec)
    assert int((deep.depths == 2).sum()) == 8


def test_single_mask_trees_use_the_whole_budget():
    """Section 4.2: with one mask the widths are [4] and [14] for BC = 10 and 30 -- no dynamic choice left."""
    rng = np.random.default_rng(2)
    for bc, width in ((10, 4), (30, 14), (60, 29)):
        B = bc // 2
        spec = esp.SpecCfg(n_probes=1, topk=B, max_nodes=B, expand_width=1)
        ids, vals, lses = _lists(rng, 1, spec.k_prime, vocab=100)
        tree = esp.build_tree(5, ids, vals, lses, spec)
        assert tree.n - 1 == width and esp.layout_block(tree, spec).m == bc


def test_pruner_replaces_repeats_with_next_best():
    spec = esp.SpecCfg(n_probes=1, topk=3, max_nodes=8, expand_width=1, prune_parent=True)
    ids = [np.array([9, 4, 5, 6], np.int32)]
    vals = [np.array([3.0, 2.0, 1.0, 0.5], np.float32)]
    tree = esp.build_tree(9, ids, vals, [4.0], spec)       # the best candidate repeats the root token
    assert list(tree.tokens) == [9, 4, 5, 6]
    off = esp.build_tree(9, ids, vals, [4.0], esp.SpecCfg(n_probes=1, topk=3, max_nodes=8, prune_parent=False))
    assert list(off.tokens) == [9, 9, 4, 5]
    st = esp.build_static_tree(9, [ids[0], np.array([4, 7, 8], np.int32)], [2, 1], spec)
    assert list(st.tokens) == [9, 4, 5, 7] and list(st.parents) == [-1, 0, 0, 1]


# ---------------------------------------------------------------- block layout and verification
def test_block_layout_rows_positions_and_mask():
    """Static [3,2] tree with two masks per node, the example of Appendix E / Figure 6."""
    tree = esp.Tree(np.array([10, 11, 12, 13, 14, 15], np.int32), np.array([-1, 0, 0, 0, 1, 1], np.int32),
                    np.array([0, 1, 1, 1, 2, 2], np.int32), np.zeros(6, np.float32))
    paper = esp.layout_block(tree, esp.SpecCfg(n_probes=2, n_anchor=0))
    assert paper.m == esp.block_complexity(2, [3, 2]) == 18          # (k+1)(1+sum K_i)
    assert list(paper.row_token[:6]) == [10, 11, 12, 13, 14, 15] and all(paper.row_token[6:] == -1)
    assert list(paper.row_pos_off[:6]) == [0, 1, 1, 1, 2, 2]
    r1, r2 = paper.probe_row[(4, 1)], paper.probe_row[(4, 2)]         # masks of node 4 (depth 2, path 0-1-4)
    assert (paper.row_pos_off[r1], paper.row_pos_off[r2]) == (3, 4)
    assert set(np.nonzero(paper.vis[r1])[0]) == {0, 1, 4, r1}
    assert set(np.nonzero(paper.vis[r2])[0]) == {0, 1, 4, r1, r2}
    assert set(np.nonzero(paper.vis[5])[0]) == {0, 1, 5}
    lean = esp.layout_block(tree, esp.SpecCfg(n_probes=2, n_anchor=1))
    assert lean.m == 6 + 2 and lean.anchors == [0]
    assert set(np.nonzero(lean.vis[7])[0]) == {0, 6, 7}
    # mask stays lower-triangular: every row only sees earlier rows and itself
    assert not np.triu(paper.vis, 1).any()


def test_verify_walk_accepts_longest_matching_path():
    tree = esp.Tree(np.array([1, 20, 21, 30, 31, 40], np.int32), np.array([-1, 0, 0, 1, 1, 4], np.int32),
                    np.array([0, 1, 1, 2, 2, 3], np.int32), np.zeros(6, np.float32))
    # model's next token after each node:  root->20, node1(20)->31, node4(31)->40, node5(40)->99
    nxt = [20, 31, 0, 0, 40, 99]
    path, out = esp.verify_walk(tree, nxt)
    assert path == [0, 1, 4, 5] and out == [20, 31, 40, 99]
    path, out = esp.verify_walk(tree, [22, 31, 0, 0, 40, 99])           # first draft wrong: only the bonus token
    assert path == [0] and out == [22]
    path, out = esp.verify_walk(tree, [21, 31, 55, 0, 40, 99])
    assert path == [0, 2] and out == [21, 55]


# ---------------------------------------------------------------- losslessness end to end
@pytest.mark.parametrize("W,n_anchor,prune", [(0, 0, True), (1, 0, False), (0, 1, False), (1, 1, True)])
def test_esp_output_equals_greedy_decoding(W, n_anchor, prune):
    """Section 2: verification is lossless -- ESP must emit exactly the greedy autoregressive stream."""
    shape = synth.TINY.replace(n_layers=2, d_model=64, n_q_heads=4, n_kv_heads=2, head_dim=16, d_ffn=160, vocab=97)
    w = synth.make_weights(shape, seed=21, gain_jitter=True, std=0.3)
    model = esp.OracleModel(shape, w)
    prompt = synth.make_prompt(shape.vocab, 17, 3)
    ref = esp.greedy_generate(model, prompt, 40, 128)
    spec = esp.SpecCfg(n_probes=3, topk=4, max_nodes=12, expand_width=W, n_anchor=n_anchor, prune_parent=prune)
    dec = esp.EspOracle(model, spec, 256)
    out = dec.generate(prompt, 40)
    assert out == ref
    assert len(set(ref)) > 5                      # not a degenerate constant stream
    assert 1.0 <= dec.tau <= spec.n_probes + 1    # at most k drafts + the bonus token per call
    assert sum(a + 1 for a in dec.accept_hist) == len(dec.emitted) - 1
    for rec in (r for r in dec.log if r["kind"] == "step"):
        _check_tree_invariants(rec["tree"], spec)
        expect_rows = (spec.n_probes + 1) * rec["tree"].n if n_anchor == 0 else rec["tree"].n + spec.n_probes
        assert rec["block"].m == expect_rows


def test_forced_perfect_draft_is_fully_accepted():
    """If the draft tree contains the true continuation, verification must accept all of it plus a bonus token."""
    shape = synth.TINY.replace(n_layers=1, d_model=32, n_q_heads=2, n_kv_heads=1, head_dim=16, d_ffn=64, vocab=61)
    w = synth.make_weights(shape, seed=4, std=0.3)
    model = esp.OracleModel(shape, w)
    prompt = synth.make_prompt(shape.vocab, 9, 8)
    ref = esp.greedy_generate(model, prompt, 12, 64)
    dec = esp.EspOracle(model, esp.SpecCfg(n_probes=2, topk=3, max_nodes=8), 64)
    assert dec.prefill(prompt) == ref[0]
    chain = esp.Tree(np.array(ref[0:4], np.int32), np.array([-1, 0, 1, 2], np.int32), np.arange(4, dtype=np.int32),
                     np.zeros(4, np.float32))
    out = dec.step(forced_tree=chain)
    assert out == ref[1:5] and dec.L == len(prompt) + 4
    assert dec.generate.__self__.emitted == ref[:5]
    while len(dec.emitted) < 12:
        dec.step()
    assert dec.emitted[:12] == ref


# ---------------------------------------------------------------- static trees (Section 4.2)
@pytest.mark.parametrize("widths,n_anchor", [((7, 2), 0), ((5, 4), 0), ((4,), 0), ((7, 5, 3), 1)])
def test_static_tree_generation_is_lossless_and_has_the_papers_block_size(widths, n_anchor):
    """Fixed branch widths [K_1..K_k]: the tree has 1 + sum K_i nodes whenever the probes offer enough
    candidates, every node carries k masks in the paper's layout (BC = (k+1)(1 + sum K_i): [7,2] -> 30,
    [4] -> 10), the Top-1 node of each depth is the only one with children, and decoding stays lossless."""
    k = len(widths)
    shape = synth.TINY.replace(n_layers=2, d_model=64, n_q_heads=4, n_kv_heads=2, head_dim=16, d_ffn=160, vocab=97)
    w = synth.make_weights(shape, seed=22, gain_jitter=True, std=0.3)
    model = esp.OracleModel(shape, w)
    prompt = synth.make_prompt(shape.vocab, 15, 4)
    ref = esp.greedy_generate(model, prompt, 30, 128)
    spec = esp.SpecCfg(n_probes=k, topk=1, max_nodes=1, n_anchor=n_anchor, static_widths=widths)
    dec = esp.EspOracle(model, spec, 256)
    assert dec.generate(prompt, 30) == ref
    full = 0
    for rec in dec.log:
        if rec["kind"] != "step":
            continue
        t = rec["tree"]
        assert t.n <= 1 + sum(widths)
        for d in range(1, k + 1):
            nodes = [i for i in range(t.n) if t.depths[i] == d]
            assert len(nodes) <= widths[d - 1]
            assert len({int(t.parents[i]) for i in nodes}) <= 1          # one parent per depth
            if nodes and d > 1:
                prev = [i for i in range(t.n) if t.depths[i] == d - 1]
                assert int(t.parents[nodes[0]]) == prev[0]               # ... the first (Top-1) node of the depth above
        if n_anchor == 0 and t.n == 1 + sum(widths):
            full += 1
            assert rec["block"].m == esp.block_complexity(k, widths)
    if n_anchor == 0:
        assert full > 0


# ---------------------------------------------------------------- mask initialisations (Section 4, mask designs)
def test_mask_init_variants():
    shape = synth.TINY.replace(n_layers=2, d_model=64, n_q_heads=4, n_kv_heads=2, head_dim=16, d_ffn=160, vocab=97)
    w = synth.make_weights(shape, seed=23, gain_jitter=True, std=0.3)
    model = esp.OracleModel(shape, w)
    prompt = synth.make_prompt(shape.vocab, 13, 5)
    E = np.stack([model.embed(int(x)) for x in prompt])
    ref = esp.greedy_generate(model, prompt, 24, 128)
    # Last K: the k masks are the embeddings of the last k prompt tokens, in prompt order
    lk = esp.mask_init_last_k(E, 3)
    assert np.array_equal(lk, E[-3:]) and np.array_equal(esp.mask_init_last_k(E[:2], 3), np.stack([E[0], E[0], E[1]]))
    base = esp.SpecCfg(n_probes=3, topk=4, max_nodes=12, expand_width=0, n_anchor=1)
    runs = {}
    for mode in ("mean", "last_k", "given"):
        dec = esp.EspOracle(model, esp.SpecCfg(**{**base.__dict__, "mask_init": mode}), 256)
        if mode == "given":
            dec.set_mask(np.tile(esp.mask_init_mean(E), (3, 1)))      # the prompt mean, given from outside
        assert dec.generate(prompt, 24) == ref                        # lossless whatever the masks are
        runs[mode] = dec
    # giving the prompt mean from outside is the mean initialisation: same trees, same masks, step by step
    a, b = runs["mean"], runs["given"]
    assert a.accept_hist == b.accept_hist and np.array_equal(a.m, b.m)
    assert all(np.array_equal(x["tree"].tokens, y["tree"].tokens) for x, y in zip(a.log, b.log) if x["kind"] == "step")
    # Last K starts from different vectors per mask, and every vector follows Eq. (mask_update_mean)
    c = runs["last_k"]
    want = lk.copy()
    for y in c.emitted:
        want = esp.mask_update(want, model.embed(y), base.lam)
    np.testing.assert_allclose(c.m, want, rtol=0, atol=1e-6)
    assert not np.allclose(c.m[0], c.m[2])


# ---------------------------------------------------------------- sampling verification (temperature > 0)
def test_philox_known_answers():
    """The counter-based generator against the published known-answer vectors."""
    rows = _rows("philox4x32_10_kat.txt")
    assert len(rows) == 3
    for r in rows:
        w = [int(x, 16) for x in r]
        assert esp.philox4x32_10(w[0:4], w[4:6]) == w[6:10]


def test_uniform_mapping_and_logarithm():
    """u = (2n+1)/2^24 with n the top 23 bits: strictly inside (0,1) and exact; the written-out fp32 logarithm
    agrees with the fp64 library logarithm to fp32 accuracy over the whole range the noise uses."""
    lib = esp._load()
    assert lib.orc_uniform_from_bits(0) == 2.0 ** -24
    assert lib.orc_uniform_from_bits(0xffffffff) == 1.0 - 2.0 ** -24
    assert lib.orc_uniform_from_bits(0x80000000) == 0.5 + 2.0 ** -24
    assert lib.orc_uniform_from_bits(0x000001ff) == 2.0 ** -24          # the low 9 bits are not used
    rng = np.random.default_rng(5)
    xs = np.concatenate([np.exp(rng.uniform(np.log(5e-8), np.log(20.0), 30000)),
                         [2.0 ** -24, 1 - 2.0 ** -24, 1.0, 0.5, 2.0, 0.70710677, 0.7071068, 16.635532]]).astype(np.float32)
    for x in xs:
        ref = math.log(float(x))
        got = lib.orc_det_logf(float(x))
        assert abs(got - ref) <= 3e-7 * max(abs(ref), 1.0), (x, got, ref)
    assert lib.orc_det_logf(1.0) == 0.0
    # -log(1 - 2^-24) must not collapse to 0: the second logarithm needs a positive argument
    assert lib.orc_det_logf(1.0 - 2.0 ** -24) < 0.0


def test_gumbel_noise_moments_and_keys():
    """Standard Gumbel: mean = Euler-Mascheroni constant, variance = pi^2/6; the noise is a function of
    (seed, position, token) and of nothing else."""
    g = np.concatenate([esp.gumbel_noise(7, p, 50000) for p in range(8)]).astype(np.float64)
    n = g.size
    assert abs(g.mean() - 0.5772156649) < 5 * math.sqrt(math.pi ** 2 / 6 / n)
    assert abs(g.var() - math.pi ** 2 / 6) < 0.03
    a = esp.gumbel_noise(7, 3, 1000)
    assert np.array_equal(a, esp.gumbel_noise(7, 3, 1000))
    assert np.array_equal(a[:10], esp.gumbel_noise(7, 3, 10))             # token v does not depend on the vocabulary size
    assert not np.array_equal(a, esp.gumbel_noise(7, 4, 1000))
    assert not np.array_equal(a, esp.gumbel_noise(8, 3, 1000))
    assert not np.array_equal(a, esp.gumbel_noise(7 + (1 << 32), 3, 1000))  # the high seed word is used
    # token v at position p is Philox word 0 of counter (v, p, 0, 0)
    x = esp.philox4x32_10([5, 3, 0, 0], [7, 0])[0]
    assert a[5] == esp._load().orc_gumbel_from_bits(x)


@pytest.mark.parametrize("temperature", [1.0, 2.0, 0.5])
def test_gumbel_max_draws_follow_the_softmax(temperature):
    """argmax(logits/T + g) is a draw from softmax(logits/T): chi-square of 60000 draws against the exact
    probabilities (5 degrees of freedom; 0.9999 quantile = 25.7)."""
    logits = np.array([1.3, -0.2, 0.7, 2.1, -1.5, 0.0], dtype=np.float32)
    p = np.exp(logits.astype(np.float64) / temperature)
    p /= p.sum()
    spec = esp.SpecCfg(temperature=temperature, seed=12345)
    n = 60000
    counts = np.zeros(len(logits))
    for pos in range(n):
        counts[esp.next_token(logits, pos, spec)] += 1
    chi2 = float(((counts - n * p) ** 2 / (n * p)).sum())
    assert chi2 < 25.7, (chi2, counts / n, p)


def test_temperature_zero_is_the_argmax_and_ties_go_to_the_lower_id():
    logits = np.array([0.5, 2.0, 2.0, -1.0], dtype=np.float32)
    assert esp.next_token(logits, 11, esp.SpecCfg()) == 1
    # with noise, the winner is the arg-max of the fp32 scores under the same tie rule
    spec = esp.SpecCfg(temperature=1.0, seed=3)
    s = esp.sample_scores(logits, 11, 1.0, 3)
    assert s.dtype == np.float32
    assert esp.next_token(logits, 11, spec) == int(np.flatnonzero(s == s.max())[0])
    assert np.array_equal(s, logits + esp.gumbel_noise(3, 11, 4))


@pytest.mark.parametrize("W,n_anchor,temperature", [(0, 0, 1.0), (1, 1, 1.0), (0, 1, 0.7)])
def test_sample_matching_is_lossless_token_by_token(W, n_anchor, temperature):
    """Section 4 "sample matching": with the draw at a position fixed by (seed, position), ESP emits exactly
    the stream plain autoregressive sampling emits; another seed gives another stream."""
    shape = synth.TINY.replace(n_layers=2, d_model=64, n_q_heads=4, n_kv_heads=2, head_dim=16, d_ffn=160, vocab=97)
    w = synth.make_weights(shape, seed=21, gain_jitter=True, std=0.3)
    model = esp.OracleModel(shape, w)
    prompt = synth.make_prompt(shape.vocab, 17, 3)
    spec = esp.SpecCfg(n_probes=3, topk=4, max_nodes=12, expand_width=W, n_anchor=n_anchor,
                       temperature=temperature, seed=99)
    ref = esp.greedy_generate(model, prompt, 40, 128, spec=spec)
    dec = esp.EspOracle(model, spec, 256)
    assert dec.generate(prompt, 40) == ref
    assert ref != esp.greedy_generate(model, prompt, 40, 128)                       # not the greedy stream
    other = dataclasses_replace(spec, seed=100)
    assert ref != esp.greedy_generate(model, prompt, 40, 128, spec=other)
    assert sum(a + 1 for a in dec.accept_hist) == len(dec.emitted) - 1


def dataclasses_replace(spec, **kw):
    import dataclasses
    return dataclasses.replace(spec, **kw)


# ---------------------------------------------------------------- which mask row proposes which depth (Section 2; Appendix E)
class _PositionPredictor:
    """Stand-in for the frozen model with a known answer at every position: whatever a row holds, a row at
    position p puts token g(p + 1) first (and g(p + 1) + 1, ... after it).  Section 2 says mask i elicits the
    token i + 1 positions ahead, i.e. a mask row at position p proposes the token of position p + 1: under
    this model every drafted node is right exactly when each depth of the tree was drawn from the mask row one
    position before it, and the walk then accepts the whole tree."""

    def __init__(self, vocab=61, d=4):
        self.V, self.d, self.n_layers = vocab, d, 1
        self.calls = []

    def g(self, p):          # token at position p; consecutive tokens differ, so the pruner never removes a right draft
        return (7 * p + 3) % self.V

    def embed(self, token):
        return np.full(self.d, float(token), np.float32)

    def new_cache(self, cap):
        z = np.zeros((1, cap, 1, 1), np.float32)
        return z, z.copy()

    def block_forward(self, kc, vc, L, x, pos, vis, want=None, need_hidden=False):
        M = len(pos)
        self.calls.append([int(p) for p in pos])
        logits = np.zeros((M, self.V), np.float32)
        for r in range(M):
            first = self.g(int(pos[r]) + 1)
            for j in range(self.V):
                logits[r, (first + j) % self.V] = -0.5 * j
        kb = np.zeros((1, M, 1, 1), np.float32)
        return logits, kb, kb.copy(), None


@pytest.mark.parametrize("n_anchor,k", [(0, 3), (1, 3), (2, 4), (0, 1)])
def test_mask_rows_feed_the_depth_one_position_ahead(n_anchor, k):
    model = _PositionPredictor()
    t = 9
    prompt = [model.g(p) for p in range(t)]
    spec = esp.SpecCfg(n_probes=k, topk=3, max_nodes=3 * k + 1, expand_width=1, n_anchor=n_anchor)
    dec = esp.EspOracle(model, spec, 256)
    out = dec.generate(prompt, 40)
    assert out == [model.g(p) for p in range(t, t + 40)]
    # position identity, every record: the row proposing depth i of the next tree sits at (new L) + i - 1
    for rec in dec.log:
        assert rec["probe_pos"] == [rec["L_after"] + i - 1 for i in range(1, len(rec["probe_pos"]) + 1)], rec["kind"]
    assert dec.log[0]["probe_pos"] == [t + j - 1 for j in range(1, k + 1)]          # prefill: mask j at t + j - 1
    # behaviour: each step accepts every depth it drafted.  Paper mode (all nodes anchored): k per step.
    # Fewer anchors: the chain behind the deepest anchored accepted node has k - delta rows left.
    steps = [r for r in dec.log if r["kind"] == "step"]
    drafted = [int(r["tree"].depths.max()) for r in steps]
    assert dec.accept_hist == drafted
    if n_anchor == 0:
        assert all(a == k for a in dec.accept_hist)
    else:
        assert max(dec.accept_hist) == k and any(len(r["probe_pos"]) < k for r in steps)   # delta > 0 occurs


def test_a_shifted_mask_row_choice_is_caught():
    """Negative control for the pin above: feeding depth i from the row one further along the chain (delta
    off by one) or from the chain in reverse order drafts wrong tokens under the position predictor."""
    model = _PositionPredictor()
    t, k = 9, 3
    prompt = [model.g(p) for p in range(t)]
    spec = esp.SpecCfg(n_probes=k, topk=3, max_nodes=3 * k + 1, expand_width=1, n_anchor=0)
    for wrong in ("shift", "reverse"):
        dec = esp.EspOracle(model, spec, 256)
        dec.prefill(prompt)
        tree, blk = dec.tree, esp.layout_block(dec.tree, spec)
        pos = dec.L + blk.row_pos_off
        logits, _, _, _ = model.block_forward(None, None, dec.L, None, pos, blk.vis)
        nxt = [int(np.argmax(logits[r])) for r in range(blk.n_nodes)]
        path, emitted = esp.verify_walk(tree, nxt)
        _, _, rows = esp.draft_source(tree, blk, path, spec)
        bad = rows[1:] if wrong == "shift" else rows[::-1]
        lists = [esp.topk_desc(logits[r], spec.k_prime) for r in bad]
        nt = esp.build_tree(emitted[-1], [l[0] for l in lists], [l[1] for l in lists],
                            [esp.log_sum_exp(logits[r]) for r in bad], spec)
        L_new = dec.L + len(path)
        right = esp.build_tree(emitted[-1], *zip(*[(esp.topk_desc(logits[r], spec.k_prime)[0], esp.topk_desc(logits[r], spec.k_prime)[1],
                                                    esp.log_sum_exp(logits[r])) for r in rows]), spec)
        top = lambda tr: [int(tr.tokens[i]) for i in range(1, tr.n) if tr.logp[i] == max(tr.logp[j] for j in range(tr.n) if tr.depths[j] == tr.depths[i])]
        assert top(right)[:2] == [model.g(L_new + 1), model.g(L_new + 2)]
        assert top(nt)[:1] != [model.g(L_new + 1)]
