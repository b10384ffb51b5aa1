"""GPU parity tests (need a B200): the CUDA library, called through its C ABI, against the CPU oracle."""
import numpy as np
import pytest
import torch

import synth
from oracle import esp as O

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def pu():
    from tests import parity_util
    return parity_util


TOL_FP32 = 1e-4   # of the logit range, fp32 model
TOL_BF16 = 2e-2   # of the logit range, bf16 model


# ------------------------------------------------------------------ config 1: tiny fp32 model, full length
@pytest.mark.parametrize("W,n_anchor,prune", [(0, 1, True), (0, 1, False), (1, 0, False), (0, 0, False)])
def test_tiny_fp32_full_parity(pu, W, n_anchor, prune):
    shape = synth.TINY
    w = synth.make_weights(shape, seed=0)
    prompt = synth.make_prompt(shape.vocab, 64, 0)
    B = 32 if n_anchor == 1 else 20
    spec = O.SpecCfg(n_probes=3, topk=4, max_nodes=B, expand_width=W, n_anchor=n_anchor, prune_parent=prune)
    run = pu.ParityRun(shape, w, spec, prompt, 64, TOL_FP32)
    out = run.run()
    model = O.OracleModel(shape, w)
    assert out == O.greedy_generate(model, prompt, 64, 256)           # lossless, and equal to the oracle stream
    dec = O.EspOracle(model, spec, 512)
    assert out == dec.generate(prompt, 64)
    assert run.accepts == dec.accept_hist[:len(run.accepts)]          # same accepted lengths, step by step
    g, _ = pu.gpu_generate(shape, run.wd, pu.GREEDY, prompt, 64)
    assert g == out                                                   # GPU ESP == GPU greedy
    if not prune:
        assert max(run.accepts) >= 1                                  # drafts really get accepted here
    run.close()


@pytest.mark.parametrize("widths,n_anchor", [((7, 2), 0), ((15, 4), 0), ((7, 5, 3), 1)])
def test_tiny_fp32_static_tree_parity(pu, widths, n_anchor):
    """Static trees with the paper's branch widths ([7,2] = BC 30, [15,4] = BC 60 with two masks per node)."""
    shape = synth.TINY
    w = synth.make_weights(shape, seed=3, gain_jitter=True, std=0.3)
    prompt = synth.make_prompt(shape.vocab, 50, 7)
    spec = O.SpecCfg(n_probes=len(widths), topk=1, max_nodes=1, n_anchor=n_anchor, static_widths=widths)
    run = pu.ParityRun(shape, w, spec, prompt, 24, TOL_FP32)
    out = run.run()
    assert out == O.greedy_generate(O.OracleModel(shape, w), prompt, 24, 256)
    if n_anchor == 0:
        assert run.h.state()["n_rows"] <= (len(widths) + 1) * (1 + sum(widths))
    run.close()


@pytest.mark.parametrize("mode", ["last_k", "sample", "mu_plus_5_sigma"])
def test_tiny_fp32_mask_init_variants_parity(pu, mode):
    """Mask initialisations of Section 4: the last k prompt embeddings, a draw from N(mu, sigma^2 I) with the
    embedding table's mean and standard deviation (drawn here, handed over through esp_set_mask), mu + 5 sigma."""
    shape = synth.TINY
    w = synth.make_weights(shape, seed=3, gain_jitter=True, std=0.3)
    prompt = synth.make_prompt(shape.vocab, 50, 8)
    k = 3
    given = None
    if mode != "last_k":
        emb = w["embed"].float().numpy()
        mu, sigma = float(emb.mean()), float(emb.std())
        rng = np.random.default_rng(4)
        given = (mu + sigma * rng.standard_normal((k, shape.d_model))).astype(np.float32) if mode == "sample" \
            else np.full((k, shape.d_model), mu + 5 * sigma, np.float32)
    spec = O.SpecCfg(n_probes=k, topk=4, max_nodes=20, expand_width=0, n_anchor=1,
                     mask_init="last_k" if mode == "last_k" else "given")
    run = pu.ParityRun(shape, w, spec, prompt, 24, TOL_FP32, given_mask=given)
    out = run.run()
    assert out == O.greedy_generate(O.OracleModel(shape, w), prompt, 24, 256)
    run.close()


def test_tiny_fp32_nontrivial_stream(pu):
    """Same model family with wider weights and jittered norm gains, so the stream is not one repeated token."""
    shape = synth.TINY
    w = synth.make_weights(shape, seed=3, gain_jitter=True, std=0.3)
    prompt = synth.make_prompt(shape.vocab, 97, 5)       # ragged last prefill chunk (97 = 64 + 33)
    spec = O.SpecCfg(n_probes=3, topk=4, max_nodes=20, expand_width=1, n_anchor=0)
    run = pu.ParityRun(shape, w, spec, prompt, 40, TOL_FP32)
    out = run.run()
    assert len(set(out)) > 10
    assert out == O.greedy_generate(O.OracleModel(shape, w), prompt, 40, 256)
    g, _ = pu.gpu_generate(shape, run.wd, pu.GREEDY, prompt, 40)
    assert g == out
    run.close()


def test_forced_drafts_are_accepted_and_compacted(pu):
    """Drive acceptance lengths random-init models never reach: the tree is set to contain the true
    continuation (found by GPU greedy decoding), so several nodes are accepted and their KV rows move."""
    shape = synth.TINY
    w = synth.make_weights(shape, seed=3, gain_jitter=True, std=0.3)
    prompt = synth.make_prompt(shape.vocab, 40, 6)
    spec = O.SpecCfg(n_probes=2, topk=4, max_nodes=16, expand_width=0, n_anchor=1)
    run = pu.ParityRun(shape, w, spec, prompt, 48, TOL_FP32)
    truth, _ = pu.gpu_generate(shape, run.wd, pu.GREEDY, prompt, 48)
    st = run.prefill()
    rng = np.random.default_rng(0)
    while len(run.emitted) < 40:
        n = len(run.emitted)
        depth = int(rng.integers(0, 4))
        # a bushy tree: distractor siblings first, the true chain woven in at varying row indices
        toks, pars = [run.emitted[-1]], [-1]
        cur = 0
        for dpt in range(depth):
            sib = [int(t) for t in rng.integers(0, shape.vocab, size=int(rng.integers(0, 3))) if int(t) != truth[n + dpt]]
            for t in sib:
                toks.append(t); pars.append(cur)
            toks.append(truth[n + dpt]); pars.append(cur)
            nxt = len(toks) - 1
            cur = nxt
        order = sorted(range(len(toks)), key=lambda i: (0 if i == 0 else _depth(pars, i), i))
        remap = {o: i for i, o in enumerate(order)}
        forced = O.Tree(np.array([toks[o] for o in order], np.int32),
                        np.array([-1 if pars[o] < 0 else remap[pars[o]] for o in order], np.int32),
                        np.zeros(len(order), np.int32), np.zeros(len(order), np.float32))
        st = run.step(st, forced=forced)
        assert run.accepts[-1] >= depth
    assert run.emitted[:40] == truth[:40]
    assert max(run.accepts) >= 3
    s = run.h.stats()
    assert s.emitted == len(run.emitted) - 1 and s.steps == len(run.accepts) and s.device_error == 0
    assert list(s.accept_hist)[:5] == [run.accepts.count(a) for a in range(5)]
    run.close()


def _depth(pars, i):
    d = 0
    while pars[i] >= 0:
        i = pars[i]
        d += 1
    return d


# ------------------------------------------------------------------ bf16 models on the tensor-core path
BF16_SMALL = synth.TINY.replace(name="bf16-small", dtype="bf16", tied=False, n_layers=3, d_model=512, n_q_heads=4,
                                n_kv_heads=2, head_dim=128, d_ffn=688, vocab=5000)


@pytest.mark.parametrize("qk_norm,W,n_anchor,plen", [(True, 0, 1, 150), (False, 1, 0, 700)])
def test_bf16_small_parity(pu, qk_norm, W, n_anchor, plen):
    shape = BF16_SMALL.replace(qk_norm=qk_norm, rms_eps=1e-6 if qk_norm else 1e-5)
    w = synth.make_weights(shape, seed=1, gain_jitter=True, std=0.05)
    prompt = synth.make_prompt(shape.vocab, plen, 2)
    spec = O.SpecCfg(n_probes=3, topk=5, max_nodes=16 if n_anchor else 12, expand_width=W, n_anchor=n_anchor)
    run = pu.ParityRun(shape, w, spec, prompt, 32, TOL_BF16)
    out = run.run()
    assert len(set(out)) > 8
    g, _ = pu.gpu_generate(shape, run.wd, pu.GREEDY, prompt, 32)
    assert g == out                                      # bit-exact GPU ESP == GPU greedy
    # the CUDA-core GEMM path must agree with the tensor-core path to bf16 accuracy as well
    run2 = pu.ParityRun(shape, w, spec, prompt, 8, TOL_BF16, gemm_impl=1, w_dev=run.wd)
    run2.run()
    run.close(); run2.close()


def test_bf16_forced_acceptance_bitwise_equals_greedy(pu):
    """Accepted draft nodes must carry exactly the bits that plain decoding produces: force long accepted
    paths and compare the ESP stream, token for token, with GPU greedy decoding."""
    shape = BF16_SMALL
    w = synth.make_weights(shape, seed=4, gain_jitter=True, std=0.05)
    wd = pu.to_device(w)
    prompt = synth.make_prompt(shape.vocab, 333, 3)
    n_new = 96
    truth, _ = pu.gpu_generate(shape, wd, pu.GREEDY, prompt, n_new, max_seq_len=600)
    import paper_2603_17942_b200 as P
    spec = O.SpecCfg(n_probes=3, topk=5, max_nodes=24, expand_width=0, n_anchor=1)
    h = P.Handle(shape, pu.c_spec(spec), wd, max_seq_len=600)
    out = [h.prefill(prompt)]
    rng = np.random.default_rng(1)
    accepted = []
    while len(out) < n_new - 8:
        depth = int(rng.integers(0, 6))
        n = len(out)
        toks = [out[-1]] + [truth[n + i] for i in range(depth)]
        h.set_tree(np.array(toks, np.int32), np.arange(-1, depth, dtype=np.int32))
        new = h.step()
        accepted.append(len(new) - 1)
        out.extend(new)
    assert out == truth[:len(out)]
    assert max(accepted) >= 4 and sum(accepted) > len(accepted)
    assert h.stats().device_error == 0
    h.close()


@pytest.mark.parametrize("n_seq", [2, 3, 5])
def test_bf16_batch_of_sequences_equals_each_sequence_alone(pu, n_seq):
    """Sequences are independent (each has its own cache, masks and tree): a handle holding several of them,
    prefilled with different prompts (the last one later than the others), must emit for each exactly the stream
    a single-sequence handle emits.  On the tensor-core path up to three consecutive sequences share one pass
    through the layers (one weight stream, MMA N = 80 per sequence): 2 -> one pass of 2, 3 -> one pass of 3,
    5 -> passes of 3 and 2."""
    import paper_2603_17942_b200 as P
    shape = BF16_SMALL
    w = synth.make_weights(shape, seed=5, gain_jitter=True, std=0.05)
    wd = pu.to_device(w)
    spec = O.SpecCfg(n_probes=3, topk=5, max_nodes=16, expand_width=0, n_anchor=1)
    lens = (90, 300, 17, 130, 64)[:n_seq]
    prompts = [synth.make_prompt(shape.vocab, n, 10 + i) for i, n in enumerate(lens)]
    n_new, max_seq = 24, 400
    alone = []
    for pr in prompts:
        h1 = P.Handle(shape, pu.c_spec(spec), wd, max_seq_len=max_seq)
        alone.append(h1.generate(pr, n_new))
        h1.close()
    h = P.Handle(shape, pu.c_spec(spec), wd, max_seq_len=max_seq, max_batch=n_seq)
    outs = [[h.prefill(prompts[i], i)] for i in range(n_seq - 1)] + [[]]
    for step in range(200):
        if step == 3:
            outs[-1].append(h.prefill(prompts[-1], n_seq - 1))   # a sequence joins while the others are decoding
        if all(len(o) >= n_new for o in outs):
            break
        P.esp_step(h.h, h.tokens_out, h.n_out)
        for i in range(n_seq):
            outs[i].extend(int(t) for t in h.tokens_out[i, :h.n_out[i]])
    assert h.stats().device_error == 0
    for i in range(n_seq):
        assert outs[i][:n_new] == alone[i], f"sequence {i}"
    h.close()


# ------------------------------------------------------------------ config 3 / 4 kernel shapes (full width, few layers)
@pytest.mark.parametrize("base,topk,B", [(synth.LLAMA3_8B, 10, 64), (synth.QWEN3_8B, 8, 48)])
def test_full_width_shapes_parity(pu, base, topk, B):
    """Every GEMM, attention and LM-head launch has the shape it has in the full model (d_model 4096, 32/8
    heads of 128, the real FFN and vocabulary sizes, 4 probes, <= 64-node trees); only the layer count is cut
    so the CPU oracle finishes in seconds."""
    shape = base.replace(n_layers=2)
    w = synth.make_weights(shape, seed=0, device="cuda")
    wh = synth.weights_to_host(w)
    prompt = synth.make_prompt(shape.vocab, 200, 0)
    spec = O.SpecCfg(n_probes=4, topk=topk, max_nodes=B, expand_width=0, n_anchor=1)
    run = pu.ParityRun(shape, wh, spec, prompt, 4, TOL_BF16, w_dev=w)
    out = run.run()
    g, _ = pu.gpu_generate(shape, w, pu.GREEDY, prompt, 4)
    assert g == out
    assert run.h.stats().device_error == 0
    run.close()


def test_full_width_stream_is_invariant_across_cache_split_growth(pu):
    """While a sequence grows, the number of cache splits grows, the captured step graph changes with it and the
    attention launch moves from one CTA per (split, head group, row tile) to the persistent kernel.  None of this
    may change a bit: the ESP stream with forced multi-token acceptances stays equal to plain decoding while the
    length crosses several split boundaries, that hand-over among them."""
    import paper_2603_17942_b200 as P
    shape = synth.LLAMA3_8B.replace(n_layers=2)
    w = synth.make_weights(shape, seed=2, device="cuda")
    prompt = synth.make_prompt(shape.vocab, 1990, 8)
    n_new, max_seq = 640, 3000
    truth, _ = pu.gpu_generate(shape, w, pu.GREEDY, prompt, n_new, max_seq_len=max_seq)
    spec = O.SpecCfg(n_probes=4, topk=10, max_nodes=64, expand_width=0, n_anchor=1)
    h = P.Handle(shape, pu.c_spec(spec), w, max_seq_len=max_seq)
    out = [h.prefill(prompt)]
    rng = np.random.default_rng(3)
    while len(out) < n_new - 8:
        n = len(out)
        if rng.integers(0, 2):
            depth = int(rng.integers(1, 6))
            toks = [out[-1]] + [truth[n + i] for i in range(depth)]
            h.set_tree(np.array(toks, np.int32), np.arange(-1, depth, dtype=np.int32))
        out.extend(h.step())
    assert out == truth[:len(out)]
    assert len(prompt) + len(out) > 2304 + 256          # past the hand-over (10 splits of 256 keys) and one more split
    assert h.stats().device_error == 0
    h.close()


# ------------------------------------------------------------------ blocks of more than 80 rows (BC = 120)
@pytest.mark.parametrize("widths", [(), (15, 10, 4)])
def test_tiny_fp32_block_complexity_120_parity(pu, widths):
    """The paper's largest block: k = 3 masks behind every one of 30 tree nodes, BC = (k+1) * 30 = 120 rows
    (Section 3.3; Appendix on increasing block complexity), dynamic and static tree."""
    shape = synth.TINY
    w = synth.make_weights(shape, seed=2, gain_jitter=True, std=0.3)
    prompt = synth.make_prompt(shape.vocab, 70, 4)
    spec = O.SpecCfg(n_probes=3, topk=10, max_nodes=30, expand_width=1, n_anchor=0, prune_parent=False, static_widths=widths)
    run = pu.ParityRun(shape, w, spec, prompt, 40, TOL_FP32)
    out = run.run()
    assert out == O.greedy_generate(O.OracleModel(shape, w), prompt, 40, 256)
    assert run.h.state()["n_rows"] == 120
    g, _ = pu.gpu_generate(shape, run.wd, pu.GREEDY, prompt, 40)
    assert g == out
    run.close()


def test_bf16_block_complexity_120_parity_and_batch(pu):
    """The same block on the tensor-core path (MMA N = 128 per sequence, two sequences per weight stream): parity
    per step, bitwise equal to greedy decoding, and two sequences in one handle equal to each alone."""
    import paper_2603_17942_b200 as P
    shape = BF16_SMALL
    w = synth.make_weights(shape, seed=6, gain_jitter=True, std=0.05)
    spec = O.SpecCfg(n_probes=3, topk=10, max_nodes=30, expand_width=1, n_anchor=0)
    prompts = [synth.make_prompt(shape.vocab, n, 20 + i) for i, n in enumerate((210, 75, 140))]
    run = pu.ParityRun(shape, w, spec, prompts[0], 24, TOL_BF16)
    out = run.run()
    assert run.h.state()["n_rows"] == 120
    g, _ = pu.gpu_generate(shape, run.wd, pu.GREEDY, prompts[0], 24)
    assert g == out
    n_new, max_seq = 20, 400
    alone = []
    for pr in prompts:
        h1 = P.Handle(shape, pu.c_spec(spec), run.wd, max_seq_len=max_seq)
        alone.append(h1.generate(pr, n_new))
        h1.close()
    h = P.Handle(shape, pu.c_spec(spec), run.wd, max_seq_len=max_seq, max_batch=3)     # passes of 2 and 1
    outs = [[h.prefill(prompts[i], i)] for i in range(3)]
    while not all(len(o) >= n_new for o in outs):
        P.esp_step(h.h, h.tokens_out, h.n_out)
        for i in range(3):
            outs[i].extend(int(t) for t in h.tokens_out[i, :h.n_out[i]])
    assert h.stats().device_error == 0
    for i in range(3):
        assert outs[i][:n_new] == alone[i], f"sequence {i}"
    h.close()
    run.close()


def test_full_width_block_complexity_120_parity(pu):
    """Llama-3-8B-shape GEMMs, attention and LM head with 120-row blocks (two layers)."""
    shape = synth.LLAMA3_8B.replace(n_layers=2)
    w = synth.make_weights(shape, seed=0, device="cuda")
    wh = synth.weights_to_host(w)
    prompt = synth.make_prompt(shape.vocab, 200, 0)
    spec = O.SpecCfg(n_probes=3, topk=10, max_nodes=30, expand_width=1, n_anchor=0)
    run = pu.ParityRun(shape, wh, spec, prompt, 3, TOL_BF16, w_dev=w)
    out = run.run()
    g, _ = pu.gpu_generate(shape, w, pu.GREEDY, prompt, 3)
    assert g == out
    assert run.h.state()["n_rows"] == 120 and run.h.stats().device_error == 0
    run.close()


# ------------------------------------------------------------------ limits of the configuration space
@pytest.mark.parametrize("spec_kw,plen", [
    (dict(n_probes=3, topk=12, max_nodes=32, expand_width=1, n_anchor=0, prune_parent=False), 64),   # 128 rows: the largest block
    (dict(n_probes=8, topk=2, max_nodes=12, expand_width=1, n_anchor=1), 33),                        # the most probes
    (dict(n_probes=1, topk=31, max_nodes=32, expand_width=0, n_anchor=1), 5),                        # the longest Top-K' list (32 with the pruner's spare)
    (dict(n_probes=2, topk=3, max_nodes=8, expand_width=0, n_anchor=0), 1),                          # a one-token prompt
    (dict(n_probes=2, topk=3, max_nodes=8, expand_width=1, n_anchor=2), 2),
    (dict(n_probes=1, topk=1, max_nodes=2, expand_width=1, n_anchor=1), 129),                        # the smallest tree, a ragged third prefill block
])
def test_tiny_fp32_limits_parity(pu, spec_kw, plen):
    shape = synth.TINY
    w = synth.make_weights(shape, seed=8, gain_jitter=True, std=0.3)
    prompt = synth.make_prompt(shape.vocab, plen, 9)
    spec = O.SpecCfg(**spec_kw)
    run = pu.ParityRun(shape, w, spec, prompt, 24, TOL_FP32)
    out = run.run()
    assert out == O.greedy_generate(O.OracleModel(shape, w), prompt, 24, 256)
    if spec.n_probes == 3:
        assert run.h.state()["n_rows"] == 128
    assert run.h.stats().device_error == 0
    run.close()


def test_bf16_largest_block_parity(pu):
    """128 rows (32 nodes x (3 probes + 1)) on the tensor-core path."""
    shape = BF16_SMALL
    w = synth.make_weights(shape, seed=9, gain_jitter=True, std=0.05)
    prompt = synth.make_prompt(shape.vocab, 100, 3)
    spec = O.SpecCfg(n_probes=3, topk=12, max_nodes=32, expand_width=1, n_anchor=0, prune_parent=False)
    run = pu.ParityRun(shape, w, spec, prompt, 16, TOL_BF16)
    out = run.run()
    assert run.h.state()["n_rows"] == 128
    g, _ = pu.gpu_generate(shape, run.wd, pu.GREEDY, prompt, 16)
    assert g == out
    run.close()


# ------------------------------------------------------------------ sample matching (temperature > 0)
def test_sampling_noise_bitwise_equals_oracle():
    """The Gumbel noise of the CUDA path and of the oracle are the same fp32 numbers, bit for bit."""
    import paper_2603_17942_b200 as P
    n = 200_000
    out = torch.empty(n, device="cuda")
    for seed, pos in [(0, 0), (99, 17), ((5 << 32) | 12345, 4096), (2 ** 64 - 1, 2 ** 31 + 5)]:
        P.esp_debug_gumbel(seed, pos, n, out)
        torch.cuda.synchronize()
        ref = O.gumbel_noise(seed, pos, n)
        got = out.cpu().numpy()
        assert np.array_equal(got.view(np.uint32), ref.view(np.uint32)), (seed, pos)


@pytest.mark.parametrize("W,n_anchor,prune,temperature", [(0, 1, True, 1.0), (1, 0, False, 1.0), (0, 0, False, 0.6)])
def test_tiny_fp32_sample_matching_parity(pu, W, n_anchor, prune, temperature):
    """Section 4 "sample matching": every step against the oracle (noisy scores taken on the GPU's logits, bit for
    bit), the stream equal to the oracle's sampled stream and to plain sampling on the GPU with the same seed."""
    shape = synth.TINY
    w = synth.make_weights(shape, seed=0)
    prompt = synth.make_prompt(shape.vocab, 64, 0)
    B = 32 if n_anchor == 1 else 20
    spec = O.SpecCfg(n_probes=3, topk=4, max_nodes=B, expand_width=W, n_anchor=n_anchor, prune_parent=prune,
                     temperature=temperature, seed=(7 << 32) | 2024)
    run = pu.ParityRun(shape, w, spec, prompt, 64, TOL_FP32)
    out = run.run()
    model = O.OracleModel(shape, w)
    assert out == O.greedy_generate(model, prompt, 64, 256, spec=spec)     # plain sampling in the oracle
    dec = O.EspOracle(model, spec, 512)
    assert out == dec.generate(prompt, 64)
    import dataclasses
    plain = dataclasses.replace(pu.GREEDY, temperature=temperature, seed=spec.seed)
    g, _ = pu.gpu_generate(shape, run.wd, plain, prompt, 64)
    assert g == out                                                        # GPU ESP == GPU plain sampling
    assert out != O.greedy_generate(model, prompt, 64, 256)                # and it is not the greedy stream
    assert len(set(out)) > 16
    run.close()


def test_bf16_sample_matching_equals_plain_sampling(pu):
    """bf16 tensor-core path: parity per step, and the ESP stream at temperature 1 equals one-token-per-call
    sampling with the same seed (a row in a tree block draws what it would draw alone)."""
    import dataclasses
    shape = BF16_SMALL
    w = synth.make_weights(shape, seed=1, gain_jitter=True, std=0.05)
    prompt = synth.make_prompt(shape.vocab, 300, 2)
    spec = O.SpecCfg(n_probes=3, topk=5, max_nodes=16, expand_width=0, n_anchor=1, temperature=1.0, seed=31337)
    run = pu.ParityRun(shape, w, spec, prompt, 32, TOL_BF16)
    out = run.run()
    plain = dataclasses.replace(pu.GREEDY, temperature=1.0, seed=31337)
    g, _ = pu.gpu_generate(shape, run.wd, plain, prompt, 32)
    assert g == out
    g2, _ = pu.gpu_generate(shape, run.wd, dataclasses.replace(plain, seed=31338), prompt, 32)
    assert g2 != out
    assert run.h.stats().device_error == 0
    run.close()


# ------------------------------------------------------------------ errors are reported, not raised from the device
def test_host_side_errors(pu):
    import paper_2603_17942_b200 as P
    shape = synth.TINY
    w = pu.to_device(synth.make_weights(shape, seed=0))
    with pytest.raises(P.EspError) as e:
        P.Handle(shape, P.spec_cfg(n_probes=4, topk=4, max_nodes=70, n_anchor=0), w, 128)   # (k+1)*70 rows
    assert e.value.code == -1
    with pytest.raises(P.EspError):
        P.Handle(shape.replace(head_dim=48), P.spec_cfg(), w, 128)
    h = P.Handle(shape, P.spec_cfg(n_probes=2, topk=4, max_nodes=8), w, 96)
    with pytest.raises(P.EspError) as e:
        h.step()
    assert e.value.code == -7                                   # step before prefill
    with pytest.raises(P.EspError) as e:
        h.prefill(np.array([1, 2, shape.vocab], np.int32))
    assert e.value.code == -3
    with pytest.raises(P.EspError) as e:
        h.prefill(np.zeros(97, np.int32))
    assert e.value.code == -3                                   # longer than max_seq_len
    h.prefill(synth.make_prompt(shape.vocab, 80, 1))
    with pytest.raises(P.EspError) as e:
        h.set_tree(np.array([1, 2], np.int32), np.array([-1, 1], np.int32))   # parent not before child
    assert e.value.code == -8
    with pytest.raises(P.EspError) as e:
        for _ in range(40):
            h.step()
    assert e.value.code == -4                                   # sequence full
    assert h.stats().device_error == 0
    h.close()


# ------------------------------------------------------------------ asynchronous steps
def test_async_steps_then_reads_equal_synchronous_steps(pu):
    """esp_step_async only enqueues; every step keeps its own result record and esp_read hands them back oldest
    first.  A run of N enqueued steps followed by N reads must give, step by step, the tokens of N synchronous
    steps, the same final state and the same continuation -- also while the host, which between reads knows
    the cache length only as an upper bound (k + 1 per unread step), sizes the attention launches for more
    cache splits than there are (the bound crosses a split boundary here: 256-position splits, L near 250)."""
    import paper_2603_17942_b200 as P
    shape = BF16_SMALL
    w = synth.make_weights(shape, seed=7, gain_jitter=True, std=0.05)
    wd = pu.to_device(w)
    prompt = synth.make_prompt(shape.vocab, 236, 9)
    spec = O.SpecCfg(n_probes=3, topk=5, max_nodes=16, expand_width=0, n_anchor=1)
    hs = P.Handle(shape, pu.c_spec(spec), wd, max_seq_len=700)
    ha = P.Handle(shape, pu.c_spec(spec), wd, max_seq_len=700)
    assert hs.prefill(prompt) == ha.prefill(prompt)
    n = 40
    sync_tokens = [hs.step() for _ in range(n)]
    for _ in range(n):
        ha.step_async()
    async_tokens = [ha.read() for _ in range(n)]
    assert async_tokens == sync_tokens
    assert ha.read() == []                                   # nothing unread is left
    sa, ss = ha.state(), hs.state()
    assert sa["L"] == ss["L"] and sa["n_rows"] == ss["n_rows"]
    assert list(sa["row_token"][:sa["n_rows"]]) == list(ss["row_token"][:ss["n_rows"]])
    assert np.array_equal(sa["mask_vec"], ss["mask_vec"])
    assert ha.stats().emitted == hs.stats().emitted and ha.stats().steps == hs.stats().steps
    assert [ha.step() for _ in range(6)] == [hs.step() for _ in range(6)]
    assert sum(hs.stats().rows_hist) == hs.stats().steps        # every step is counted in the block-size histogram
    assert ha.stats().device_error == 0 and hs.stats().device_error == 0
    # one step more than there are result records is refused, and nothing is lost
    hb = P.Handle(shape, pu.c_spec(pu.GREEDY), wd, max_seq_len=236 + P.ESP_MAX_UNREAD_STEPS + 300)
    hb.prefill(prompt)
    for _ in range(P.ESP_MAX_UNREAD_STEPS):
        hb.step_async()
    with pytest.raises(P.EspError) as e:
        hb.step_async()
    assert e.value.code == -7                                # ESP_E_STATE
    first = hb.read()
    hb.step_async()                                          # one record is free again
    assert len(first) == 1
    ha.close(); hs.close(); hb.close()
