"""The kernel that runs all decoder layers of a step in one persistent launch against the path that launches one
kernel per operation (need a B200).  Both are driven through the C ABI; the second is selected with
esp_debug_set_layer_kernel(h, 1).  They run the same arithmetic in the same order, so everything is compared
bit for bit: the logits of every row of every step, the residual stream after the last layer, the emitted
tokens and the next row table.  (Parity with the CPU oracle is the job of test_gpu_parity.py, whose bf16
single-sequence cases run through the all-layers kernel by default.)"""
import numpy as np
import pytest
import torch

import synth
from oracle import esp as O

pytestmark = pytest.mark.gpu

SMALL = synth.TINY.replace(name="bf16-small", dtype="bf16", tied=False, n_layers=3, d_model=512, n_q_heads=4,
                           n_kv_heads=2, head_dim=128, d_ffn=688, vocab=5000)


def _pair(shape, wd, spec, max_seq_len):
    import paper_2603_17942_b200 as P
    from tests import parity_util as pu
    hs, bufs = [], []
    for mode in (0, 1):
        h = P.Handle(shape, pu.c_spec(spec), wd, max_seq_len=max_seq_len)
        P.esp_debug_set_layer_kernel(h.h, mode)
        logits = torch.zeros(P.ESP_MAX_ROWS, shape.vocab, device="cuda")
        hidden = torch.zeros(P.ESP_MAX_ROWS, shape.d_model, device="cuda")
        P.esp_debug_capture(h.h, logits, hidden)
        hs.append(h)
        bufs.append((logits, hidden))
    return hs, bufs


def _same_state(a, b):
    for key in ("n_nodes", "n_rows", "L"):
        assert a[key] == b[key], key
    n = a["n_rows"]
    for key in ("row_token", "row_parent", "row_depth"):
        assert np.array_equal(a[key][:n], b[key][:n]), key
    assert np.array_equal(a["mask_vec"], b["mask_vec"])


@pytest.mark.parametrize("qk_norm,plen,n_anchor", [(False, 333, 1), (True, 150, 0), (False, 40, 1)])
def test_all_layers_kernel_equals_kernel_per_operation_bitwise(qk_norm, plen, n_anchor):
    from tests import parity_util as pu
    shape = SMALL.replace(qk_norm=qk_norm, rms_eps=1e-6 if qk_norm else 1e-5)
    w = synth.make_weights(shape, seed=6, gain_jitter=True, std=0.05)
    wd = pu.to_device(w)
    prompt = synth.make_prompt(shape.vocab, plen, 5)
    spec = O.SpecCfg(n_probes=3, topk=5, max_nodes=16 if n_anchor else 12, expand_width=0, n_anchor=n_anchor)
    (ha, hb), ((la, xa), (lb, xb)) = _pair(shape, wd, spec, plen + 120)
    assert ha.prefill(prompt) == hb.prefill(prompt)
    truth, _ = pu.gpu_generate(shape, wd, pu.GREEDY, prompt, 80, max_seq_len=plen + 120)
    out = [truth[0]]
    rng = np.random.default_rng(2)
    for step in range(24):
        if step % 3 == 2:      # a forced draft along the true continuation: accepted rows, compaction, delta > 0
            depth = int(rng.integers(1, 4))
            toks = np.array([out[-1]] + [truth[len(out) + i] for i in range(depth)], np.int32)
            par = np.arange(-1, depth, dtype=np.int32)
            ha.set_tree(toks, par); hb.set_tree(toks, par)
        sa, sb = ha.state(), hb.state()
        _same_state(sa, sb)
        ta, tb = ha.step(), hb.step()
        assert ta == tb, f"step {step}"
        n = sa["n_rows"]
        assert torch.equal(xa[:n], xb[:n]), f"residual stream differs at step {step}"
        assert torch.equal(la[:n], lb[:n]), f"logits differ at step {step}"
        out.extend(ta)
    assert out == truth[:len(out)]
    assert ha.stats().device_error == 0 and hb.stats().device_error == 0
    assert ha.stats().kernels_per_step < 16 < hb.stats().kernels_per_step
    ha.close(); hb.close()


def test_all_layers_kernel_full_width_bitwise_and_greedy():
    """Llama-3-8B widths (every GEMM, the attention items and the LM head have their real shapes), 3 layers, a
    cache long enough for several splits: both paths agree bit for bit, ESP equals greedy decoding, and a greedy
    handle (1-row blocks through the same kernel) agrees between the paths as well."""
    import paper_2603_17942_b200 as P
    from tests import parity_util as pu
    shape = synth.LLAMA3_8B.replace(n_layers=3)
    w = synth.make_weights(shape, seed=1, device="cuda")
    prompt = synth.make_prompt(shape.vocab, 1100, 3)
    spec = O.SpecCfg(n_probes=4, topk=10, max_nodes=64, expand_width=0, n_anchor=1)
    (ha, hb), ((la, xa), (lb, xb)) = _pair(shape, w, spec, 1400)
    assert ha.prefill(prompt) == hb.prefill(prompt)
    out = []
    for step in range(6):
        n = ha.state()["n_rows"]
        ta, tb = ha.step(), hb.step()
        assert ta == tb
        assert torch.equal(xa[:n], xb[:n]) and torch.equal(la[:n], lb[:n]), f"step {step}"
        out.extend(ta)
    assert ha.stats().device_error == 0 and hb.stats().device_error == 0
    ha.close(); hb.close()
    greedy = []
    for mode in (0, 1):
        h = P.Handle(shape, pu.c_spec(pu.GREEDY), w, max_seq_len=1400)
        P.esp_debug_set_layer_kernel(h.h, mode)
        greedy.append(h.generate(prompt, 8))
        assert h.stats().device_error == 0
        h.close()
    assert greedy[0] == greedy[1]
    assert greedy[0][1:1 + len(out)][:7] == out[:7]
