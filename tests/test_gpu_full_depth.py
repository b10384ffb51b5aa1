"""Configs 3 and 4 at their real depth and prompt length (need a B200 and a host with ~40 GB of free memory).

The other GPU parity tests cut the 8B shapes to two layers so that the CPU oracle finishes in seconds.  Here the
Llama-3-8B shape runs with its 32 layers and a 1024-token prompt, the Qwen3-8B shape (per-head QK-norm) with its
36 layers and a 2048-token prompt: the prefill and four decode-and-verify steps go through the parity harness
(tests/parity_util.py: logits of every row within 2e-2 of the logit range of the teacher-forced oracle, selection
and trees bit-exact given the GPU's logits, near-tie certificate), and the GPU's ESP stream must equal the GPU's
greedy stream over the config's full 256 generated tokens.  The oracle needs about a minute (Llama) to two
(Qwen3) for the prefill on 16 host cores and a few seconds per step."""
import pytest

import synth
from oracle import esp as O

pytestmark = pytest.mark.gpu

TOL_BF16 = 2e-2   # of the logit range


@pytest.mark.parametrize("base,plen,topk,B", [(synth.LLAMA3_8B, 1024, 10, 64), (synth.QWEN3_8B, 2048, 8, 48)])
def test_full_depth_parity_and_lossless_256_tokens(base, plen, topk, B):
    from tests import parity_util as pu
    shape = base
    w = synth.make_weights(shape, seed=0, device="cuda")
    prompt = synth.make_prompt(shape.vocab, plen, 0)
    spec = O.SpecCfg(n_probes=4, topk=topk, max_nodes=B, expand_width=0, n_anchor=1)
    # ---- lossless over the whole generation length: GPU ESP == GPU greedy, 256 tokens
    esp_out, st = pu.gpu_generate(shape, w, spec, prompt, 256)
    assert st.device_error == 0
    greedy_out, st = pu.gpu_generate(shape, w, pu.GREEDY, prompt, 256)
    assert st.device_error == 0
    assert esp_out == greedy_out
    assert len(set(esp_out)) > 32                              # not a degenerate stream
    # ---- prefill + 4 steps against the oracle at full depth
    wh = synth.weights_to_host(w)
    run = pu.ParityRun(shape, wh, spec, prompt, 5, TOL_BF16, w_dev=w)
    out = run.run()
    assert out == esp_out[:5]
    assert run.h.stats().device_error == 0
    print(f"{shape.name}: worst logit error {run.worst:.3e} of the range after {shape.n_layers} layers, "
          f"{run.near_ties} near-ties")
    assert run.worst <= TOL_BF16
    run.close()
