#!/usr/bin/env python
"""Benchmark of the ESP decode-and-verify step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config llama3-8b|qwen3-8b]

One "step" is one esp_step: a decoder forward over [last accepted token, draft-tree nodes, mask probes]
against the KV cache, Top-K' at the probe rows, verification, KV compaction, mask update and the next tree.
Workload (default): the Llama-3-8B-shape bf16 decoder with seeded random-init weights, a 1024-token random
prompt, 4 mask probes, Top-10 per probe, trees of at most 64 nodes, batch 1.  Weights (15 GB) are streamed
from HBM every step, far more than the L2 holds, so no cache flush is needed between steps.

Prints ONE JSON line.  `value` is accepted tokens per second with everything resident on the device
(K esp_step_async calls between two CUDA events on the library's stream; their tokens are read afterwards from
the per-step result records and must equal greedy decoding with the same kernels); `e2e` is the same metric
over a whole request of the workload through the public calls -- the prompt from host memory into esp_prefill,
then synchronous esp_step calls, each returning its tokens in host memory, until the workload's number of new
tokens (256; 128 in the batch / long-context sweep) has been emitted -- and `e2e_step` that request's steps
alone.  With N > 1 every rank runs an independent replica of the whole job (the method has no cross-GPU
exchange); `value` sums the replicas' tokens over the slowest rank's time.

`--impl reference` times the CPU oracle (oracle/) on the host cores: whole full-depth steps of the same workload,
as many of the K requested as fit its time budget.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "esp_accepted_tokens_per_s"
UNIT = "tok/s"

# DRAM bytes (read + written) of one gate/up GEMM launch from the ncu capture summarised under profiles/
# (Llama-3-8B shape, 68 rows, one sequence); None for workloads without a capture of the current kernel.
GATEUP_DRAM_TRAFFIC = {"llama3-8b": 242.9e6}

GEN_TOKENS = 256          # new tokens per request of the two model workloads
GEN_TOKENS_SWEEP = 128    # ... of the batch / long-context sweep (--batch, --prompt-len)
WORKLOADS = {
    # name: (shape attr in synth, prompt length, probes, topk, max_nodes)
    "llama3-8b": ("LLAMA3_8B", 1024, 4, 10, 64),
    "qwen3-8b": ("QWEN3_8B", 2048, 4, 8, 48),
}


def measured_peaks():
    """HBM copy bandwidth (GB/s) measured on this machine, else the fallback figure; returns (value, source)."""
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.idx = gpu_index
        self.lines = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.idx), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0: float, t1: float):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons, power = [], [], set(), []
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for ts, line in self.lines:
            if ts < t0 or ts > t1 + 0.1:
                continue
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2])); power.append(float(f[3]))
            except ValueError:
                continue
            for n, v in zip(names, f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


def random_block(n_nodes, k, seed):
    """Row layout of a 64-node random tree with a k-probe chain under the root, for the oracle sample."""
    import synth
    parents = synth.random_tree_parents(n_nodes, 4, seed)
    M = n_nodes + k
    vis = np.zeros((M, M), np.uint8)
    pos = np.zeros(M, np.int32)
    for i in range(n_nodes):
        a = i
        while a >= 0:
            vis[i, a] = 1
            a = int(parents[a])
        pos[i] = vis[i].sum() - 1
    for j in range(k):
        r = n_nodes + j
        vis[r, 0] = 1
        vis[r, n_nodes:r + 1] = 1
        pos[r] = j + 1
    return vis, pos


class OracleSample:
    """The CPU oracle on a bounded sample of the workload: whole decode-and-verify forwards -- a full-width
    block (all tree and probe rows) through EVERY decoder layer and the LM head against a KV cache of the
    prompt's length (random N(0,1) entries: the forward does not care what the cache holds), then the argmax /
    Top-K' read-out the step needs.  One such forward is one step; accepted tokens per step are taken as 1
    (random-init models accept no drafts).  Nothing is extrapolated: the sample is bounded by running few steps."""

    def __init__(self, shape, plen, k, K, B, host_weights):
        from oracle import esp as O
        self.O = O
        self.shape = shape
        self.model = O.OracleModel(shape, host_weights)
        rng = np.random.default_rng(0)
        self.L = plen
        self.kc, self.vc = self.model.new_cache(plen + 8)
        self.kc[:, :plen] = rng.standard_normal(self.kc[:, :plen].shape, dtype=np.float32)
        self.vc[:, :plen] = rng.standard_normal(self.vc[:, :plen].shape, dtype=np.float32)
        self.vis, pos = random_block(B, k, 0)
        self.pos = plen + pos
        self.M, self.B, self.kp = B + k, B, K + 1
        self.x = (rng.standard_normal((self.M, shape.d_model), dtype=np.float32) * 0.02).astype(np.float32)
        self.cores = O.num_threads()

    def step_seconds(self):
        t0 = time.perf_counter()
        logits, _, _, _ = self.model.block_forward(self.kc, self.vc, self.L, self.x, self.pos, self.vis)
        for r in range(self.B):
            self.O.topk_desc(logits[r], 1)
        for r in range(self.B, self.M):
            self.O.topk_desc(logits[r], self.kp)
            self.O.log_sum_exp(logits[r])
        return time.perf_counter() - t0

    def describe(self):
        return (f"whole steps: a {self.M}-row block through all {self.shape.n_layers} layers + LM head + selection, "
                f"KV length {self.L}, 1 token per step")


def host_weights(shape, w_dev=None, seed=0):
    """Full-depth host copies of the model for the oracle (generated on the GPU when there is one: much faster)."""
    import synth
    import torch
    if w_dev is None:
        dev = "cuda" if torch.cuda.is_available() else "cpu"
        w_dev = synth.make_weights(shape, seed=seed, device=dev)
        if dev == "cpu":
            return w_dev
    return synth.weights_to_host(w_dev)


def workload_config(name, plen, nbatch, temperature, k, K, B, rows, replicas):
    """The `config` object of the JSON line: identical for both arms."""
    return {"workload": f"{name}-shape bf16 decoder, random-init seeded weights, b={nbatch}",
            "prompt_len": plen, "batch": nbatch, "temperature": temperature, "n_probes": k, "topk": K, "max_nodes": B,
            "rows_per_step": rows, "replicas": replicas, "l2": "inputs exceed L2 (weights are re-streamed every step)"}


REFERENCE_BUDGET_S = 150.0      # timed CPU work of the reference arm; the step count is cut to fit


def run_reference(args, shape, plen, k, K, B):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    smp = OracleSample(shape, plen, k, K, B, host_weights(shape))
    n_warm = min(max(args.warmup, 0), 2)
    for _ in range(n_warm):
        smp.step_seconds()
    times = []
    t_start = time.perf_counter()
    for i in range(max(1, args.steps)):
        times.append(smp.step_seconds())
        # stop when another step of this length would pass the budget
        if time.perf_counter() - t_start + times[-1] > REFERENCE_BUDGET_S:
            break
    sec = float(np.mean(times))
    val = 1.0 / sec
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": len(times),
            "warmup": n_warm, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": workload_config(args.config, plen, 1, 0.0, k, K, B, B + k, 1),
            "note": f"the CPU oracle as it stands (bf16 weights widened exactly, fp32 arithmetic); {len(times)} of the "
                    f"{args.steps} requested steps fit the {REFERENCE_BUDGET_S:.0f} s budget",
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": smp.cores, "kind": "oracle", "sample": smp.describe()},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def algorithmic_bytes(shape, L_mean, rows):
    """Bytes one step must move: every layer matrix and the LM head once, the KV cache of L positions once,
    the K/V rows of the block written once."""
    es = 2 if shape.dtype == "bf16" else 4
    w = shape.n_params_streamed() * es
    kv_per_pos = shape.n_layers * 2 * shape.n_kv_heads * shape.head_dim * es
    return w, kv_per_pos * L_mean + kv_per_pos * rows


REPLAY_SCHEDULES = {
    # the two operating points of the paper's main table for this model size: probabilities of 0, 1, 2, 3 accepted drafts
    "1.63": [0.55, 0.30, 0.12, 0.03],       # mean 0.63 accepted drafts per step
    "1.71": [0.50, 0.33, 0.13, 0.04],       # mean 0.71
}


def replay_leg(P, shape, w, prompt, stream, k, B, n_steps, probs, seed=0):
    """Throughput under a synthetic acceptance schedule.  Random-init models accept no drafts, so the draft trees
    of this leg are set from outside (esp_set_tree): each holds the true continuation (taken from a greedy run of
    the same kernels) down to a depth drawn per step with the probabilities `probs` (the paper's tau = 1.63 / 1.71
    operating points) inside a full tree of B nodes of wrong siblings.  The emitted stream must
    equal the greedy stream token for token.  Says nothing about model quality; it shows what a step costs when
    drafts are accepted, their KV rows compacted and the host is in the loop (set_tree + step, synchronous)."""
    n_tokens = int(2.2 * n_steps) + 16   # what n_steps emit at these schedules, with a wide margin (the loop stops at the end of the known stream)
    import torch
    plen = len(prompt)
    max_seq = plen + n_tokens + 64
    hg = P.Handle(shape, P.spec_cfg(), w, max_seq_len=max_seq, stream=stream)
    truth = hg.generate(prompt, n_tokens + 8)
    hg.close()
    mean_acc = sum(i * q for i, q in enumerate(probs))
    h = P.Handle(shape, P.spec_cfg(n_probes=k, topk=10, max_nodes=B, expand_width=0, n_anchor=1), w, max_seq_len=max_seq, stream=stream)
    out = [h.prefill(prompt)]
    rng = np.random.default_rng(seed)
    per_level = (B - 1) // k
    # the schedule holds each accepted length exactly in its proportion (so that tau comes out at the operating point
    # whatever the seed), in a random order
    counts = [int(round(q * n_steps)) for q in probs]
    counts[0] += n_steps - sum(counts)
    schedule = rng.permutation(np.repeat(np.arange(len(probs)), counts))
    steps = 0
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    L_start = h.state()["L"]
    while steps < n_steps and len(out) + k + 1 < len(truth):
        n = len(out)
        a = int(min(schedule[steps], k))
        toks, pars, main = [out[-1]], [-1], 0
        for d in range(1, k + 1):
            level = []
            if d <= a:
                level.append(truth[n + d - 1])
            wrong = rng.integers(0, shape.vocab - 1, size=per_level - len(level))
            wrong = [int(t) + (int(t) >= truth[n + d - 1]) for t in wrong]      # never the true token
            first = len(toks)
            for t in level + wrong:
                toks.append(t)
                pars.append(main)
            main = first                                                        # the true node while d <= a
        h.set_tree(np.array(toks, np.int32), np.array(pars, np.int32))
        new = h.step()
        steps += 1
        if len(new) != a + 1:
            raise SystemExit(f"replay: accepted {len(new) - 1} drafts, schedule said {a}")
        out.extend(new)
    torch.cuda.synchronize()
    sec = time.perf_counter() - t0
    if out != truth[:len(out)]:
        raise SystemExit("replay: ESP stream differs from the greedy stream")
    L_end = h.state()["L"]
    err = h.stats().device_error
    h.close()
    if err:
        raise SystemExit("replay: device error word set")
    return {"tau": (len(out) - 1) / steps, "tok_s": (len(out) - 1) / sec, "steps": steps, "ms_per_step": sec / steps * 1e3,
            "L_start": L_start, "L_end": L_end,
            "note": f"synthetic acceptance schedule (forced drafts, mean {mean_acc:.2f} accepted per step), not model quality; "
                    "includes the host round trip of esp_set_tree every step; stream checked equal to greedy"}


def aggregate_over_ranks(dist, times_ms, counts, device):
    """Replicas share nothing: the job's time is the slowest rank's (MAX), its work the sum over ranks (SUM)."""
    import torch
    t = torch.tensor(list(times_ms), device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    c = torch.tensor(list(counts), device=device, dtype=torch.float64)
    dist.all_reduce(c, op=dist.ReduceOp.SUM)
    return [float(x) for x in t], [int(x) for x in c]


def run_ours(args, shape, plen, k, K, B):
    import torch
    import synth
    import paper_2603_17942_b200 as P
    from paper_2603_17942_b200 import build as esp_build

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group(backend="nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        esp_build.build()
    if dist is not None:
        dist.barrier()
    P.load_library()

    steps, warm = args.steps, max(args.warmup, 3)
    if steps > P.ESP_MAX_UNREAD_STEPS:
        raise SystemExit(f"--steps: at most {P.ESP_MAX_UNREAD_STEPS} (the steps of the timed region are enqueued without a read in between)")
    w = synth.make_weights(shape, seed=rank, device="cuda")
    prompt = synth.make_prompt(shape.vocab, plen, rank)
    if args.per_node_probes:
        # the paper's block layout: k = 3 masks behind every one of 30 tree nodes, BC = (k+1) * 30 = 120 rows
        k, K, B = 3, 10, 30
        spec = P.spec_cfg(n_probes=k, topk=K, max_nodes=B, expand_width=1, n_anchor=0, temperature=args.temperature, seed=1)
    else:
        spec = P.spec_cfg(n_probes=k, topk=K, max_nodes=B, expand_width=0, n_anchor=1, temperature=args.temperature, seed=1)
    # room for one leg (at most k+1 tokens per step): the end-to-end leg starts again from the prompt
    gen = GEN_TOKENS_SWEEP if (args.batch > 1 or args.prompt_len > 0) else GEN_TOKENS
    max_seq = max(plen + (k + 1) * (steps + warm + 20 + 16) + 64, plen + gen + (k + 1) * 24 + 64)   # the request, then up to 20 profiled steps
    stream = torch.cuda.Stream()
    nbatch = max(1, args.batch)
    h = P.Handle(shape, spec, w, max_seq_len=max_seq, max_batch=nbatch, stream=stream)

    first_tokens = []

    def prefill_all():
        first_tokens[:] = [h.prefill(prompt)]
        for i in range(1, nbatch):
            first_tokens.append(h.prefill(synth.make_prompt(shape.vocab, plen, 1000 * rank + i), i))

    prefill_all()

    def emitted_steps():
        st = h.stats()
        return int(st.emitted), int(st.steps), st

    # ---- device-resident throughput: K asynchronous steps between two events on the library's stream
    esp_stream = [first_tokens[0]]
    for _ in range(warm):
        esp_stream.extend(h.step())
    e0, s0, _ = emitted_steps()
    L0 = h.state()["L"]
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local)
    sampler.start()
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    t0 = time.time()
    with torch.cuda.stream(stream):
        ev0.record()
        for _ in range(steps):
            h.step_async()
        ev1.record()
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    t1 = time.time()
    clocks = sampler.stop(t0, t1)
    timed_stream = []                  # sequence 0's tokens of the timed steps, from their result records
    for _ in range(steps):
        timed_stream.extend(h.read())
    ms = ev0.elapsed_time(ev1)
    e1, s1, st = emitted_steps()
    L1 = h.state()["L"]
    tokens = e1 - e0
    launches = int(st.kernels_per_step) * steps
    rows = h.state()["n_rows"]

    esp_stream.extend(timed_stream)

    # ---- end to end, a whole request through the public calls: the prompt goes from host memory into esp_prefill,
    # then synchronous esp_step calls, each returning its tokens in host memory, until every sequence has `gen` new tokens
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    te0 = time.perf_counter()
    prefill_all()
    torch.cuda.synchronize()
    prefill_ms = (time.perf_counter() - te0) * 1e3
    emitted_seq = np.ones(nbatch, np.int64)       # the prefill emits every sequence's first token
    e2e_steps = 0
    while int(emitted_seq.min()) < gen and e2e_steps < 2 * gen:
        h.step()
        emitted_seq += h.n_out[:nbatch].astype(np.int64)
        e2e_steps += 1
    e2e_tokens = int(emitted_seq.sum())
    torch.cuda.synchronize()
    te1 = time.perf_counter()
    e2e_ms = (te1 - te0) * 1e3
    e2e_step_ms = (e2e_ms - prefill_ms) / max(e2e_steps, 1)
    h2d_request = nbatch * plen * 4                              # the prompts (int32 ids)
    d2h_step = nbatch * (P.ESP_MAX_PROBES + 4) * 4 + 4           # every sequence's result record + the status word

    # ---- per-kernel-group device times (events between groups), for the roofline of the dominant kernel
    n_prof = min(steps, 20)
    kinds = {kname: 0.0 for kname in P.KINDS}
    for _ in range(n_prof):
        for kname, v in P.esp_step_profiled(h.h, h.tokens_out, h.n_out).items():
            kinds[kname] += v / n_prof
    if h.stats().device_error != 0:
        raise SystemExit("device error word set during the benchmark")

    # ---- greedy decoding with the same kernels (one row per step): its rate, and the stream the timed ESP steps
    # above must have reproduced token for token (lossless verification)
    greedy_tok_s, stream_checked = None, None
    if rank == 0 and not args.no_greedy and nbatch == 1:
        n_greedy = len(esp_stream) - 1            # decode steps that emit as many tokens as the ESP legs did
        hg = P.Handle(shape, P.spec_cfg(temperature=args.temperature, seed=1), w, max_seq_len=plen + n_greedy + 64, stream=stream)
        greedy_stream = [hg.prefill(prompt)]
        for _ in range(warm):
            greedy_stream.extend(hg.step())
        n_timed = min(n_greedy - warm, P.ESP_MAX_UNREAD_STEPS)
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(stream):
            g0.record()
            for _ in range(n_timed):
                hg.step_async()
            g1.record()
        torch.cuda.synchronize()
        for _ in range(n_timed):
            greedy_stream.extend(hg.read())
        greedy_tok_s = n_timed / (g0.elapsed_time(g1) * 1e-3)
        while len(greedy_stream) < len(esp_stream):
            greedy_stream.extend(hg.step())
        hg.close()
        if greedy_stream[:len(esp_stream)] != esp_stream:
            bad = next(i for i, (x, y) in enumerate(zip(esp_stream, greedy_stream)) if x != y)
            raise SystemExit(f"the timed ESP stream differs from greedy decoding at token {bad}")
        stream_checked = len(esp_stream)

    replay = {}
    if rank == 0 and not args.no_greedy and nbatch == 1 and not args.per_node_probes and args.temperature == 0.0:
        for name, probs in REPLAY_SCHEDULES.items():
            replay[name] = replay_leg(P, shape, w, prompt, stream, k, B, 200, probs, seed=int(float(name) * 100))

    # ---- aggregate over ranks: slowest rank's time, all ranks' tokens
    if dist is not None:
        (ms, e2e_ms), (tokens, e2e_tokens, launches) = aggregate_over_ranks(dist, [ms, e2e_ms], [tokens, e2e_tokens, launches], "cuda")

    if rank == 0:
        peak, peak_src = measured_peaks()
        es = 2
        F, d = shape.d_ffn, shape.d_model
        gu_bytes = 2 * F * d * es + rows * d * es + rows * F * es   # gate+up weights, activations in, SiLU*up out
        gu_ms = kinds["gateup_gemm"] / shape.n_layers
        gu_ach = gu_bytes / (gu_ms * 1e-3) / 1e9 if gu_ms > 0 else None
        wbytes, kvbytes = algorithmic_bytes(shape, 0.5 * (L0 + L1), rows)
        kvbytes *= nbatch                    # weights once per step, every sequence's cache
        step_ms = ms / steps
        step_ach = (wbytes + kvbytes) / (step_ms * 1e-3) / 1e9
        line = {
            "metric": METRIC, "value": tokens / (ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warm,
            "ms_per_step": step_ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic",
            "config": workload_config(args.config, plen, nbatch, args.temperature, k, K, B, rows, world),
            "mean_accepted_len": tokens / (steps * world * nbatch),
            "kv_len": {"timed_start": L0, "timed_end": L1},
            "clocks": clocks,
            "e2e": {"value": e2e_tokens / (e2e_ms * 1e-3), "unit": UNIT,
                    "h2d_bytes_per_step": h2d_request / max(e2e_steps, 1), "d2h_bytes_per_step": d2h_step,
                    "h2d_bytes_per_request": h2d_request, "request_ms": e2e_ms, "request_tokens": e2e_tokens,
                    "request_steps": e2e_steps,
                    "note": "whole requests of the workload through the public calls, every rank: the prompt from host "
                            "memory into esp_prefill, then synchronous esp_step calls that return their tokens in host "
                            f"memory until {gen} new tokens per sequence; the prefill time is inside the timed region "
                            "and its bytes are spread over the steps"},
            "e2e_step": {"value": (e2e_tokens - nbatch * world) / ((e2e_ms - prefill_ms) * 1e-3), "unit": UNIT, "ms_per_step": e2e_step_ms,
                         "note": "the synchronous esp_step calls of that request alone (a step's inputs are the device "
                                 "state the step before left; its tokens land in host memory)"},
            "gpu_launches": launches,
            "stream_equals_greedy_tokens": stream_checked,
            "prefill": {"ms": prefill_ms, "prompt_tokens": plen * nbatch, "tokens_per_s": plen * nbatch / (prefill_ms * 1e-3),
                        "note": "esp_prefill of every sequence from host memory, blocks of %d prompt rows" % P.ESP_PREFILL_CHUNK},
            "roofline": {"bound": "hbm", "kernel": "k_gemm_tc<EPI_PARTIAL>, gate/up projection (235 MB of weights per launch)",
                         "achieved": gu_ach, "peak": peak, "unit": "GB/s", "frac": gu_ach / peak if gu_ach else None,
                         "traffic": GATEUP_DRAM_TRAFFIC.get(args.config) if nbatch == 1 and not args.per_node_probes else None,
                         "peak_source": peak_src, "bytes_per_launch": gu_bytes,
                         "us_per_launch": gu_ms * 1e3,
                         "measured_in": f"{n_prof} profiled steps after the timed region (an event after every kernel)"},
            "step_roofline": {"bound": "hbm", "bytes_per_step": wbytes + kvbytes, "weight_bytes": wbytes,
                              "kv_bytes": kvbytes, "achieved": step_ach, "peak": peak, "unit": "GB/s",
                              "frac": step_ach / peak, "frac_of_8TBs_nominal": step_ach / 8000.0,
                              "peak_source": peak_src},
            "kernel_group_ms_per_step": kinds,
            "greedy_tok_s": greedy_tok_s,
            "replay": replay or None,
        }
        if not args.no_cpu and world == 1:
            smp = OracleSample(shape, plen, k, K, B, host_weights(shape, w))
            smp.step_seconds()                               # warm: page the weights in, start the thread pool
            secs = sorted(smp.step_seconds() for _ in range(3))
            sec = secs[1]
            line["cpu_baseline"] = {"value": 1.0 / sec, "unit": UNIT, "cores": smp.cores, "kind": "oracle",
                                    "sample": smp.describe() + "; median of 3 after one warm-up", "ms_per_step": sec * 1e3}
        else:
            line["cpu_baseline"] = None
        print(json.dumps(line), flush=True)
    h.close()
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def run_attention_op(args):
    """Tree-attention operator alone (32 query / 8 KV heads of 128, KV length 4096, a 64-node random tree of
    depth <= 5 plus 4 mask-probe rows, N(0,1) bf16 cache), batch 1 and batch 16: device time per call, achieved
    KV bytes/s and FLOP/s.  Between timed calls a 512 MB buffer is rewritten so the cache is read from HBM."""
    import torch
    import synth
    import paper_2603_17942_b200 as P
    from paper_2603_17942_b200 import build as esp_build
    esp_build.build()
    torch.cuda.set_device(0)
    R, Hq, Hkv, h, L, n_nodes, n_probes = P.ESP_MAX_ROWS, 32, 8, 128, args.prompt_len or 4096, 64, 4
    M = n_nodes + n_probes
    peak, peak_src = measured_peaks()
    flush = torch.zeros(512 << 20, dtype=torch.uint8, device="cuda")
    results = {}
    for batch in (1, 16):
        cap = L + R
        q, kc, vc, kb, vb = synth.random_qkv((batch, R, Hq, h), (batch, Hkv, cap, h), (batch, Hkv, M, h), seed=batch, device="cuda")
        kc[:, :, L:L + M] = kb
        vc[:, :, L:L + M] = vb
        anc = np.zeros((batch, R, 2), np.uint64)
        depth = np.zeros((batch, R), np.int32)
        for s in range(batch):
            vis, pos = random_block(n_nodes, n_probes, 10 * batch + s)
            depth[s, :M] = pos
            for r in range(M):
                for i in np.nonzero(vis[r])[0]:
                    anc[s, r, i // 64] |= np.uint64(1) << np.uint64(i % 64)
            for r in range(M, R):
                anc[s, r, r // 64] = np.uint64(1) << np.uint64(r % 64)
        anc_d, depth_d = torch.from_numpy(anc.view(np.int64)).cuda(), torch.from_numpy(depth).cuda()
        out = torch.zeros_like(q)
        nb = P.esp_tree_attention_scratch_bytes(batch, Hq, h, cap)
        scratch = torch.zeros(nb, dtype=torch.uint8, device="cuda")
        times = []
        for it in range(args.warmup + args.steps):
            flush.add_(1)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            P.esp_tree_attention(1, batch, M, L, cap, Hq, Hkv, h, 16, q, kc, vc, anc_d, depth_d, out, scratch, nb,
                                 torch.cuda.current_stream().cuda_stream)
            e1.record()
            torch.cuda.synchronize()
            if it >= args.warmup:
                times.append(e0.elapsed_time(e1) * 1e3)
        us = float(np.median(times))
        kv_bytes = batch * Hkv * (L + M) * h * 2 * 2
        flops = 4.0 * batch * M * Hq * (L + 6) * h          # QK^T and PV over the cache and a row's own path
        results[f"b{batch}"] = {"us": us, "kv_bytes": kv_bytes, "achieved_GBs": kv_bytes / us / 1e3,
                                "frac_of_hbm_peak": kv_bytes / us / 1e3 / peak, "achieved_TFLOPs": flops / us / 1e6}
    line = {"metric": "tree_attention_us", "value": results["b16"]["us"], "unit": "us", "n_gpus": 1, "steps": args.steps,
            "warmup": args.warmup, "higher_is_better": False, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": f"tree-attention operator, 32/8 heads x 128, KV {L}, 64-node tree + 4 probes, batch 1 and 16",
                       "l2": "512 MB buffer rewritten between calls"},
            "results": results, "peak_GBs": peak, "peak_source": peak_src, "gpu_launches": 2 * args.steps}
    print(json.dumps(line), flush=True)


def run_layer_kernel_trace(args, shape, plen, k, K, B):
    """The all-layers persistent kernel (esp_debug_set_layer_kernel mode 0) against the default path of one kernel
    per operation, on the same workload: device ms per step of both, and where the persistent kernel's time goes
    per layer -- for each of its ten phases the time its first CTA spends in the phase and then in the grid
    barrier behind it (averages over the layers after the first and over 5 traced steps)."""
    import torch
    import synth
    import paper_2603_17942_b200 as P
    from paper_2603_17942_b200 import build as esp_build
    esp_build.build()
    torch.cuda.set_device(0)
    w = synth.make_weights(shape, seed=0, device="cuda")
    prompt = synth.make_prompt(shape.vocab, plen, 0)
    spec = P.spec_cfg(n_probes=k, topk=K, max_nodes=B, expand_width=0, n_anchor=1)
    stream = torch.cuda.Stream()
    steps = min(args.steps, P.ESP_MAX_UNREAD_STEPS)
    h = P.Handle(shape, spec, w, max_seq_len=plen + (k + 1) * (2 * steps + 40) + 64, stream=stream)
    h.prefill(prompt)
    out = {}
    for mode, name in ((1, "kernel_per_operation"), (0, "all_layers_kernel")):
        P.esp_debug_set_layer_kernel(h.h, mode)
        for _ in range(max(args.warmup, 3)):
            h.step()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(stream):
            e0.record()
            for _ in range(steps):
                h.step_async()
            e1.record()
        torch.cuda.synchronize()
        for _ in range(steps):
            h.read()
        out[name + "_ms_per_step"] = e0.elapsed_time(e1) / steps
    names = ["attention norm", "QKV GEMM", "q/k/v finish", "attention over the cache", "attention tail + merge", "O GEMM",
             "FFN norm", "gate/up GEMM", "SiLU*up", "down GEMM"]
    acc = np.zeros((10, 2))
    n_tr = 5
    for _ in range(n_tr):
        P.esp_step_profiled(h.h, h.tokens_out, h.n_out)
        tl = P.esp_debug_layer_timeline(h.h, shape.n_layers).astype(np.int64).reshape(-1, 8)
        body = np.concatenate([[0], tl[1:, 0] - tl[:-1, 1]]).reshape(-1, 10)
        wait = (tl[:, 1] - tl[:, 0]).reshape(-1, 10)
        acc[:, 0] += body[1:].mean(axis=0) / n_tr
        acc[:, 1] += wait[1:].mean(axis=0) / n_tr
    out["phase_us"] = {nm: {"phase": round(float(a[0]) / 1e3, 2), "barrier": round(float(a[1]) / 1e3, 2)} for nm, a in zip(names, acc)}
    out["layer_us"] = round(float(acc.sum()) / 1e3, 2)
    err = h.stats().device_error
    h.close()
    if err:
        raise SystemExit("device error word set")
    print(json.dumps({"metric": "all_layers_kernel_trace", "config": workload_config(args.config, plen, 1, 0.0, k, K, B, B + k, 1),
                      "steps": steps, **out}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="llama3-8b", choices=sorted(WORKLOADS) + ["attention-op"])
    ap.add_argument("--prompt-len", type=int, default=0, help="override the workload's prompt / KV length")
    ap.add_argument("--batch", type=int, default=1, help="independent sequences in one handle (long-context / batch sweep)")
    ap.add_argument("--temperature", type=float, default=0.0,
                    help="0 = greedy matching (default); > 0 = sample matching at that temperature")
    ap.add_argument("--per-node-probes", action="store_true",
                    help="k = 3 probes behind each of 30 tree nodes (block complexity 120) instead of the default block")
    ap.add_argument("--layers", type=int, default=0, help="cut the layer count (smaller captures under a profiler)")
    ap.add_argument("--trace-layer-kernel", action="store_true",
                    help="time the all-layers persistent kernel against the default path and print its per-phase trace")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle leg")
    ap.add_argument("--no-greedy", action="store_true", help="skip the greedy-decoding leg")
    args = ap.parse_args()
    import synth
    if args.config == "attention-op":
        if int(os.environ.get("RANK", "0")) == 0:
            run_attention_op(args)
        return
    name, plen, k, K, B = WORKLOADS[args.config]
    if args.prompt_len > 0:
        plen = args.prompt_len
    shape = getattr(synth, name)
    if args.layers > 0:
        shape = shape.replace(n_layers=args.layers)
    if args.trace_layer_kernel:
        if int(os.environ.get("RANK", "0")) == 0:
            run_layer_kernel_trace(args, shape, plen, k, K, B)
    elif args.impl == "reference":
        run_reference(args, shape, plen, k, K, B)
    else:
        run_ours(args, shape, plen, k, K, B)


if __name__ == "__main__":
    main()
