"""Shared harness of the GPU parity tests: drives the CUDA library through its C ABI and checks
every step against the CPU oracle, teacher-forced on the GPU's own token stream.

Per step it checks
  * block layout: the GPU's row table (tokens, parents, position offsets, row count) equals the oracle's
    layout of the same tree;
  * logits of every row (tree nodes and mask probes) against the oracle's block forward over the same
    rows and the oracle's own KV cache and mask vector: max |diff| <= tol * (logit range);
  * selection, bit-exact given the GPU's logits: argmax / Top-K' lists equal a full sort of the dumped
    logits, log-sum-exp agrees to fp32 rounding;
  * sample matching (temperature > 0): a node's token is the arg-max of the oracle's noisy scores of the
    GPU's logits at the node's position, bit for bit;
  * verification: the oracle's walk over the GPU's per-node argmax gives the GPU's emitted tokens;
  * next tree: the oracle's Algorithm 1 fed with the GPU's Top-K' lists and lse gives the GPU's next
    row table exactly;
  * where the GPU's argmax differs from the oracle's on the same inputs, the oracle's top-1/top-2 gap
    must be below the logit tolerance (a near-tie), otherwise it is a bug.
"""
from __future__ import annotations

import numpy as np
import torch

import paper_2603_17942_b200 as P
from oracle import esp as O


def to_device(w, device="cuda"):
    wd = {k: ([t.to(device) for t in v] if isinstance(v, list) else v.to(device)) for k, v in w.items()}
    if w["lm_head"] is w["embed"]:
        wd["lm_head"] = wd["embed"]
    return wd


def c_spec(o: O.SpecCfg):
    return P.spec_cfg(n_probes=o.n_probes, topk=o.topk, max_nodes=o.max_nodes, expand_width=o.expand_width,
                      n_anchor=o.n_anchor, prune_parent=o.prune_parent, prune_root=o.prune_root,
                      ema_per_token=o.ema_per_token, lam=o.lam, static_widths=o.static_widths,
                      mask_init={"mean": 0, "last_k": 1, "given": 2}[o.mask_init],
                      temperature=o.temperature, seed=o.seed)


class ParityRun:
    def __init__(self, shape, w_host, spec: O.SpecCfg, prompt, max_new, tol, gemm_impl=None, w_dev=None, given_mask=None):
        self.shape, self.spec, self.tol = shape, spec, tol
        self.model = O.OracleModel(shape, w_host)
        self.wd = w_dev if w_dev is not None else to_device(w_host)
        self.prompt = np.asarray(prompt, np.int32)
        self.max_new = max_new
        self.h = P.Handle(shape, c_spec(spec), self.wd, max_seq_len=len(prompt) + max_new + 16)
        if gemm_impl is not None:
            P.esp_debug_set_gemm(self.h.h, gemm_impl)
        self.logits = torch.zeros(P.ESP_MAX_ROWS, shape.vocab, device="cuda")
        P.esp_debug_capture(self.h.h, self.logits, None)
        self.kc, self.vc = self.model.new_cache(len(prompt) + max_new + 16 + P.ESP_MAX_ROWS)
        self.L = 0
        self.m = None
        self.given_mask = given_mask
        if given_mask is not None:
            self.h.set_mask(given_mask)
        self.near_ties = 0
        self.worst = 0.0
        self.emitted = []
        self.accepts = []

    # ---- helpers
    def _cmp_logits(self, got, ref, what):
        rng = float(ref.max() - ref.min())
        err = float(np.abs(got - ref).max()) / rng
        self.worst = max(self.worst, err)
        assert err <= self.tol, f"{what}: logits off by {err:.3e} of the logit range (tol {self.tol})"
        return rng

    def _scores(self, row_logits, pos):
        """What a node row's arg-max is taken over: the logits, or the noisy scores for the token at position pos."""
        if self.spec.temperature > 0:
            return O.sample_scores(row_logits, pos, self.spec.temperature, self.spec.seed)
        return row_logits

    def _check_selection(self, gl, st, rows_nodes, rows_probes, node_pos):
        kp = self.spec.k_prime
        for r in rows_nodes:
            ids, vals = O.topk_desc(self._scores(gl[r], node_pos[r] + 1), 1)
            assert st["topk_ids"][r, 0] == ids[0] and st["topk_vals"][r, 0] == vals[0], f"argmax row {r}"
        for r in rows_probes:
            ids, vals = O.topk_desc(gl[r], kp)
            assert list(st["topk_ids"][r, :kp]) == list(ids), f"Top-K' ids row {r}"
            assert np.array_equal(st["topk_vals"][r, :kp], vals), f"Top-K' values row {r}"
            assert abs(float(st["lse"][r]) - float(O.log_sum_exp(gl[r]))) <= 2e-5 * max(1.0, abs(float(st["lse"][r])))

    def _near_tie(self, ref_row, gpu_tok, rng, what, pos):
        ref_row = self._scores(ref_row, pos + 1)
        o_ids, o_vals = O.topk_desc(ref_row, 2)
        if int(o_ids[0]) != int(gpu_tok):
            gap = float(ref_row[o_ids[0]] - ref_row[gpu_tok])
            scale = 1.0 / self.spec.temperature if self.spec.temperature > 0 else 1.0
            assert gap <= 2 * self.tol * rng * max(1.0, scale), f"{what}: GPU picked {gpu_tok}, oracle {o_ids[0]}, gap {gap} is not a near-tie"
            self.near_ties += 1

    def _tree_from_state(self, st):
        N = st["n_nodes"]
        return O.Tree(st["row_token"][:N].copy(), st["row_parent"][:N].copy(), st["row_depth"][:N].copy(), np.zeros(N, np.float32))

    def _check_next_tree(self, st_after, root, ids, vals, lses):
        tree = O.next_tree(root, ids, vals, lses, self.spec) if self.spec.n_probes else O.root_only(root)
        N = st_after["n_nodes"]
        assert N == tree.n, f"next tree size {N} vs oracle {tree.n}"
        assert list(st_after["row_token"][:N]) == list(tree.tokens)
        assert list(st_after["row_parent"][:N]) == list(tree.parents)
        assert list(st_after["row_depth"][:N]) == list(tree.depths)
        blk = O.layout_block(tree, self.spec)
        assert st_after["n_rows"] == blk.m
        assert list(st_after["row_depth"][:blk.m]) == list(blk.row_pos_off)
        assert all(st_after["row_token"][N:blk.m] == -1)

    # ---- prefill
    def prefill(self):
        sp, t, k = self.spec, len(self.prompt), self.spec.n_probes
        first = self.h.prefill(self.prompt)
        st = self.h.state()
        gl = self.logits.cpu().numpy()
        E = np.stack([self.model.embed(int(x)) for x in self.prompt])
        if sp.mask_init == "last_k" and k:
            self.m = O.mask_init_last_k(E, k)
        elif sp.mask_init == "given":
            self.m = np.array(self.given_mask, np.float32).reshape(max(k, 1), -1)
        else:
            self.m = np.tile(O.mask_init_mean(E), (max(k, 1), 1))
        M = t + k
        x = np.concatenate([E, self.m[:k]], 0) if k else E
        want = np.zeros(M, np.uint8)
        want[t - 1:] = 1
        ref, kb, vb, _ = self.model.block_forward(self.kc, self.vc, 0, x, np.arange(M), np.tril(np.ones((M, M), np.uint8)), want)
        self.kc[:, :t], self.vc[:, :t] = kb[:, :t], vb[:, :t]
        self.L = t
        # the last prefill chunk holds the final (t-1) % chunk + 1 prompt rows followed by the k mask rows
        r0 = (t - 1) % P.ESP_PREFILL_CHUNK
        rng = self._cmp_logits(gl[r0:r0 + 1 + k], ref[t - 1:], "prefill")
        self._check_selection(gl, st, [r0], range(r0 + 1, r0 + 1 + k), {r0: t - 1})
        assert first == st["topk_ids"][r0, 0]
        self._near_tie(ref[t - 1], first, rng, "prefill", t - 1)
        self.emitted.append(first)
        self.m = O.mask_update(self.m, self.model.embed(first), sp.lam)
        assert st["L"] == t
        np.testing.assert_allclose(st["mask_vec"], self.m, rtol=0, atol=1e-6 * max(1.0, float(np.abs(self.m).max())))
        kp = sp.k_prime
        ids = [st["topk_ids"][r0 + j, :kp] for j in range(1, k + 1)]
        vals = [st["topk_vals"][r0 + j, :kp] for j in range(1, k + 1)]
        lses = [st["lse"][r0 + j] for j in range(1, k + 1)]
        self._check_next_tree(st, first, ids, vals, lses)
        return st

    # ---- one decode-and-verify step
    def step(self, st_before, forced=None):
        sp, k = self.spec, self.spec.n_probes
        if forced is not None:
            self.h.set_tree(forced.tokens, forced.parents)
            st_before = self.h.state()
        tree = self._tree_from_state(st_before)
        blk = O.layout_block(tree, sp)
        assert st_before["n_rows"] == blk.m and st_before["L"] == self.L
        assert list(st_before["row_depth"][:blk.m]) == list(blk.row_pos_off)
        toks = self.h.step()
        st = self.h.state()
        gl = self.logits.cpu().numpy()
        probe_of_row = {row: j for (_, j), row in blk.probe_row.items()}
        x = np.stack([self.model.embed(int(t)) if t >= 0 else self.m[probe_of_row[r] - 1] for r, t in enumerate(blk.row_token)])
        ref, kb, vb, _ = self.model.block_forward(self.kc, self.vc, self.L, x, self.L + blk.row_pos_off, blk.vis)
        rng = self._cmp_logits(gl[:blk.m], ref, f"step {len(self.accepts)}")
        node_pos = {r: self.L + int(blk.row_pos_off[r]) for r in range(blk.n_nodes)}
        self._check_selection(gl, st, range(blk.n_nodes), range(blk.n_nodes, blk.m), node_pos)
        gpu_next = [int(st["topk_ids"][r, 0]) for r in range(blk.n_nodes)]
        path, out = O.verify_walk(tree, gpu_next)
        assert toks == out, f"emitted {toks} vs verify walk {out}"
        for p in path:
            self._near_tie(ref[p], gpu_next[p], rng, f"step {len(self.accepts)} node {p}", node_pos[p])
        a = len(path) - 1
        for j, p in enumerate(path):
            self.kc[:, self.L + j], self.vc[:, self.L + j] = kb[:, p], vb[:, p]
        self.L += a + 1
        assert st["L"] == self.L
        for y in out:
            self.m = O.mask_update(self.m, self.model.embed(y), sp.lam) if sp.ema_per_token else self.m
        if not sp.ema_per_token:
            self.m = O.mask_update(self.m, self.model.embed(out[-1]), sp.lam)
        np.testing.assert_allclose(st["mask_vec"], self.m, rtol=0, atol=2e-6 * max(1.0, float(np.abs(self.m).max())))
        ids = vals = lses = ()
        if k:
            _, _, rows = O.draft_source(tree, blk, path, sp)   # pinned by the position-predictor test of the oracle
            kp = sp.k_prime
            ids = [st["topk_ids"][r, :kp] for r in rows]
            vals = [st["topk_vals"][r, :kp] for r in rows]
            lses = [st["lse"][r] for r in rows]
        self._check_next_tree(st, out[-1], ids, vals, lses)
        self.emitted.extend(out)
        self.accepts.append(a)
        return st

    def run(self):
        st = self.prefill()
        while len(self.emitted) < self.max_new:
            st = self.step(st)
        return self.emitted[:self.max_new]

    def close(self):
        self.h.close()


def gpu_generate(shape, w_dev, spec: O.SpecCfg, prompt, max_new, gemm_impl=None, max_seq_len=None):
    h = P.Handle(shape, c_spec(spec), w_dev, max_seq_len=max_seq_len or (len(prompt) + max_new + 16))
    if gemm_impl is not None:
        P.esp_debug_set_gemm(h.h, gemm_impl)
    out = h.generate(np.asarray(prompt, np.int32), max_new)
    stats = h.stats()
    h.close()
    return out, stats


GREEDY = O.SpecCfg(n_probes=0, topk=1, max_nodes=1)
