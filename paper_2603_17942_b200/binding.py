"""ctypes binding of ``libesp_b200.so`` -- argument marshalling only.

Function names mirror ``include/esp.h``.  PyTorch appears here only as the
owner of device memory and streams: tensors are turned into raw pointers and
the library does all the work.  There is no CPU fallback; if the library is
missing, loading raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Dict, List, Optional, Sequence

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libesp_b200.so")

ESP_MAX_ROWS = 128
ESP_MAX_PROBES = 8
ESP_MAX_KPRIME = 32
ESP_PREFILL_CHUNK = 120
ESP_MAX_UNREAD_STEPS = 1024

ERRORS = {0: "ESP_OK", -1: "ESP_E_BADCFG", -2: "ESP_E_WORKSPACE", -3: "ESP_E_PROMPT", -4: "ESP_E_FULL",
          -5: "ESP_E_DEVICE", -6: "ESP_E_CUDA", -7: "ESP_E_STATE", -8: "ESP_E_ARG"}

EXPORTS = ["esp_workspace_bytes", "esp_init", "esp_prefill", "esp_step", "esp_step_async", "esp_read", "esp_set_mask", "esp_set_tree",
           "esp_debug_state", "esp_debug_capture", "esp_debug_set_gemm", "esp_debug_set_layer_kernel", "esp_debug_layer_timeline", "esp_step_profiled", "esp_get_stats",
           "esp_debug_wait_selftest", "esp_debug_gumbel", "esp_free",
           "esp_tree_attention_scratch_bytes", "esp_tree_attention", "esp_tree_attention_status", "esp_tree_attention_static", "esp_gemm_scratch_bytes",
           "esp_gemm_bf16"]

__all__ = ["EspError", "esp_model_cfg", "esp_spec_cfg", "esp_weights", "esp_stats", "load_library", "model_cfg",
           "spec_cfg", "Handle", "ESP_MAX_ROWS", "ESP_MAX_PROBES", "ESP_MAX_KPRIME", "ESP_PREFILL_CHUNK", "ESP_MAX_UNREAD_STEPS", "ESP_STATIC_SCRATCH_BYTES", "EXPORTS", "LIB_PATH", "KINDS"] + EXPORTS


class EspError(RuntimeError):
    def __init__(self, code: int, where: str):
        super().__init__(f"{where} failed: {ERRORS.get(code, code)}")
        self.code = code


class esp_model_cfg(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("n_layers", "d_model", "n_q_heads", "n_kv_heads", "head_dim", "d_ffn",
                                              "vocab", "dtype", "tied_embeddings", "qk_norm")] + \
               [("rope_base", ctypes.c_float), ("rms_eps", ctypes.c_float), ("max_seq_len", ctypes.c_int32),
                ("max_batch", ctypes.c_int32)]


class esp_spec_cfg(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("n_probes", "topk", "max_nodes", "expand_width", "n_anchor",
                                              "prune_parent", "prune_root", "ema_per_token")] + [("lam", ctypes.c_float)] + \
               [("static_widths", ctypes.c_int32 * ESP_MAX_PROBES), ("mask_init", ctypes.c_int32),
                ("temperature", ctypes.c_float), ("seed_lo", ctypes.c_uint32), ("seed_hi", ctypes.c_uint32)]


_PP = ctypes.POINTER(ctypes.c_void_p)


class esp_weights(ctypes.Structure):
    _fields_ = [("embed", ctypes.c_void_p), ("lm_head", ctypes.c_void_p), ("final_norm", ctypes.c_void_p)] + \
               [(n, _PP) for n in ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down", "norm_attn", "norm_ffn",
                                   "q_norm", "k_norm")]


class esp_stats(ctypes.Structure):
    _fields_ = [("steps", ctypes.c_int64), ("emitted", ctypes.c_int64), ("accept_hist", ctypes.c_int64 * (ESP_MAX_PROBES + 1)),
                ("device_error", ctypes.c_int32), ("kernels_per_step", ctypes.c_int32), ("rows_hist", ctypes.c_int64 * 4)]


_lib = None


def load_library(path: Optional[str] = None):
    """dlopen the CUDA library (raises OSError if it was not built)."""
    global _lib
    if _lib is None or path is not None:
        p = path or LIB_PATH
        if not os.path.exists(p):
            raise OSError(f"{p} not found: build it with `python -m paper_2603_17942_b200.build` "
                          f"(there is no fallback implementation)")
        lib = ctypes.CDLL(p)
        for name in EXPORTS:
            getattr(lib, name).restype = None if name == "esp_free" else ctypes.c_int
        if path is not None:
            return lib
        _lib = lib
    return _lib


def _check(rc: int, where: str):
    if rc != 0:
        raise EspError(rc, where)


def _vp(x) -> ctypes.c_void_p:
    if x is None:
        return ctypes.c_void_p(None)
    if hasattr(x, "data_ptr"):
        return ctypes.c_void_p(x.data_ptr())
    if isinstance(x, np.ndarray):
        return ctypes.c_void_p(x.ctypes.data)
    return ctypes.c_void_p(int(x))


def model_cfg(shape, max_seq_len: int, max_batch: int = 1) -> esp_model_cfg:
    """esp_model_cfg from any object with the shape fields (see synth.ModelShape)."""
    return esp_model_cfg(shape.n_layers, shape.d_model, shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.d_ffn,
                         shape.vocab, 0 if shape.dtype == "fp32" else 1, int(bool(shape.tied)), int(bool(shape.qk_norm)),
                         float(shape.rope_base), float(shape.rms_eps), int(max_seq_len), int(max_batch))


def spec_cfg(n_probes=0, topk=1, max_nodes=1, expand_width=1, n_anchor=0, prune_parent=True, prune_root=False,
             ema_per_token=True, lam=0.1, static_widths=(), mask_init=0, temperature=0.0, seed=0) -> esp_spec_cfg:
    widths = (ctypes.c_int32 * ESP_MAX_PROBES)(*[int(w) for w in static_widths])
    return esp_spec_cfg(n_probes, topk, max_nodes, expand_width, n_anchor, int(prune_parent), int(prune_root),
                        int(ema_per_token), float(lam), widths, int(mask_init), float(temperature),
                        int(seed) & 0xffffffff, (int(seed) >> 32) & 0xffffffff)


# ---------------------------------------------------------------- raw calls (same names as the header)
def esp_workspace_bytes(model: esp_model_cfg, spec: esp_spec_cfg) -> int:
    out = ctypes.c_size_t(0)
    _check(load_library().esp_workspace_bytes(ctypes.byref(model), ctypes.byref(spec), ctypes.byref(out)), "esp_workspace_bytes")
    return out.value


def esp_init(model: esp_model_cfg, spec: esp_spec_cfg, weights: esp_weights, workspace, workspace_bytes: int, stream=None):
    h = ctypes.c_void_p(None)
    _check(load_library().esp_init(ctypes.byref(model), ctypes.byref(spec), ctypes.byref(weights), _vp(workspace),
                                   ctypes.c_size_t(workspace_bytes), _vp(stream), ctypes.byref(h)), "esp_init")
    return h


def esp_prefill(h, seq: int, prompt: np.ndarray) -> int:
    prompt = np.ascontiguousarray(prompt, dtype=np.int32)
    first = ctypes.c_int32(-1)
    _check(load_library().esp_prefill(h, ctypes.c_int32(seq), _vp(prompt), ctypes.c_int32(len(prompt)), ctypes.byref(first)), "esp_prefill")
    return first.value


def esp_step(h, tokens_out: np.ndarray, n_out: np.ndarray):
    _check(load_library().esp_step(h, _vp(tokens_out), _vp(n_out)), "esp_step")


def esp_step_async(h):
    _check(load_library().esp_step_async(h), "esp_step_async")


def esp_read(h, tokens_out: np.ndarray, n_out: np.ndarray):
    _check(load_library().esp_read(h, _vp(tokens_out), _vp(n_out)), "esp_read")


def esp_set_mask(h, seq: int, mask):
    mask = np.ascontiguousarray(mask, dtype=np.float32)
    _check(load_library().esp_set_mask(h, ctypes.c_int32(seq), _vp(mask)), "esp_set_mask")


def esp_set_tree(h, seq: int, tokens, parents):
    tokens = np.ascontiguousarray(tokens, dtype=np.int32)
    parents = np.ascontiguousarray(parents, dtype=np.int32)
    _check(load_library().esp_set_tree(h, ctypes.c_int32(seq), _vp(tokens), _vp(parents), ctypes.c_int32(len(tokens))), "esp_set_tree")


def esp_debug_state(h, seq: int, d_model: int, n_probes: int = 1) -> Dict[str, object]:
    R, KP = ESP_MAX_ROWS, ESP_MAX_KPRIME
    out = {"row_token": np.zeros(R, np.int32), "row_parent": np.zeros(R, np.int32), "row_depth": np.zeros(R, np.int32),
           "topk_ids": np.zeros((R, KP), np.int32), "topk_vals": np.zeros((R, KP), np.float32),
           "lse": np.zeros(R, np.float32), "mask_vec": np.zeros((max(n_probes, 1), d_model), np.float32)}
    nn, nr, L = ctypes.c_int32(), ctypes.c_int32(), ctypes.c_int32()
    _check(load_library().esp_debug_state(h, ctypes.c_int32(seq), _vp(out["row_token"]), _vp(out["row_parent"]),
                                          _vp(out["row_depth"]), ctypes.byref(nn), ctypes.byref(nr), ctypes.byref(L),
                                          _vp(out["topk_ids"]), _vp(out["topk_vals"]), _vp(out["lse"]), _vp(out["mask_vec"])),
           "esp_debug_state")
    out.update(n_nodes=nn.value, n_rows=nr.value, L=L.value)
    return out


def esp_debug_capture(h, logits=None, hidden=None):
    _check(load_library().esp_debug_capture(h, _vp(logits), _vp(hidden)), "esp_debug_capture")


def esp_debug_set_gemm(h, impl: int):
    _check(load_library().esp_debug_set_gemm(h, ctypes.c_int32(impl)), "esp_debug_set_gemm")


def esp_debug_set_layer_kernel(h, mode: int):
    """1: one kernel per operation (default), 0: all decoder layers in one persistent cooperative kernel."""
    _check(load_library().esp_debug_set_layer_kernel(h, ctypes.c_int32(mode)), "esp_debug_set_layer_kernel")


def esp_debug_layer_timeline(h, n_layers: int) -> np.ndarray:
    """Global-timer stamps (ns) of the last profiled step: [n_layers][10 barriers][8 words] (see esp.h)."""
    out = np.zeros(n_layers * 80, np.uint64)
    n = ctypes.c_int32(0)
    _check(load_library().esp_debug_layer_timeline(h, _vp(out), ctypes.c_int32(out.size), ctypes.byref(n)), "esp_debug_layer_timeline")
    return out[:n.value].reshape(-1, 10, 8)


KINDS = ("norm_and_partial_consumers", "qkv_gemm", "tree_attention", "o_gemm", "gateup_gemm", "down_gemm", "lmhead_topk", "select_tree")


def esp_step_profiled(h, tokens_out: np.ndarray, n_out: np.ndarray) -> Dict[str, float]:
    ms = np.zeros(8, np.float32)
    _check(load_library().esp_step_profiled(h, _vp(ms), _vp(tokens_out), _vp(n_out)), "esp_step_profiled")
    return {k: float(v) for k, v in zip(KINDS, ms)}


def esp_get_stats(h) -> esp_stats:
    st = esp_stats()
    _check(load_library().esp_get_stats(h, ctypes.byref(st)), "esp_get_stats")
    return st


def esp_debug_wait_selftest(scratch, stream=None) -> int:
    """Runs the bounded-wait self-test; returns the device status code the kernel recorded (1 = timed out)."""
    st = ctypes.c_int32(-1)
    _check(load_library().esp_debug_wait_selftest(_vp(scratch), _vp(stream), ctypes.byref(st)), "esp_debug_wait_selftest")
    return st.value


def esp_debug_gumbel(seed: int, position: int, n_tokens: int, noise_out, stream=None):
    _check(load_library().esp_debug_gumbel(ctypes.c_uint32(seed & 0xffffffff), ctypes.c_uint32((seed >> 32) & 0xffffffff),
                                           ctypes.c_uint32(position), ctypes.c_int32(n_tokens), _vp(noise_out), _vp(stream)),
           "esp_debug_gumbel")


def esp_free(h):
    load_library().esp_free(h)


def esp_tree_attention_scratch_bytes(batch: int, n_q_heads: int, head_dim: int, cap: int) -> int:
    out = ctypes.c_size_t(0)
    _check(load_library().esp_tree_attention_scratch_bytes(ctypes.c_int32(batch), ctypes.c_int32(n_q_heads),
                                                           ctypes.c_int32(head_dim), ctypes.c_int32(cap), ctypes.byref(out)),
           "esp_tree_attention_scratch_bytes")
    return out.value


def esp_tree_attention(dtype: int, batch: int, n_rows: int, L: int, cap: int, n_q_heads: int, n_kv_heads: int, head_dim: int,
                       dcap: int, q, kcache, vcache, anc, depth, out, scratch, scratch_bytes: int, stream=None):
    _check(load_library().esp_tree_attention(
        ctypes.c_int32(dtype), ctypes.c_int32(batch), ctypes.c_int32(n_rows), ctypes.c_int32(L), ctypes.c_int32(cap),
        ctypes.c_int32(n_q_heads), ctypes.c_int32(n_kv_heads), ctypes.c_int32(head_dim), ctypes.c_int32(dcap), _vp(q),
        _vp(kcache), _vp(vcache), _vp(anc), _vp(depth), _vp(out), _vp(scratch), ctypes.c_size_t(scratch_bytes), _vp(stream)),
        "esp_tree_attention")


ESP_STATIC_SCRATCH_BYTES = 32 << 20


def esp_tree_attention_static(dtype: int, batch: int, n_rows: int, L: int, cap: int, n_q_heads: int, n_kv_heads: int,
                              head_dim: int, dcap: int, q, kcache, vcache, anc, depth, out, stream=None):
    """esp_tree_attention with the library's built-in 32 MiB scratch array: no scratch argument, no allocation."""
    _check(load_library().esp_tree_attention_static(
        ctypes.c_int32(dtype), ctypes.c_int32(batch), ctypes.c_int32(n_rows), ctypes.c_int32(L), ctypes.c_int32(cap),
        ctypes.c_int32(n_q_heads), ctypes.c_int32(n_kv_heads), ctypes.c_int32(head_dim), ctypes.c_int32(dcap), _vp(q),
        _vp(kcache), _vp(vcache), _vp(anc), _vp(depth), _vp(out), _vp(stream)), "esp_tree_attention_static")


def esp_tree_attention_status(scratch=None, stream=None) -> int:
    """Device status word of the last tree attention on `scratch` (None: on the built-in array); raises EspError(ESP_E_DEVICE) if set."""
    st = ctypes.c_int32(0)
    _check(load_library().esp_tree_attention_status(_vp(scratch), _vp(stream), ctypes.byref(st)), "esp_tree_attention_status")
    return st.value


def esp_gemm_scratch_bytes() -> int:
    out = ctypes.c_size_t(0)
    _check(load_library().esp_gemm_scratch_bytes(ctypes.byref(out)), "esp_gemm_scratch_bytes")
    return out.value


def esp_gemm_bf16(impl: int, rows: int, n_out: int, k_in: int, x, w, y, scratch, scratch_bytes: int, stream=None):
    _check(load_library().esp_gemm_bf16(ctypes.c_int32(impl), ctypes.c_int32(rows), ctypes.c_int32(n_out), ctypes.c_int32(k_in),
                                        _vp(x), _vp(w), _vp(y), _vp(scratch), ctypes.c_size_t(scratch_bytes), _vp(stream)),
           "esp_gemm_bf16")


# ---------------------------------------------------------------- convenience: a handle that keeps its tensors alive
class Handle:
    """esp_init + the tensors it points at.  ``weights`` is a dict of CUDA tensors (see synth.make_weights)."""

    def __init__(self, shape, spec: esp_spec_cfg, weights: Dict[str, object], max_seq_len: int, max_batch: int = 1, stream=None):
        import torch
        self.shape, self.spec = shape, spec
        self.model = model_cfg(shape, max_seq_len, max_batch)
        self.weights = weights
        self.max_batch = max_batch
        w = esp_weights()
        w.embed, w.lm_head, w.final_norm = weights["embed"].data_ptr(), weights["lm_head"].data_ptr(), weights["final_norm"].data_ptr()
        self._arrays = []
        for n in ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down", "norm_attn", "norm_ffn", "q_norm", "k_norm"):
            arr = (ctypes.c_void_p * shape.n_layers)(*[t.data_ptr() for t in weights[n]])
            self._arrays.append(arr)
            setattr(w, n, ctypes.cast(arr, _PP))
        self._w = w
        self.workspace_bytes = esp_workspace_bytes(self.model, spec)
        self.workspace = torch.empty(self.workspace_bytes, dtype=torch.uint8, device=weights["embed"].device)
        self.stream = stream
        sp = stream.cuda_stream if stream is not None else None
        self.h = esp_init(self.model, spec, w, self.workspace, self.workspace_bytes, sp)
        self.tokens_out = np.zeros((max_batch, ESP_MAX_PROBES + 1), np.int32)
        self.n_out = np.zeros(max_batch, np.int32)

    def prefill(self, prompt, seq: int = 0) -> int:
        return esp_prefill(self.h, seq, prompt)

    def step(self, seq: int = 0) -> List[int]:
        esp_step(self.h, self.tokens_out, self.n_out)
        return [int(t) for t in self.tokens_out[seq, :self.n_out[seq]]]

    def step_async(self):
        esp_step_async(self.h)

    def read(self, seq: int = 0) -> List[int]:
        esp_read(self.h, self.tokens_out, self.n_out)
        return [int(t) for t in self.tokens_out[seq, :self.n_out[seq]]]

    def generate(self, prompt, max_new: int, seq: int = 0) -> List[int]:
        out = [self.prefill(prompt, seq)]
        while len(out) < max_new:
            out.extend(self.step(seq))
        return out[:max_new]

    def set_tree(self, tokens, parents, seq: int = 0):
        esp_set_tree(self.h, seq, tokens, parents)

    def set_mask(self, mask, seq: int = 0):
        esp_set_mask(self.h, seq, mask)

    def state(self, seq: int = 0):
        return esp_debug_state(self.h, seq, self.shape.d_model, self.spec.n_probes)

    def stats(self) -> esp_stats:
        return esp_get_stats(self.h)

    def close(self):
        if self.h is not None:
            esp_free(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
