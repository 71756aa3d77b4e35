"""Thin ctypes binding of the C-ABI library (include/medusa.h): same names, argument marshalling only.

torch is used for device memory and streams; every computation of the path runs inside the CUDA
library.  Loading fails loudly if the library has not been built; creating a context fails if no CUDA
device is present.  There is no CPU fallback.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libmedusa_b200.so")

OK, ERR_INVALID_ARG, ERR_SHAPE, ERR_UNSUPPORTED, ERR_CACHE_FULL, ERR_CUDA, ERR_TIMEOUT, ERR_STATE = 0, -1, -2, -3, -4, -5, -6, -7
F32, BF16 = 0, 1
GREEDY, TYPICAL, REJECTION = 0, 1, 2  # REJECTION: the noise row is gumbel[V] followed by uniform[T]
(WS_LOGITS, WS_HIDDEN, WS_TREE_K, WS_TREE_V, WS_K_CACHE, WS_V_CACHE, WS_HEAD_LOGITS, WS_TOPK_IDX, WS_TREE_TOK,
 WS_ACC_NODES, WS_STATE, WS_H_LAST, WS_EMITTED, WS_TAP_X_IN, WS_TAP_X_OUT, WS_TAP_ATT, WS_TAP_XN_OUT) = range(17)
(OPT_STEP_GRAPHS, OPT_ATTENTION_KERNEL, OPT_ATTENTION_LENGTH_HINT, OPT_LAYER_TAP, OPT_SPIN_LIMIT,
 OPT_WITHHOLD_LOAD, OPT_ACTIVATION_PLANES, OPT_PACK_WEIGHTS) = range(8)
LAYER_KEYS = ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "w_gate", "w_up", "w_down")


class MedusaError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__("medusa error %d: %s" % (code, msg))
        self.code = code


class ModelDesc(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("d", C.c_int32), ("n_heads", C.c_int32), ("head_dim", C.c_int32),
                ("ffn", C.c_int32), ("vocab", C.c_int32), ("n_medusa", C.c_int32), ("dtype", C.c_int32),
                ("L_max", C.c_int32), ("n_kv_heads", C.c_int32), ("rms_eps", C.c_float), ("rope_theta", C.c_float),
                ("max_tree_nodes", C.c_int32), ("max_batch", C.c_int32)]


class TreeBuffers(C.Structure):
    _fields_ = [("T", C.c_int32), ("P", C.c_int32), ("depth", C.c_int32), ("topk", C.c_int32),
                ("mask", C.c_void_p), ("pos", C.c_void_p), ("tree_idx", C.c_void_p), ("parent", C.c_void_p),
                ("retrieve", C.c_void_p)]


class AcceptParams(C.Structure):
    _fields_ = [("mode", C.c_int32), ("temperature", C.c_float), ("eps", C.c_float), ("delta", C.c_float)]


class Weights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("final_norm", C.c_void_p), ("lm_head", C.c_void_p),
                ("layers_host", C.POINTER(C.c_void_p)), ("medusa_w1", C.c_void_p), ("medusa_w2", C.c_void_p)]


_lib = None


def use_checked_library():
    """Selects the checked flavour of the library (built with `python -m paper_2401_10774_b200.build --debug-checks`):
    the same entry points, plus device-side validation kernels after the stages of a step.  Call before the first use."""
    global LIB_PATH
    if _lib is not None:
        raise RuntimeError("the CUDA library is already open; choose the flavour before the first call")
    LIB_PATH = os.path.join(_PKG, "libmedusa_b200_checked.so")


def lib():
    """Opens the CUDA library; raises if it is missing (build it with `python -m paper_2401_10774_b200.build`)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("%s not found: the CUDA library must be built first "
                               "(python -m paper_2401_10774_b200.build); there is no fallback path" % LIB_PATH)
        L = C.CDLL(LIB_PATH)
        L.medusa_last_error.restype = C.c_char_p
        L.medusa_last_error.argtypes = [C.c_void_p]
        L.medusa_workspace_ptr.restype = C.c_void_p
        L.medusa_workspace_ptr.argtypes = [C.c_void_p, C.c_int32]
        _lib = L
    return _lib


def _ptr(t):
    """Device (torch) tensor, numpy array, raw int address or None -> c_void_p."""
    if t is None:
        return C.c_void_p(0)
    if isinstance(t, int):
        return C.c_void_p(t)
    if isinstance(t, np.ndarray):
        return C.c_void_p(t.ctypes.data)
    return C.c_void_p(t.data_ptr())


def default_tree_paths(per_depth_topk, n_nodes) -> np.ndarray:
    tk = np.ascontiguousarray(per_depth_topk, dtype=np.int32)
    out = np.full((max(n_nodes - 1, 1), tk.size), -1, dtype=np.int32)
    n = lib().medusa_default_tree_paths(_ptr(tk), C.c_int32(tk.size), C.c_int32(n_nodes), _ptr(out))
    if n < 0:
        raise MedusaError(n, "medusa_default_tree_paths")
    return out[:n]


def tree_paths_from_accuracies(acc, n_nodes):
    """acc: [depth][topk] accuracies in [0, 1] -> (paths [n_nodes-1][depth], expected accepted speculated tokens)"""
    a = np.ascontiguousarray(acc, dtype=np.float64)
    if a.ndim != 2:
        raise ValueError("acc must be a [depth][topk] table")
    depth, topk = a.shape
    out = np.full((max(n_nodes - 1, 1), depth), -1, dtype=np.int32)
    expect = C.c_double(0.0)
    n = lib().medusa_tree_paths_from_accuracies(_ptr(a), C.c_int32(depth), C.c_int32(topk), C.c_int32(n_nodes), _ptr(out),
                                                C.byref(expect))
    if n < 0:
        raise MedusaError(n, "medusa_tree_paths_from_accuracies")
    return out[:n], expect.value


def build_tree_buffers(ctx, paths, max_depth=None) -> dict:
    """Host tree buffers as numpy arrays; uploads them into `ctx` if it is not None."""
    paths = np.ascontiguousarray(paths, dtype=np.int32)
    if paths.ndim == 1:
        paths = paths.reshape(0, max_depth or 1)
    n_paths, md = paths.shape
    T = n_paths + 1
    W = (T + 63) // 64
    mask = np.zeros(T * W, dtype=np.uint64)
    pos, tree_idx, parent = (np.zeros(T, dtype=np.int32) for _ in range(3))
    retrieve = np.full(T * (md + 1), -1, dtype=np.int32)
    tb = TreeBuffers(mask=mask.ctypes.data, pos=pos.ctypes.data, tree_idx=tree_idx.ctypes.data,
                     parent=parent.ctypes.data, retrieve=retrieve.ctypes.data)
    h = ctx.handle if ctx is not None else C.c_void_p(0)
    rc = lib().medusa_build_tree_buffers(h, _ptr(paths), C.c_int32(n_paths), C.c_int32(md), C.byref(tb))
    if rc != OK:
        raise MedusaError(rc, ctx.last_error() if ctx is not None else "invalid tree")
    if W > 1:
        mask = mask.reshape(T, W)
    tree = dict(T=tb.T, P=tb.P, depth=tb.depth, topk=tb.topk, mask=mask, pos=pos, tree_idx=tree_idx, parent=parent,
                retrieve=retrieve[: tb.P * (tb.depth + 1)].reshape(tb.P, tb.depth + 1).copy())
    if ctx is not None:
        ctx.tree = tree
    return tree


class Context:
    """Owns a medusa_ctx.  Methods mirror the C entry points and take device tensors (torch) as arguments."""

    def __init__(self, cfg: dict, dtype: int, L_max: int, device: int = 0, stream=None):
        self.cfg = dict(cfg)
        self.dtype = dtype
        self.L_max = L_max
        self.tree = None
        self._keep = []
        desc = ModelDesc(n_layers=cfg["n_layers"], d=cfg["d"], n_heads=cfg["n_heads"], head_dim=cfg["head_dim"],
                         ffn=cfg["ffn"], vocab=cfg["vocab"], n_medusa=cfg["n_medusa"], dtype=dtype, L_max=L_max,
                         n_kv_heads=cfg.get("n_kv_heads", 0), rms_eps=cfg.get("rms_eps", 1e-5), rope_theta=cfg.get("rope_theta", 1e4),
                         max_tree_nodes=cfg.get("max_tree_nodes", 0), max_batch=cfg.get("max_batch", 0))
        self.handle = C.c_void_p(0)
        sp = C.c_void_p(0 if stream is None else int(stream))
        rc = lib().medusa_create(C.byref(self.handle), C.byref(desc), C.c_int32(device), sp)
        if rc != OK:
            msg = self.last_error() if self.handle else "medusa_create failed (no CUDA device? unsupported shape?)"
            if self.handle:
                lib().medusa_destroy(self.handle)
                self.handle = C.c_void_p(0)
            raise MedusaError(rc, msg)

    def close(self):
        if self.handle:
            lib().medusa_destroy(self.handle)
            self.handle = C.c_void_p(0)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def last_error(self) -> str:
        return lib().medusa_last_error(self.handle).decode()

    def _check(self, rc):
        if rc != OK:
            raise MedusaError(rc, self.last_error())

    # ---- per-operation entry points -------------------------------------------------------------------
    def build_tree_buffers(self, paths, max_depth=None):
        return build_tree_buffers(self, paths, max_depth)

    def medusa_heads(self, h, W1, W2, root_token, topk_idx, topk_val, logits_dump, tree_tok):
        self._check(lib().medusa_heads(self.handle, _ptr(h), _ptr(W1), _ptr(W2), _ptr(root_token), _ptr(topk_idx),
                                       _ptr(topk_val), _ptr(logits_dump), _ptr(tree_tok)))

    def tree_attention(self, q, k_new, v_new, k_cache, v_cache, cache_len, apply_rope, out, lse=None):
        self._check(lib().medusa_tree_attention(self.handle, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(k_cache),
                                                _ptr(v_cache), _ptr(cache_len), C.c_int32(1 if apply_rope else 0),
                                                _ptr(out), _ptr(lse)))

    def evaluate_posterior(self, logits, tree_tok, params: AcceptParams, gumbel, best, accept_len, next_root,
                           acc_nodes):
        self._check(lib().medusa_evaluate_posterior(self.handle, _ptr(logits), _ptr(tree_tok), C.byref(params),
                                                    _ptr(gumbel), _ptr(best), _ptr(accept_len), _ptr(next_root),
                                                    _ptr(acc_nodes)))

    def accept_and_update_kv(self, tree_k, tree_v, k_cache, v_cache, acc_nodes, accept_len, max_commit, cache_len,
                             hidden, h_last, tree_tok, emitted, n_emitted):
        self._check(lib().medusa_accept_and_update_kv(self.handle, _ptr(tree_k), _ptr(tree_v), _ptr(k_cache),
                                                      _ptr(v_cache), _ptr(acc_nodes), _ptr(accept_len),
                                                      C.c_int32(max_commit), _ptr(cache_len), _ptr(hidden),
                                                      _ptr(h_last), _ptr(tree_tok), _ptr(emitted), _ptr(n_emitted)))

    # ---- driver ---------------------------------------------------------------------------------------
    def load_weights(self, w: dict):
        """w: dict of device tensors (embed, final_norm, lm_head, layers=[{...}], medusa_w1, medusa_w2)."""
        n = self.cfg["n_layers"]
        arr = (C.c_void_p * max(n * 9, 1))()
        for l in range(n):
            for j, k in enumerate(LAYER_KEYS):
                arr[l * 9 + j] = w["layers"][l][k].data_ptr()
        cw = Weights(embed=w["embed"].data_ptr(), final_norm=w["final_norm"].data_ptr(),
                     lm_head=w["lm_head"].data_ptr(), layers_host=C.cast(arr, C.POINTER(C.c_void_p)),
                     medusa_w1=w["medusa_w1"].data_ptr() if w.get("medusa_w1") is not None else None,
                     medusa_w2=w["medusa_w2"].data_ptr() if w.get("medusa_w2") is not None else None)
        self._keep.append(w)  # the library keeps raw pointers: keep the tensors alive
        self._check(lib().medusa_load_weights(self.handle, C.byref(cw)))

    def reset(self):
        self._check(lib().medusa_reset(self.handle))

    def prefill(self, prompt_dev, n=None):
        self._check(lib().medusa_prefill(self.handle, _ptr(prompt_dev), C.c_int32(int(n if n is not None else prompt_dev.numel()))))

    def tree_pass(self, tokens_dev):
        self._check(lib().medusa_tree_pass(self.handle, _ptr(tokens_dev)))

    def decode_step(self, params: AcceptParams, gumbel=None, max_commit=1 << 30, emitted_host=None, n_emitted_host=None):
        self._check(lib().medusa_decode_step(self.handle, C.byref(params), _ptr(gumbel), C.c_int32(int(max_commit)),
                                             _ptr(emitted_host), _ptr(n_emitted_host)))

    def select_sequence(self, b: int):
        self._check(lib().medusa_select_sequence(self.handle, C.c_int32(int(b))))

    def decode_step_batch(self, params: AcceptParams, gumbel=None, max_commit=1 << 30, emitted_host=None, n_emitted_host=None):
        self._check(lib().medusa_decode_step_batch(self.handle, C.byref(params), _ptr(gumbel), C.c_int32(int(max_commit)),
                                                   _ptr(emitted_host), _ptr(n_emitted_host)))

    def heads_loss_and_grads(self, hidden, labels, loss, grad_w1, grad_w2, lam=None):
        """Medusa-1 objective and its gradient w.r.t. the heads (device tensors; lam: host floats [K] or None)."""
        n = int(hidden.shape[0])
        la = None if lam is None else np.ascontiguousarray(lam, dtype=np.float32)
        self._check(lib().medusa_heads_loss_and_grads(self.handle, _ptr(hidden), _ptr(labels), C.c_int32(n), _ptr(la),
                                                      _ptr(loss), _ptr(grad_w1), _ptr(grad_w2)))

    def generate(self, prompt_host: np.ndarray, G: int, params: AcceptParams, gumbel_host=None) -> dict:
        prompt = np.ascontiguousarray(prompt_host, dtype=np.int32)
        out = np.zeros(max(G, 1), dtype=np.int32)
        hist = np.zeros(max(G, 1), dtype=np.int32)
        steps = C.c_int32(0)
        g = None if gumbel_host is None else np.ascontiguousarray(gumbel_host, dtype=np.float32)
        self._check(lib().medusa_generate(self.handle, _ptr(prompt), C.c_int32(prompt.size), C.c_int32(G),
                                          C.byref(params), _ptr(g), _ptr(out), _ptr(hist), C.byref(steps)))
        return dict(tokens=out[:G], steps=steps.value, emitted_per_step=hist[: steps.value])

    PROF_NAMES = ("gemm", "tree_attention", "heads_gemv", "elementwise", "topk_expand", "posterior", "commit", "other")

    def set_profiling(self, on: bool):
        self._check(lib().medusa_set_profiling(self.handle, C.c_int32(1 if on else 0)))

    def get_profile(self, reset: bool = True) -> dict:
        ms = np.zeros(8, dtype=np.float64)
        n = np.zeros(8, dtype=np.int64)
        self._check(lib().medusa_get_profile(self.handle, _ptr(ms), _ptr(n), C.c_int32(1 if reset else 0)))
        return {k: dict(ms=float(ms[i]), launches=int(n[i])) for i, k in enumerate(self.PROF_NAMES)}

    def set_option(self, option: int, value: int):
        self._check(lib().medusa_set_option(self.handle, C.c_int32(option), C.c_int64(int(value))))

    def step_graph_info(self) -> dict:
        n, r = C.c_int32(0), C.c_int64(0)
        self._check(lib().medusa_step_graph_info(self.handle, C.byref(n), C.byref(r)))
        return dict(graphs=n.value, replays=r.value)

    def device_status(self) -> int:
        return lib().medusa_device_status(self.handle)

    def workspace_ptr(self, which: int) -> int:
        return lib().medusa_workspace_ptr(self.handle, C.c_int32(which)) or 0

    # ---- inspection helpers (host copies of context-owned buffers) ----
    def read_workspace(self, which: int, shape, np_dtype, offset_elems: int = 0) -> np.ndarray:
        """Host copy of (part of) a workspace buffer as a numpy array (bf16 buffers: pass np.uint16)."""
        out = np.empty(shape, dtype=np_dtype)
        self._check(lib().medusa_read_workspace(self.handle, C.c_int32(which),
                                                C.c_int64(offset_elems * out.itemsize), _ptr(out),
                                                C.c_int64(out.nbytes)))
        return out

    def state(self) -> dict:
        s = self.read_workspace(WS_STATE, (8,), np.int32).tolist()
        return dict(cache_len=s[0], root=s[1], best=s[2], accept_len=s[3], next_root=s[4], n_emitted=s[5], status=s[6])


def stream_read(buf, nbytes: int, sink, stream=None):
    """medusa_stream_read: enqueue one read-only pass over `nbytes` bytes of device tensor `buf` (timing aid)."""
    rc = lib().medusa_stream_read(_ptr(buf), C.c_int64(int(nbytes)), _ptr(sink), C.c_int32(int(sink.numel())),
                                  C.c_void_p(0 if stream is None else int(stream)))
    if rc != OK:
        raise MedusaError(rc, "medusa_stream_read")


def tree_attention_static(q, k_new, v_new, k_cache, v_cache, cache_len, mask, T, H, L_max, L_hint, out, lse=None,
                          stream=None):
    """medusa_tree_attention_static: tree attention (bf16, head_dim 128, inputs already rotated) that needs no
    context and allocates nothing -- its split-KV scratch is a fixed array inside the library.  For callers that
    cannot allocate device memory when they call (own memory pool, no implicit synchronisation allowed, no
    context).  Arguments are device tensors; `mask` is the uint64 [T] ancestor mask on the device."""
    rc = lib().medusa_tree_attention_static(_ptr(q), _ptr(k_new), _ptr(v_new), _ptr(k_cache), _ptr(v_cache),
                                            _ptr(cache_len), _ptr(mask), C.c_int32(T), C.c_int32(H), C.c_int32(L_max),
                                            C.c_int32(L_hint), _ptr(out), _ptr(lse),
                                            C.c_void_p(0 if stream is None else int(stream)))
    if rc != OK:
        raise MedusaError(rc, "medusa_tree_attention_static failed (see stderr for the reason)")
