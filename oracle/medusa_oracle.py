"""ctypes front end of the CPU oracle (medusa_oracle.c).  TEST INFRASTRUCTURE, NOT THE PRODUCT.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this module.  It holds
no arithmetic of its own: every function marshals numpy arrays into the C oracle and back (the heads' training
objective, re-exported at the end, is the one exception: it is written out in numpy in medusa1_training.py).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "medusa_oracle.c")
_LIB = os.path.join(_HERE, "libmedusa_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain C, OpenMP over independent rows only)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fopenmp", "-ffp-contract=off", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


class _Model(C.Structure):
    _fields_ = [
        ("n_layers", C.c_int32), ("d", C.c_int32), ("n_heads", C.c_int32), ("head_dim", C.c_int32),
        ("ffn", C.c_int32), ("vocab", C.c_int32), ("n_medusa", C.c_int32), ("wdtype", C.c_int32),
        ("n_kv_heads", C.c_int32), ("kv_bf16", C.c_int32),
        ("rms_eps", C.c_double), ("rope_theta", C.c_double),
        ("embed", C.c_void_p), ("final_norm", C.c_void_p), ("lm_head", C.c_void_p),
        ("layers", C.POINTER(C.c_void_p)),
        ("medusa_w1", C.c_void_p), ("medusa_w2", C.c_void_p),
    ]


class _Tree(C.Structure):
    _fields_ = [
        ("T", C.c_int32), ("P", C.c_int32), ("depth", C.c_int32), ("topk", C.c_int32),
        ("mask", C.c_void_p), ("pos", C.c_void_p), ("tree_idx", C.c_void_p), ("parent", C.c_void_p),
        ("retrieve", C.c_void_p),
    ]


def lib():
    global _lib
    with _lock:
        if _lib is None:
            _lib = C.CDLL(build())
            _lib.ora_silu.restype = C.c_double
            _lib.ora_silu.argtypes = [C.c_double]
            _lib.ora_rope.argtypes = [C.c_void_p, C.c_int32, C.c_int64, C.c_double]
            _lib.ora_rmsnorm.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_double, C.c_void_p]
    return _lib


def _p(a):
    return None if a is None else C.c_void_p(a.ctypes.data)


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


# ----------------------------------------------------------------------------- trees

def default_tree_paths(per_depth_topk, n_nodes):
    tk = _i32(per_depth_topk)
    depth = int(tk.size)
    out = np.full((max(n_nodes - 1, 1), depth), -1, dtype=np.int32)
    n = lib().ora_default_tree_paths(_p(tk), C.c_int32(depth), C.c_int32(n_nodes), _p(out))
    if n < 0:
        raise ValueError("ora_default_tree_paths rejected its arguments")
    return out[:n]


def tree_paths_from_accuracies(acc, n_nodes):
    """Sec. 2.3.3 greedy node adding; acc: [depth][topk] accuracies in [0, 1] -> (paths [n_nodes-1][depth], expected
    number of accepted speculated tokens)"""
    a = np.ascontiguousarray(acc, dtype=np.float64)
    depth, topk = a.shape
    out = np.full((max(n_nodes - 1, 1), depth), -1, dtype=np.int32)
    expect = C.c_double(0.0)
    n = lib().ora_tree_paths_from_accuracies(_p(a), C.c_int32(depth), C.c_int32(topk), C.c_int32(n_nodes), _p(out),
                                             C.byref(expect))
    if n < 0:
        raise ValueError("ora_tree_paths_from_accuracies rejected its arguments")
    return out[:n], expect.value


def build_tree_buffers(paths, max_depth=None):
    """-> dict(T, P, depth, topk, mask u64[T] (u64[T][ceil(T/64)] for trees of more than 64 nodes), pos, tree_idx,
    parent i32[T], retrieve i32[P][depth+1])"""
    paths = _i32(paths)
    if paths.ndim == 1:
        paths = paths.reshape(0, max_depth or 1)
    n_paths, md = paths.shape
    T = n_paths + 1
    dims = np.zeros(4, dtype=np.int32)
    W = (T + 63) // 64
    mask = np.zeros(T * W, dtype=np.uint64)
    pos = np.zeros(T, dtype=np.int32)
    tree_idx = np.zeros(T, dtype=np.int32)
    parent = np.zeros(T, dtype=np.int32)
    retrieve = np.full((T, md + 1), -1, dtype=np.int32)
    rc = lib().ora_build_tree_buffers(_p(paths), C.c_int32(n_paths), C.c_int32(md), _p(dims), _p(mask), _p(pos),
                                      _p(tree_idx), _p(parent), _p(retrieve))
    if rc != 0:
        raise ValueError("ora_build_tree_buffers: invalid tree (code %d)" % rc)
    T, P, depth, topk = (int(x) for x in dims)
    retrieve = retrieve.reshape(-1)[: P * (depth + 1)].reshape(P, depth + 1).copy()
    if W > 1:
        mask = mask.reshape(T, W)
    return dict(T=T, P=P, depth=depth, topk=topk, mask=mask, pos=pos, tree_idx=tree_idx, parent=parent,
                retrieve=retrieve)


def chain_tree(T):
    """Tree buffers of a chain (node i's parent is i-1): tree attention reduces to causal attention."""
    mask = np.array([(1 << (i + 1)) - 1 for i in range(T)], dtype=np.uint64)
    return dict(T=T, P=1, depth=T - 1, topk=1, mask=mask, pos=np.arange(T, dtype=np.int32),
                tree_idx=np.arange(T, dtype=np.int32), parent=np.arange(-1, T - 1, dtype=np.int32),
                retrieve=np.arange(T, dtype=np.int32).reshape(1, T))


# ----------------------------------------------------------------------------- heads / top-k / candidates

def _wdtype(a):
    if a.dtype == np.float32:
        return 0
    if a.dtype == np.uint16:
        return 1
    raise TypeError("weights must be float32 or bf16 bit patterns (uint16), got %s" % a.dtype)


def medusa_heads(h, W1, W2):
    """h [d]; W1 [K][d][d]; W2 [K][V][d] (float32 or uint16 bf16 bits) -> (x [K][d], logits [K][V]) float64"""
    h = _f64(h)
    W1 = np.ascontiguousarray(W1)
    W2 = np.ascontiguousarray(W2)
    K, V, d = W2.shape
    x = np.zeros((K, d), dtype=np.float64)
    z = np.zeros((K, V), dtype=np.float64)
    lib().ora_medusa_heads(_p(h), _p(W1), _p(W2), C.c_int32(_wdtype(W2)), C.c_int32(K), C.c_int32(d), C.c_int32(V),
                           _p(x), _p(z))
    return x, z


def topk(values_f32, k):
    v = _f32(values_f32)
    out = np.zeros(k, dtype=np.int32)
    lib().ora_topk(_p(v), C.c_int32(v.size), C.c_int32(k), _p(out))
    return out


def expand_candidates(root, topk_idx, tree):
    tk = _i32(topk_idx)
    T, P, depth = tree["T"], tree["P"], tree["depth"]
    tree_tok = np.zeros(T, dtype=np.int32)
    cand = np.zeros((P, depth + 1), dtype=np.int32)
    lib().ora_expand_candidates(C.c_int32(int(root)), _p(tk), C.c_int32(tree["topk"]), _p(_i32(tree["tree_idx"])),
                                C.c_int32(T), _p(_i32(tree["retrieve"])), C.c_int32(P), C.c_int32(depth),
                                _p(tree_tok), _p(cand))
    return tree_tok, cand


# ----------------------------------------------------------------------------- attention

def tree_attention(q, k_new, v_new, k_cache, v_cache, L, mask, pos, apply_rope=True, rope_theta=1e4):
    """q [T][H][D]; k_new, v_new [T][Hkv][D]; caches [Hkv][L_max][D] (float32), Hkv dividing H (grouped-query
    attention: query head h reads key/value head h // (H // Hkv)) -> (out [T][H][D], lse [T][H]) float64"""
    q, k_new, v_new = _f32(q), _f32(k_new), _f32(v_new)
    k_cache, v_cache = _f32(k_cache), _f32(v_cache)
    T, H, D = q.shape
    Hkv = k_new.shape[1]
    if H % Hkv or v_new.shape != k_new.shape or k_cache.shape[0] != Hkv or v_cache.shape != k_cache.shape:
        raise ValueError("inconsistent head counts")
    L_max = k_cache.shape[1]
    out = np.zeros((T, H, D), dtype=np.float64)
    lse = np.zeros((T, H), dtype=np.float64)
    mask = np.ascontiguousarray(mask, dtype=np.uint64)
    lib().ora_tree_attention(_p(q), _p(k_new), _p(v_new), _p(k_cache), _p(v_cache), C.c_int32(T), C.c_int32(H),
                             C.c_int32(Hkv), C.c_int32(D), C.c_int32(int(L)), C.c_int32(L_max), _p(mask), _p(_i32(pos)),
                             C.c_int32(1 if apply_rope else 0), C.c_double(rope_theta), _p(out), _p(lse))
    return out, lse


# ----------------------------------------------------------------------------- model plumbing

LAYER_KEYS = ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "w_gate", "w_up", "w_down")


class Model:
    """Holds numpy weights (float32, or uint16 bf16 bit patterns) and the C struct pointing at them."""

    def __init__(self, cfg: dict, weights: dict, kv_bf16: bool = False):
        """kv_bf16: every pass holds its tree keys/values (and therefore everything committed to the cache) as a
        bfloat16 KV cache holds them -- the storage precision the bf16 workloads define."""
        self.cfg = dict(cfg)
        self.w = weights
        any_w = np.ascontiguousarray(weights["lm_head"])
        wd = _wdtype(any_w)
        keep = []

        def ptr(a):
            a = np.ascontiguousarray(a)
            if _wdtype(a) != wd:
                raise TypeError("all weights must share one dtype")
            keep.append(a)
            return a.ctypes.data

        n_layers = cfg["n_layers"]
        arr = (C.c_void_p * (n_layers * 9))()
        for l in range(n_layers):
            for j, key in enumerate(LAYER_KEYS):
                arr[l * 9 + j] = ptr(weights["layers"][l][key])
        self._arr = arr
        self._keep = keep
        self.c = _Model(
            n_layers=n_layers, d=cfg["d"], n_heads=cfg["n_heads"], head_dim=cfg["head_dim"], ffn=cfg["ffn"],
            vocab=cfg["vocab"], n_medusa=cfg["n_medusa"], wdtype=wd, n_kv_heads=cfg.get("n_kv_heads", 0),
            kv_bf16=1 if kv_bf16 else 0,
            rms_eps=cfg.get("rms_eps", 1e-5), rope_theta=cfg.get("rope_theta", 1e4),
            embed=ptr(weights["embed"]), final_norm=ptr(weights["final_norm"]), lm_head=ptr(weights["lm_head"]),
            layers=C.cast(arr, C.POINTER(C.c_void_p)),
            medusa_w1=ptr(weights["medusa_w1"]) if cfg["n_medusa"] else None,
            medusa_w2=ptr(weights["medusa_w2"]) if cfg["n_medusa"] else None,
        )

    def cache_shape(self, L_max):
        c = self.cfg
        return (c["n_layers"], self.kv_heads, L_max, c["head_dim"])

    @property
    def kv_heads(self):
        return self.cfg.get("n_kv_heads", 0) or self.cfg["n_heads"]


def _ctree(tree):
    keep = [np.ascontiguousarray(tree["mask"], dtype=np.uint64), _i32(tree["pos"]), _i32(tree["tree_idx"]),
            _i32(tree["parent"]), _i32(tree["retrieve"])]
    t = _Tree(T=tree["T"], P=tree["P"], depth=tree["depth"], topk=tree["topk"], mask=keep[0].ctypes.data,
              pos=keep[1].ctypes.data, tree_idx=keep[2].ctypes.data, parent=keep[3].ctypes.data,
              retrieve=keep[4].ctypes.data)
    return t, keep


def tree_pass(model: Model, tokens, tree, L, k_cache, v_cache, want_logits=True):
    """One backbone pass over the tree tokens.  caches: float64 [N_L][H][L_max][D].
    -> dict(logits [T][V], hidden [T][d], tree_k, tree_v [N_L][T][Hkv][D]) float64"""
    c = model.cfg
    tokens = _i32(tokens)
    T = tokens.size
    L_max = k_cache.shape[2]
    assert k_cache.dtype == np.float64 and k_cache.flags.c_contiguous
    assert v_cache.dtype == np.float64 and v_cache.flags.c_contiguous
    tk = np.zeros((c["n_layers"], T, model.kv_heads, c["head_dim"]), dtype=np.float64)
    tv = np.zeros_like(tk)
    hidden = np.zeros((T, c["d"]), dtype=np.float64)
    logits = np.zeros((T, c["vocab"]), dtype=np.float64) if want_logits else None
    mask = np.ascontiguousarray(tree["mask"], dtype=np.uint64)
    lib().ora_tree_pass(C.byref(model.c), _p(tokens), _p(mask), _p(_i32(tree["pos"])), C.c_int32(T), C.c_int32(int(L)),
                        C.c_int32(L_max), _p(k_cache), _p(v_cache), _p(tk), _p(tv), _p(hidden), _p(logits))
    return dict(logits=logits, hidden=hidden, tree_k=tk, tree_v=tv)


def layer(model: Model, l, x_in, tree, L, k_cache_l, v_cache_l, kv_bf16=False):
    """Layer l alone on a given layer input x_in [T][d]; k_cache_l, v_cache_l: THIS layer's cache, float64
    [Hkv][L_max][D].  kv_bf16: the tree keys/values are held as a bfloat16 cache holds them.
    -> dict(x_out [T][d], att [T][H*D], tree_k, tree_v [T][Hkv][D]) float64"""
    c = model.cfg
    x = np.array(x_in, dtype=np.float64, order="C")
    T = x.shape[0]
    L_max = k_cache_l.shape[1]
    assert k_cache_l.dtype == np.float64 and k_cache_l.flags.c_contiguous
    assert v_cache_l.dtype == np.float64 and v_cache_l.flags.c_contiguous
    tk = np.zeros((T, model.kv_heads, c["head_dim"]), dtype=np.float64)
    tv = np.zeros_like(tk)
    att = np.zeros((T, c["n_heads"] * c["head_dim"]), dtype=np.float64)
    mask = np.ascontiguousarray(tree["mask"], dtype=np.uint64)
    lib().ora_layer(C.byref(model.c), C.c_int32(int(l)), _p(x), _p(mask), _p(_i32(tree["pos"])), C.c_int32(T),
                    C.c_int32(int(L)), C.c_int32(L_max), _p(k_cache_l), _p(v_cache_l), _p(tk), _p(tv),
                    C.c_int32(1 if kv_bf16 else 0), _p(att))
    return dict(x_out=x, att=att, tree_k=tk, tree_v=tv)


def final_norm_lm_head(model: Model, x=None, hidden_in=None, want_logits=True):
    """hidden = final RMSNorm(x) (if x is given); logits = LM head of hidden_in if given, else of that hidden."""
    c = model.cfg
    src = x if x is not None else hidden_in
    T = np.asarray(src).shape[0]
    xx = None if x is None else _f64(x)
    hi = None if hidden_in is None else _f64(hidden_in)
    hidden = np.zeros((T, c["d"]), dtype=np.float64) if x is not None else None
    logits = np.zeros((T, c["vocab"]), dtype=np.float64) if want_logits else None
    lib().ora_final_norm_lm_head(C.byref(model.c), _p(xx), _p(hi), C.c_int32(T), _p(hidden), _p(logits))
    return dict(hidden=hidden, logits=logits)


# ----------------------------------------------------------------------------- acceptance / commit

GREEDY, TYPICAL, REJECTION = 0, 1, 2


def evaluate_posterior(logits_f32, tree_tok, tree, mode=GREEDY, tau=0.0, eps=0.09, delta=0.3, gumbel=None, uniform=None):
    """Acceptance of one step.  mode REJECTION (needs tau > 0, gumbel [V] and uniform [T]) also returns `rejected`, the
    tokens struck out at the last accepted node."""
    lg = _f32(logits_f32)
    T, V = lg.shape
    tok = _i32(tree_tok)
    if tok.size and (tok.min() < 0 or tok.max() >= V):
        raise ValueError("tree token outside the vocabulary [0, %d)" % V)
    W = tree["depth"] + 1
    if mode == REJECTION:
        if not tau > 0.0 or gumbel is None or uniform is None:
            raise ValueError("rejection sampling needs a temperature above zero, a Gumbel row and one uniform per node")
        g, u = _f32(gumbel), _f32(uniform)
        if g.size != V or u.size != tree["T"]:
            raise ValueError("gumbel must have V entries and uniform T")
        best, alen, nroot, nrej, margin = C.c_int32(), C.c_int32(), C.c_int32(), C.c_int32(), C.c_double()
        acc = np.full(W, -1, dtype=np.int32)
        rej = np.full(tree["T"], -1, dtype=np.int32)
        par, ret = _i32(tree["parent"]), _i32(tree["retrieve"])
        lib().ora_evaluate_rejection(_p(lg), C.c_int32(V), _p(tok), _p(par), C.c_int32(tree["T"]),
                                     _p(ret), C.c_int32(tree["P"]), C.c_int32(tree["depth"]),
                                     C.c_double(tau), _p(g), _p(u), C.byref(best), C.byref(alen), C.byref(nroot), _p(acc),
                                     _p(rej), C.byref(nrej), C.byref(margin))
        return dict(best=best.value, accept_len=alen.value, next_root=nroot.value, acc_nodes=acc,
                    min_margin=margin.value, rejected=rej[:nrej.value].copy())
    best = C.c_int32()
    alen = C.c_int32()
    nroot = C.c_int32()
    margin = C.c_double()
    acc = np.full(W, -1, dtype=np.int32)
    g = None if gumbel is None else _f32(gumbel)
    lib().ora_evaluate_posterior(_p(lg), C.c_int32(V), _p(_i32(tree_tok)), _p(_i32(tree["retrieve"])),
                                 C.c_int32(tree["P"]), C.c_int32(tree["depth"]), C.c_int32(mode), C.c_double(tau),
                                 C.c_double(eps), C.c_double(delta), _p(g), C.byref(best), C.byref(alen),
                                 C.byref(nroot), _p(acc), C.byref(margin))
    return dict(best=best.value, accept_len=alen.value, next_root=nroot.value, acc_nodes=acc,
                min_margin=margin.value)


def typical_decision(row_f32, token, tau, eps, delta):
    """One typical-acceptance decision on one logits row -> dict(ok, p, H, threshold) (the oracle's own numbers)."""
    row = _f32(row_f32)
    pc, ent, thr = C.c_double(), C.c_double(), C.c_double()
    fn = lib().ora_typical_decision
    fn.restype = C.c_int32
    ok = fn(_p(row), C.c_int32(row.size), C.c_double(tau), C.c_double(eps), C.c_double(delta), C.c_int32(int(token)),
            C.byref(pc), C.byref(ent), C.byref(thr))
    return dict(ok=bool(ok), p=pc.value, H=ent.value, threshold=thr.value)


def accept_and_update_kv(tree_k, tree_v, k_cache, v_cache, acc_nodes, accept_len, max_commit, L, hidden, tree_tok):
    """In-place on the float64 caches.  -> dict(L, h_last, emitted, moved_src, moved_dst)"""
    NL, T, H, D = tree_k.shape
    L_max = k_cache.shape[2]
    d = hidden.shape[1]
    W = len(acc_nodes)
    n_max = max(W, max_commit, 1)
    h_last = np.zeros(d, dtype=np.float64)
    emitted = np.full(n_max, -1, dtype=np.int32)
    src = np.full(n_max, -1, dtype=np.int32)
    dst = np.full(n_max, -1, dtype=np.int32)
    n_em = C.c_int32()
    tree_k, tree_v, hidden = _f64(tree_k), _f64(tree_v), _f64(hidden)
    assert k_cache.dtype == np.float64 and k_cache.flags.c_contiguous
    newL = lib().ora_accept_and_update_kv(
        C.c_int32(NL), C.c_int32(H), C.c_int32(D), C.c_int32(T), C.c_int32(L_max), _p(tree_k), _p(tree_v),
        _p(k_cache), _p(v_cache), _p(_i32(acc_nodes)), C.c_int32(int(accept_len)), C.c_int32(int(max_commit)),
        C.c_int32(int(L)), _p(hidden), C.c_int32(d), _p(h_last), _p(_i32(tree_tok)), _p(emitted), C.byref(n_em),
        _p(src), _p(dst))
    n = n_em.value if newL >= 0 else 0
    return dict(L=newL, h_last=h_last, emitted=emitted[:n], moved_src=src[:n], moved_dst=dst[:n])


# ----------------------------------------------------------------------------- drivers

def generate(model: Model, tree, prompt, G, L_max, mode=GREEDY, tau=0.0, eps=0.09, delta=0.3, gumbel=None,
             return_cache=False):
    prompt = _i32(prompt)
    out = np.zeros(G, dtype=np.int32)
    hist = np.zeros(G, dtype=np.int32)
    ct, keep = _ctree(tree)
    kc = vc = None
    if return_cache:
        kc = np.zeros(model.cache_shape(L_max), dtype=np.float64)
        vc = np.zeros_like(kc)
    g = None if gumbel is None else _f32(gumbel)
    lib().ora_generate.restype = C.c_int32
    steps = lib().ora_generate(C.byref(model.c), C.byref(ct), _p(prompt), C.c_int32(prompt.size), C.c_int32(G),
                               C.c_int32(L_max), C.c_int32(mode), C.c_double(tau), C.c_double(eps), C.c_double(delta),
                               _p(g), _p(out), _p(hist), _p(kc), _p(vc))
    del keep
    return dict(tokens=out, steps=steps, emitted_per_step=hist[:steps], k_cache=kc, v_cache=vc)


def generate_plain(model: Model, prompt, G, L_max, return_cache=False):
    prompt = _i32(prompt)
    out = np.zeros(G, dtype=np.int32)
    kc = vc = None
    if return_cache:
        kc = np.zeros(model.cache_shape(L_max), dtype=np.float64)
        vc = np.zeros_like(kc)
    L = lib().ora_generate_plain(C.byref(model.c), _p(prompt), C.c_int32(prompt.size), C.c_int32(G), C.c_int32(L_max),
                                 _p(out), _p(kc), _p(vc))
    return dict(tokens=out, L=L, k_cache=kc, v_cache=vc)


# ----------------------------------------------------------------------------- building blocks (for the pins)

def silu(u):
    return lib().ora_silu(float(u))


def rope(v, pos, theta=1e4):
    v = _f64(v).copy()
    lib().ora_rope(_p(v), C.c_int32(v.size), C.c_int64(int(pos)), C.c_double(theta))
    return v


def rmsnorm(x, g, eps=1e-5):
    x = _f64(x)
    g = _f32(g)
    y = np.zeros_like(x)
    lib().ora_rmsnorm(_p(x), _p(g), C.c_int32(x.size), C.c_double(eps), _p(y))
    return y


# the training objective of the heads (Sec. 2.2.1, Eq. 1) is written out in numpy in a module of its own
from .medusa1_training import medusa1_loss_and_grads  # noqa: E402,F401
