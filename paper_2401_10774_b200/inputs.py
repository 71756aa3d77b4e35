"""Seeded synthetic inputs shared by the tests, the benchmark and the smoke check.

This module holds none of the method's arithmetic: it only draws random numbers, rounds them to the
storage type and names the model shapes.  Both the CUDA library and the CPU oracle are fed the arrays
made here.  Everything is drawn from numpy's counter-based Philox generator keyed by (seed, stream), so
each tensor can be regenerated independently and in parallel.
"""
from __future__ import annotations

import zlib
from concurrent.futures import ThreadPoolExecutor

import numpy as np

# ----------------------------------------------------------------------------- shapes

MODEL_SHAPES = {
    # tiny fp32 reference model (2-layer Llama-style decoder, 2 Medusa heads)
    "tiny": dict(n_layers=2, d=256, n_heads=4, head_dim=64, ffn=688, vocab=1024, n_medusa=2,
                 rms_eps=1e-5, rope_theta=1e4),
    # Llama-7B shape, 4 Medusa heads
    "7b": dict(n_layers=32, d=4096, n_heads=32, head_dim=128, ffn=11008, vocab=32000, n_medusa=4,
               rms_eps=1e-5, rope_theta=1e4),
    # Llama-13B shape, 5 Medusa heads
    "13b": dict(n_layers=40, d=5120, n_heads=40, head_dim=128, ffn=13824, vocab=32000, n_medusa=5,
                rms_eps=1e-5, rope_theta=1e4),
    # Mistral-7B shape (the backbone of the paper's Zephyr-7B model): grouped-query attention, 8 key/value heads
    # for 32 query heads; its 4096-token sliding window never cuts a cache of at most 4096 positions
    "mistral7b": dict(n_layers=32, d=4096, n_heads=32, n_kv_heads=8, head_dim=128, ffn=14336, vocab=32000, n_medusa=5,
                      rms_eps=1e-5, rope_theta=1e4),
}


def kv_heads(cfg: dict) -> int:
    """Key/value heads of a shape: `n_kv_heads` if given and non-zero, else one per query head."""
    return cfg.get("n_kv_heads", 0) or cfg["n_heads"]

# per-depth top-k of the Cartesian tree the sparse tree is cut from, and the node budget (root included)
TREE_SPECS = {
    "dense22": dict(per_depth_topk=(2, 2), n_nodes=7),
    "sparse64_d4": dict(per_depth_topk=(4, 3, 2, 2), n_nodes=64),
    "sparse64_d5": dict(per_depth_topk=(4, 3, 2, 2, 2), n_nodes=64),
}
# Trees of more than 64 nodes (the paper's Sec. 3.3.1 / Fig. 4 studies sparse trees of up to 256 nodes): the same
# surrogate construction (score prod 1/(rank+1), best n nodes), wider per-depth top-k.
LARGE_TREE_SPECS = {
    "sparse128_d4": dict(per_depth_topk=(6, 4, 3, 2), n_nodes=128),
    "sparse256_d4": dict(per_depth_topk=(10, 6, 4, 3), n_nodes=256),
    "sparse256_d5": dict(per_depth_topk=(10, 6, 4, 3, 2), n_nodes=256),
    "sparse100_d3": dict(per_depth_topk=(7, 5, 3), n_nodes=100),
}


def model_shape(name: str, **override) -> dict:
    cfg = dict(MODEL_SHAPES[name])
    cfg.update(override)
    return cfg


# ----------------------------------------------------------------------------- random streams

def _stream_id(stream) -> int:
    if isinstance(stream, int):
        return stream
    return zlib.crc32(str(stream).encode()) | (1 << 40)


def rng(seed: int, stream=0) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[int(seed), _stream_id(stream)]))


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit patterns (uint16), round to nearest even.  Inputs must be finite."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    if x.size >= (1 << 16):
        try:  # same rounding, two orders of magnitude faster on large arrays
            import torch

            return torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
        except ImportError:
            pass
    u = x.view(np.uint32)
    r = ((u >> 16) & 1) + np.uint32(0x7FFF)
    return ((u + r) >> 16).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def normal(shape, std: float, seed: int, stream, dtype: str = "f32", mean: float = 0.0) -> np.ndarray:
    """N(mean, std^2) array; dtype "f32" -> float32, "bf16" -> uint16 bit patterns of the rounded values."""
    g = rng(seed, stream)
    n = int(np.prod(shape))
    out = np.empty(n, dtype=np.float32 if dtype == "f32" else np.uint16)
    chunk = 1 << 24
    for s in range(0, n, chunk):
        e = min(n, s + chunk)
        x = g.standard_normal(e - s, dtype=np.float32)
        if std != 1.0:
            x *= np.float32(std)
        if mean != 0.0:
            x += np.float32(mean)
        out[s:e] = x if dtype == "f32" else to_bf16_bits(x)
    return out.reshape(shape)


def as_f32(a: np.ndarray) -> np.ndarray:
    """Exact float32 view of the stored values (widens bf16 bit patterns)."""
    return bf16_bits_to_f32(a) if a.dtype == np.uint16 else np.ascontiguousarray(a, dtype=np.float32)


# ----------------------------------------------------------------------------- model weights

LAYER_KEYS = ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "w_gate", "w_up", "w_down")


def make_weights(cfg: dict, seed: int, dtype: str = "f32", std: float = 0.02, gain_std: float = 0.0,
                 head_init: str = "normal", head_noise: float = 0.002, threads: int = 8) -> dict:
    """Random-init weights of a Llama-style decoder plus K Medusa heads.

    Every matrix and the embedding ~ N(0, std^2); norm gains = 1 (+ N(0, gain_std^2) if asked);
    head_init "normal": W1_k, W2_k ~ N(0, std^2);  "lm_copy": W1_k ~ N(0, std^2), W2_k = LM head + N(0, head_noise^2).
    All matrices are stored [out][in].  dtype "bf16" stores uint16 bit patterns.
    """
    d, F, V, K = cfg["d"], cfg["ffn"], cfg["vocab"], cfg["n_medusa"]
    hd = cfg["n_heads"] * cfg["head_dim"]
    hkd = kv_heads(cfg) * cfg["head_dim"]
    jobs = {}

    def mat(name, shape):
        jobs[name] = lambda: normal(shape, std, seed, name, dtype)

    def gain(name):
        jobs[name] = lambda: normal((d,), gain_std, seed, name, dtype, mean=1.0)

    mat("embed", (V, d))
    mat("lm_head", (V, d))
    gain("final_norm")
    for l in range(cfg["n_layers"]):
        gain("l%d.attn_norm" % l)
        mat("l%d.wq" % l, (hd, d))
        mat("l%d.wk" % l, (hkd, d))
        mat("l%d.wv" % l, (hkd, d))
        mat("l%d.wo" % l, (d, hd))
        gain("l%d.ffn_norm" % l)
        mat("l%d.w_gate" % l, (F, d))
        mat("l%d.w_up" % l, (F, d))
        mat("l%d.w_down" % l, (d, F))
    for k in range(K):
        mat("medusa%d.w1" % k, (d, d))
        if head_init == "normal":
            mat("medusa%d.w2" % k, (V, d))
    with ThreadPoolExecutor(max_workers=threads) as ex:
        futs = {name: ex.submit(fn) for name, fn in jobs.items()}
        res = {name: f.result() for name, f in futs.items()}
    if head_init == "lm_copy":
        lm = as_f32(res["lm_head"])
        for k in range(K):
            w2 = lm + normal((V, d), head_noise, seed, "medusa%d.w2noise" % k, "f32")
            res["medusa%d.w2" % k] = w2 if dtype == "f32" else to_bf16_bits(w2)
    elif head_init != "normal":
        raise ValueError(head_init)
    w = dict(embed=res["embed"], lm_head=res["lm_head"], final_norm=res["final_norm"], layers=[])
    for l in range(cfg["n_layers"]):
        w["layers"].append({k: res["l%d.%s" % (l, k)] for k in LAYER_KEYS})
    if K:
        w["medusa_w1"] = np.stack([res["medusa%d.w1" % k] for k in range(K)])
        w["medusa_w2"] = np.stack([res["medusa%d.w2" % k] for k in range(K)])
    else:
        w["medusa_w1"] = w["medusa_w2"] = None
    return w


def make_prompt(n: int, vocab: int, seed: int) -> np.ndarray:
    return rng(seed, "prompt").integers(0, vocab, size=n, dtype=np.int64).astype(np.int32)


# ----------------------------------------------------------------------------- operator inputs

def attention_inputs(T: int, H: int, D: int, L: int, L_max: int, seed: int, dtype: str = "bf16", Hkv: int = 0) -> dict:
    """q [T][H][D], k_new, v_new [T][Hkv][D] and caches [Hkv][L_max][D] (Hkv = H unless given), all N(0,1);
    cache rows >= L are zero."""
    Hkv = Hkv or H
    out = {"q": normal((T, H, D), 1.0, seed, "q", dtype)}
    for name in ("k_new", "v_new"):
        out[name] = normal((T, Hkv, D), 1.0, seed, name, dtype)
    for name in ("k_cache", "v_cache"):
        c = np.zeros((Hkv, L_max, D), dtype=np.float32 if dtype == "f32" else np.uint16)
        if L:
            c[:, :L, :] = normal((Hkv, L, D), 1.0, seed, name, dtype)
        out[name] = c
    return out


def heads_inputs(d: int, V: int, K: int, seed: int, dtype: str = "bf16", std: float = 0.02) -> dict:
    """h ~ N(0,1) (a normalised hidden state has unit RMS), W1 [K][d][d], W2 [K][V][d] ~ N(0, std^2), root token."""
    return dict(
        h=normal((d,), 1.0, seed, "h", dtype),
        W1=normal((K, d, d), std, seed, "W1", dtype),
        W2=normal((K, V, d), std, seed, "W2", dtype),
        root=int(rng(seed, "root").integers(0, V)),
    )


def uniform_noise(steps: int, n: int, seed: int) -> np.ndarray:
    """Uniform numbers in [0, 1), float32 [steps][n] (one per tree node and step: the draws of rejection sampling)."""
    u = rng(seed, "uniform").random((steps, n), dtype=np.float64).astype(np.float32)
    return np.minimum(u, np.float32(0.99999994))


def gumbel_noise(steps: int, V: int, seed: int) -> np.ndarray:
    """Standard Gumbel noise -log(-log u), float32 [steps][V], for replayable sampling."""
    u = rng(seed, "gumbel").random((steps, V), dtype=np.float64)
    u = np.clip(u, 1e-300, 1.0 - 1e-16)
    return (-np.log(-np.log(u))).astype(np.float32)
