"""Algorithmic byte / flop accounting of the decode step (what the method must move; no padded tiles, no re-reads).

The same accounting style as the paper's roofline study (App. G, Table 5): each operator reads its inputs
once and writes its outputs once.  `operational_intensity_*` reproduce the paper's printed figures when
given its fp16 shapes and its unfused attention (score matrix materialised).
"""
from __future__ import annotations


def linear_bytes(T: int, N: int, K: int, w_bytes: int = 2, x_bytes: int = 2, y_bytes: int = 4) -> int:
    """One Y[T][N] = X[T][K] W[N][K]^T launch: weights once, activations in, result out."""
    return N * K * w_bytes + T * K * x_bytes + T * N * y_bytes


def linear_flops(T: int, N: int, K: int) -> int:
    return 2 * T * N * K


def attention_bytes(T: int, H: int, D: int, L: int, e: int = 2, Hkv: int = 0) -> int:
    """tree_attention, one layer: K and V cache rows 0..L-1 (Hkv key/value heads, H unless given), q and out
    (H heads), k_new and v_new (Hkv heads)."""
    Hkv = Hkv or H
    return 2 * L * Hkv * D * e + 2 * T * H * D * e + 2 * T * Hkv * D * e


def attention_flops(T: int, H: int, D: int, L: int) -> int:
    return 4 * T * H * D * (L + T)


def heads_bytes(d: int, V: int, K: int, e: int = 2) -> int:
    """medusa_heads: W1 and W2 of K heads, read once (vectors are negligible but counted)."""
    return K * (d * d + V * d) * e + K * (2 * d * 4 + V * 4)


def step_bytes(cfg: dict, T: int, L: int, K_used: int, e: int = 2) -> dict:
    """Bytes one full tree-verification step must move, by stage (bf16 weights / cache, float logits)."""
    d, F, V, H, D, NL = cfg["d"], cfg["ffn"], cfg["vocab"], cfg["n_heads"], cfg["head_dim"], cfg["n_layers"]
    HD = H * D
    HkvD = (cfg.get("n_kv_heads", 0) or H) * D  # key/value heads: fewer than H with grouped-query attention
    gemm_w = NL * ((HD + 2 * HkvD) * d + d * HD + 2 * F * d + d * F) * e + V * d * e
    out = dict(
        gemm_weights=gemm_w,
        heads=K_used * (d * d + V * d) * e,
        kv_read=NL * 2 * L * HkvD * e,
        tree_kv_write=NL * 2 * T * HkvD * e,
        logits_write_read=2 * T * V * 4,
        commit=NL * 2 * 2 * (cfg.get("depth", 4) + 1) * HkvD * e,
    )
    out["total"] = sum(out.values())
    return out


def gemm_launch_bytes_per_step(cfg: dict, T: int, planes: int = 2) -> int:
    """Sum of linear_bytes over the GEMM launches of one tree pass (split activations count both planes)."""
    d, F, V, H, D, NL = cfg["d"], cfg["ffn"], cfg["vocab"], cfg["n_heads"], cfg["head_dim"], cfg["n_layers"]
    HD = H * D
    HkvD = (cfg.get("n_kv_heads", 0) or H) * D
    xb = 2 * planes
    per_layer = (linear_bytes(T, HD, d, 2, xb) + 2 * linear_bytes(T, HkvD, d, 2, xb) + linear_bytes(T, d, HD, 2, xb)
                 + 2 * linear_bytes(T, F, d, 2, xb) + linear_bytes(T, d, F, 2, xb))
    return NL * per_layer + linear_bytes(T, V, d, 2, xb)


# ---- the paper's own accounting (App. G Table 5), used to pin this module against its printed tables ----

def operational_intensity_attention_unfused(s: int, q: int, d: int, e: int = 2) -> float:
    """QK^T and PV per head with the score matrix written and read: flops 4*s*q*d, bytes e*2*(q*d + s*d + s*q)."""
    return (4.0 * s * q * d) / (e * 2.0 * (q * d + s * d + s * q))


def operational_intensity_linear(q: int, h: int, i: int, e: int = 2) -> float:
    """One up/gate/down linear on q tokens: flops 2*q*h*i, bytes e*(h*i + q*(h+i))."""
    return (2.0 * q * h * i) / (e * (h * i + q * (h + i)))


def hbm_peak_gbs():
    """(GB/s, source): the measured STREAM-style copy bandwidth recorded beside the package, else the fallback."""
    import json
    import os

    p = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "MEASURED_PEAKS.json")
    if os.path.exists(p):
        return float(json.load(open(p))["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def tensor_peak_tflops():
    """(TFLOP/s, source): the measured dense bf16 throughput (a burst of a library GEMM) recorded beside the package, else
    the fallback."""
    import json
    import os

    p = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "MEASURED_PEAKS.json")
    if os.path.exists(p):
        return float(json.load(open(p))["bf16_tflops"]), "measured"
    return 1590.0, "fallback"


# ---- DRAM traffic taken from profiler captures ----
# A capture describes the kernel source it was taken from: the figure is reported only while the SHA-256 of that
# source file still equals the one recorded with the capture, so a changed kernel never inherits an old number.
# bytes = dram__bytes_read.sum + dram__bytes_write.sum per launch, the launch-weighted mean over one step's launches
# (the four layer shapes captured on a 2-layer model of the same width: a layer's traffic does not depend on the
# depth; the LM head's figure is its weights plus the logits).
CAPTURED_TRAFFIC = {
    # (kernel, model): (bytes per launch, source file, sha256 of that file at capture time)
    ("gemm_tc_kernel", "7b"): (104.7e6, "csrc/gemm_tc.cu", "d371a33e5f1094de73990377575a87e12406dff52e9c6ee929cd7b7f5c87c7f7"),
}


def captured_traffic(kernel: str, model: str):
    """-> (bytes per launch or None, note)"""
    import hashlib
    import os

    rec = CAPTURED_TRAFFIC.get((kernel, model))
    if rec is None:
        return None, "no profiler capture of %s at the %s shape" % (kernel, model)
    nbytes, rel, sha = rec
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), rel)
    try:
        now = hashlib.sha256(open(path, "rb").read()).hexdigest()
    except OSError:
        return None, "kernel source %s not found" % rel
    if now != sha:
        return None, "the profiler capture of %s is older than its source (%s changed since): not reported" % (kernel, rel)
    return nbytes, "profiler capture of %s taken from the current %s" % (kernel, rel)
