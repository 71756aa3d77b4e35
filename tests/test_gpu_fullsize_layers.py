"""Full-width parity of the backbone on ALL 64 tree rows at the flat tolerances (2e-2 for attention outputs and
normalised hidden states, 5e-2 for logits), layer by layer at full depth.

Through N_L layers the end-to-end error of any bf16 implementation grows like sqrt(N_L) (the bf16 KV cache alone
injects an independent rounding error per layer), so a flat end-to-end bound cannot hold at 32 or 40 layers.  What
can and must hold is the flat bound for EVERY layer on that layer's own input: the GPU's residual stream entering
layer l and the GPU's cache of layer l are handed to the oracle's single-layer function ("teacher forcing"), and
that layer's attention output, its keys/values, and the normalised residual stream it leaves are compared on all 64
rows.  The oracle holds the tree keys/values as a bfloat16 cache holds them: that rounding is the workload's storage
format, not kernel arithmetic.  The end-to-end figure is printed as a report.
"""
import numpy as np
import pytest

from paper_2401_10774_b200 import inputs as I

pytestmark = pytest.mark.gpu

TOL_HIDDEN_BF16 = 2e-2
TOL_LOGIT_BF16 = 5e-2
TOL_KV_BF16 = 5e-2  # keys reach |k| ~ 6, where one bfloat16 step is 3.1e-2: a rounding tie may land one step apart


def _gpu():
    import torch
    from paper_2401_10774_b200 import binding as B
    from tests import gpu_util as U
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    return torch, B, U


def _planes(ctx, B, which, rows, width):
    """A split activation [2][64][width] (bf16 planes hi, lo) as the float values hi + lo of the first `rows` rows."""
    p = I.bf16_bits_to_f32(ctx.read_workspace(which, (2, 64, width), np.uint16))
    return (p[0].astype(np.float64) + p[1].astype(np.float64))[:rows]


# the last field picks the attention kernel inside the pass: 0 the library's default (the mma.sync kernel at this cache
# length), 2 the tcgen05 kernel forced (the default from 1536 cached keys on).  Both take q as two bfloat16 planes and are
# held to the same flat bounds.
# (the sixth field is the prompt length: 520 = eight full prefill passes and a ragged one, the cache tiles end ragged too;
# 1600 = past the 1536 keys from which the library itself picks the tcgen05 kernel inside a pass)
CASES = [("7b", 32, "sparse64_d4", (0, 15, 31), 0, 520), ("13b", 40, "sparse64_d5", (0, 39), 0, 520),
         ("7b", 1, "sparse64_d4", (0,), 0, 520), ("13b", 1, "sparse64_d5", (0,), 0, 520), ("7b", 1, "sparse64_d4", (0,), 2, 520),
         ("13b", 1, "sparse64_d5", (0,), 2, 520), ("13b", 1, "sparse64_d5", (0,), 0, 1600)]


def _case_id(c):
    return "%s_%dlayers%s%s" % (c[0], c[1], "_tcgen05_attention" if c[4] == 2 else "", "_L%d" % c[5] if c[5] != 520 else "")


@pytest.mark.parametrize("shape,n_layers,tree_name,tap_layers,attn_kernel,n_prompt", CASES, ids=[_case_id(c) for c in CASES])
def test_every_row_of_a_layer_at_the_flat_tolerance(oracle, shape, n_layers, tree_name, tap_layers, attn_kernel, n_prompt):
    torch, B, U = _gpu()
    tol_hidden = TOL_HIDDEN_BF16
    cfg = I.model_shape(shape, n_layers=n_layers)
    L_max = 4096
    w = I.make_weights(cfg, seed=40, dtype="bf16")
    ctx = U.make_ctx(cfg, "bf16", L_max, I.TREE_SPECS[tree_name])
    ctx.load_weights(U.dev_weights(w))
    if attn_kernel:
        ctx.set_option(B.OPT_ATTENTION_KERNEL, attn_kernel)
    om = oracle.Model(cfg, w, kv_bf16=True)
    ot = oracle.build_tree_buffers(oracle.default_tree_paths(**I.TREE_SPECS[tree_name]))
    d, V, T = cfg["d"], cfg["vocab"], ot["T"]
    H, Hkv, D = cfg["n_heads"], I.kv_heads(cfg), cfg["head_dim"]
    prompt = I.make_prompt(n_prompt, V, 41)
    ctx.prefill(torch.from_numpy(prompt).cuda())
    assert ctx.state()["cache_len"] == n_prompt
    tok = I.rng(5, "treetok").integers(0, V, size=T).astype(np.int32)
    tok_dev = torch.from_numpy(tok).cuda()
    report = []
    for l in tap_layers:
        ctx.set_option(B.OPT_LAYER_TAP, l)
        ctx.tree_pass(tok_dev)
        assert ctx.device_status() == 0
        x_in = ctx.read_workspace(B.WS_TAP_X_IN, (64, d), np.float32)[:T]
        x_out = ctx.read_workspace(B.WS_TAP_X_OUT, (64, d), np.float32)[:T]
        att = _planes(ctx, B, B.WS_TAP_ATT, T, H * D)
        xn_out = _planes(ctx, B, B.WS_TAP_XN_OUT, T, d)
        off = l * Hkv * L_max * D
        kc = I.bf16_bits_to_f32(ctx.read_workspace(B.WS_K_CACHE, (Hkv, L_max, D), np.uint16, offset_elems=off))[:, :n_prompt]
        vc = I.bf16_bits_to_f32(ctx.read_workspace(B.WS_V_CACHE, (Hkv, L_max, D), np.uint16, offset_elems=off))[:, :n_prompt]
        tk = I.bf16_bits_to_f32(ctx.read_workspace(B.WS_TREE_K, (64, Hkv, D), np.uint16, offset_elems=l * 64 * Hkv * D))[:T]
        tv = I.bf16_bits_to_f32(ctx.read_workspace(B.WS_TREE_V, (64, Hkv, D), np.uint16, offset_elems=l * 64 * Hkv * D))[:T]
        ref = oracle.layer(om, l, x_in, ot, n_prompt, np.ascontiguousarray(kc, dtype=np.float64),
                           np.ascontiguousarray(vc, dtype=np.float64), kv_bf16=True)
        gain = w["layers"][l + 1]["attn_norm"] if l + 1 < n_layers else w["final_norm"]
        xn_ref = np.stack([oracle.rmsnorm(ref["x_out"][t], I.as_f32(gain), cfg.get("rms_eps", 1e-5)) for t in range(T)])
        e_att = float(np.abs(att - ref["att"]).max())
        e_xn = float(np.abs(xn_out - xn_ref).max())
        e_k = float(np.abs(tk - ref["tree_k"]).max())
        e_v = float(np.abs(tv - ref["tree_v"]).max())
        # the residual stream itself, relative to its own scale (reported; the normalised form above is the criterion)
        e_x_rel = float(np.abs(x_out - ref["x_out"]).max() / np.sqrt(np.mean(ref["x_out"] ** 2)))
        report.append((l, e_att, e_xn, e_k, e_v, e_x_rel))
        assert e_att <= tol_hidden, "layer %d: attention output max |err| %.3g on 64 rows" % (l, e_att)
        assert e_xn <= tol_hidden, "layer %d: normalised hidden max |err| %.3g on 64 rows" % (l, e_xn)
        assert e_k <= TOL_KV_BF16 and e_v <= TOL_KV_BF16, "layer %d: tree K/V max |err| %.3g / %.3g" % (l, e_k, e_v)
    # the closing stage on the GPU's own final hidden state: every logit of every row
    hid = ctx.read_workspace(B.WS_HIDDEN, (T, d), np.float32)
    lg = ctx.read_workspace(B.WS_LOGITS, (T, V), np.float32)
    lg_ref = oracle.final_norm_lm_head(om, hidden_in=hid)["logits"]
    e_lg = float(np.abs(lg - lg_ref).max())
    assert e_lg <= TOL_LOGIT_BF16, "logits max |err| %.3g on 64 rows" % e_lg
    ctx.set_option(B.OPT_LAYER_TAP, -1)
    line = "%s width, %d layers, all %d rows, L=%d, attention kernel %d: " % (shape, n_layers, T, n_prompt, attn_kernel)
    line += "; ".join("layer %d att %.3g norm-hidden %.3g K %.3g V %.3g x(rel) %.3g" % r for r in report)
    line += "; logits on the GPU's hidden %.3g" % e_lg
    if n_layers == 1:
        # one layer deep the whole pass is within the flat tolerances against the oracle's own pass on its own cache
        kc0 = np.zeros(om.cache_shape(n_prompt + 8))
        vc0 = np.zeros_like(kc0)
        L = 0
        while L < n_prompt:
            n = min(64, n_prompt - L)
            last = oracle.tree_pass(om, prompt[L:L + n], oracle.chain_tree(n), L, kc0, vc0, want_logits=False)
            oracle.accept_and_update_kv(last["tree_k"], last["tree_v"], kc0, vc0, np.arange(n), n - 1, n, L, last["hidden"],
                                        prompt[L:L + n])
            L += n
        full = oracle.tree_pass(om, tok, ot, n_prompt, kc0, vc0)
        e_h, e_l = float(np.abs(hid - full["hidden"]).max()), float(np.abs(lg - full["logits"]).max())
        line += "; end to end vs the oracle's own pass: hidden %.3g logits %.3g" % (e_h, e_l)
        assert e_h <= tol_hidden and e_l <= TOL_LOGIT_BF16, line
    print(line)
    ctx.close()
