"""Trees of more than 64 nodes (paper Sec. 3.3.1, Fig. 4: sparse trees of up to 256 nodes) on the GPU against the oracle:
ancestor masks of several 64-bit words, projections and attention run in tiles of 64 token rows."""
import numpy as np
import pytest

from paper_2401_10774_b200 import inputs as I

pytestmark = pytest.mark.gpu

TOL_ATTN_BF16 = 2e-2
TOL_HIDDEN_BF16 = 2e-2
TOL_LOGIT_BF16 = 5e-2
TOL_F32 = 5e-4


def _gpu():
    import torch
    from paper_2401_10774_b200 import binding as B
    from tests import gpu_util as U
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    return torch, B, U


def _spec(name):
    return I.LARGE_TREE_SPECS[name] if name in I.LARGE_TREE_SPECS else I.TREE_SPECS[name]


ATT_CASES = [
    # dtype, H, D, L, L_max, tree, key/value heads
    ("bf16", 4, 128, 0, 64, "sparse128_d4", 0),        # tree keys only, two query tiles
    ("bf16", 4, 128, 100, 128, "sparse256_d5", 0),     # short cache (one key range), four query tiles
    ("bf16", 8, 128, 1000, 1024, "sparse256_d4", 2),   # several key ranges, grouped-query attention
    ("bf16", 32, 128, 2100, 2176, "sparse100_d3", 0),  # ragged: 100 nodes = one full and one partial query tile
    ("f32", 3, 64, 37, 48, "sparse128_d4", 0),         # the generic kernel
    ("bf16", 3, 64, 333, 512, "sparse256_d5", 0),      # generic kernel, bf16, head dim 64
]


@pytest.mark.parametrize("case", ATT_CASES, ids=["%s_H%d_D%d_L%d_%s" % (c[0], c[1], c[2], c[3], c[5]) for c in ATT_CASES])
def test_large_tree_attention_parity(oracle, case):
    torch, B, U = _gpu()
    dt, H, D, L, L_max, tree_name, Hkv = case
    spec = _spec(tree_name)
    cfg = dict(n_layers=0, d=H * D, n_heads=H, n_kv_heads=Hkv, head_dim=D, ffn=8, vocab=8, n_medusa=5,
               max_tree_nodes=spec["n_nodes"])
    ctx = U.make_ctx(cfg, dt, L_max, spec)
    t = ctx.tree
    T = t["T"]
    assert T == spec["n_nodes"]
    a = I.attention_inputs(T, H, D, L, L_max, 25, dtype=dt, Hkv=Hkv)
    dev = {k: U.to_dev(v) for k, v in a.items()}
    out = U.empty_act((T, H, D), ctx.dtype)
    lse = torch.zeros((T, H), dtype=torch.float32, device="cuda")
    cache_len = torch.tensor([L], dtype=torch.int32, device="cuda")
    ctx.tree_attention(dev["q"], dev["k_new"], dev["v_new"], dev["k_cache"], dev["v_cache"], cache_len, True, out, lse)
    torch.cuda.synchronize()
    ot = oracle.build_tree_buffers(oracle.default_tree_paths(**spec))
    assert np.array_equal(np.asarray(t["mask"]), np.asarray(ot["mask"]))
    ref, ref_lse = oracle.tree_attention(*(I.as_f32(a[k]) for k in ("q", "k_new", "v_new", "k_cache", "v_cache")), L,
                                         ot["mask"], ot["pos"], apply_rope=True)
    tol = TOL_ATTN_BF16 if dt == "bf16" else 2e-4
    err = np.abs(U.to_host_f32(out) - ref).max()
    assert err <= tol, "max |err| %.3g > %.3g" % (err, tol)
    assert np.abs(U.to_host_f32(lse) - ref_lse).max() <= (5e-2 if dt == "bf16" else 1e-3)
    assert ctx.device_status() == 0
    ctx.close()


def test_a_tree_larger_than_the_context_was_created_for_is_refused():
    torch, B, U = _gpu()
    cfg = dict(n_layers=0, d=256, n_heads=2, head_dim=128, ffn=8, vocab=8, n_medusa=5)  # max_tree_nodes not given: 64
    ctx = B.Context(cfg, B.BF16, 64)
    with pytest.raises(B.MedusaError) as e:
        ctx.build_tree_buffers(B.default_tree_paths(**_spec("sparse128_d4")))
    assert e.value.code == B.ERR_SHAPE
    ctx.build_tree_buffers(B.default_tree_paths(**_spec("sparse64_d4")))
    ctx.close()
    with pytest.raises(B.MedusaError) as e:
        B.Context(dict(cfg, max_tree_nodes=257), B.BF16, 64)
    assert e.value.code == B.ERR_SHAPE


PASS_CASES = [
    ("tiny_f32_100nodes", dict(n_medusa=3), "f32", "sparse100_d3", 40, TOL_F32, TOL_F32),
    ("small_bf16_128nodes", dict(d=512, n_heads=4, head_dim=128, ffn=1408, vocab=2048, n_medusa=4, n_layers=3), "bf16",
     "sparse128_d4", 70, TOL_HIDDEN_BF16, TOL_LOGIT_BF16),
    ("small_bf16_256nodes_gqa", dict(d=512, n_heads=4, n_kv_heads=2, head_dim=128, ffn=1408, vocab=2048, n_medusa=5, n_layers=2),
     "bf16", "sparse256_d5", 150, TOL_HIDDEN_BF16, TOL_LOGIT_BF16),
]


@pytest.mark.parametrize("case", PASS_CASES, ids=[c[0] for c in PASS_CASES])
def test_large_tree_pass_parity(oracle, case):
    torch, B, U = _gpu()
    name, over, dt, tree_name, n_prompt, tol_h, tol_l = case
    spec = _spec(tree_name)
    cfg = I.model_shape("tiny", max_tree_nodes=spec["n_nodes"], **over)
    L_max = 512
    w = I.make_weights(cfg, seed=3, dtype=dt, gain_std=0.1)
    ctx = U.make_ctx(cfg, dt, L_max, spec)
    ctx.load_weights(U.dev_weights(w))
    om = oracle.Model(cfg, w, kv_bf16=(dt == "bf16"))
    ot = oracle.build_tree_buffers(oracle.default_tree_paths(**spec))
    prompt = I.make_prompt(n_prompt, cfg["vocab"], 4)
    ctx.prefill(torch.from_numpy(prompt).cuda())
    assert ctx.state()["cache_len"] == n_prompt
    kc = np.zeros(om.cache_shape(L_max))
    vc = np.zeros_like(kc)
    L = 0
    while L < n_prompt:
        n = min(64, n_prompt - L)
        last = oracle.tree_pass(om, prompt[L:L + n], oracle.chain_tree(n), L, kc, vc, want_logits=False)
        oracle.accept_and_update_kv(last["tree_k"], last["tree_v"], kc, vc, np.arange(n), n - 1, n, L, last["hidden"], prompt[L:L + n])
        L += n
    T, d, V = ot["T"], cfg["d"], cfg["vocab"]
    NL, Hkv, D = cfg["n_layers"], I.kv_heads(cfg), cfg["head_dim"]
    R = 64 * ((T + 63) // 64)
    tok = I.rng(5, "treetok").integers(0, V, size=T).astype(np.int32)
    ctx.tree_pass(torch.from_numpy(tok).cuda())
    ref = oracle.tree_pass(om, tok, ot, n_prompt, kc, vc)
    hid = ctx.read_workspace(B.WS_HIDDEN, (T, d), np.float32)
    lgt = ctx.read_workspace(B.WS_LOGITS, (T, V), np.float32)
    tk = U.read_act(ctx, B.WS_TREE_K, (NL, R, Hkv, D))[:, :T]
    tv = U.read_act(ctx, B.WS_TREE_V, (NL, R, Hkv, D))[:, :T]
    eh, el = np.abs(hid - ref["hidden"]).max(), np.abs(lgt - ref["logits"]).max()
    assert eh <= tol_h, "hidden max |err| %.3g" % eh
    assert el <= tol_l, "logits max |err| %.3g" % el
    tol_kv = 5e-2 if dt == "bf16" else TOL_F32
    assert np.abs(tk - ref["tree_k"]).max() <= tol_kv and np.abs(tv - ref["tree_v"]).max() <= tol_kv
    assert ctx.device_status() == 0
    ctx.close()


def test_large_tree_greedy_decode_token_exact_on_the_tiny_model(oracle):
    # the exactness of greedy acceptance with a 100-node tree: the fp32 model's token stream equals the oracle's and
    # plain greedy decoding's
    torch, B, U = _gpu()
    spec = _spec("sparse100_d3")
    cfg = I.model_shape("tiny", n_medusa=3, max_tree_nodes=100)
    w = I.make_weights(cfg, seed=0, dtype="f32", head_init="lm_copy")
    ctx = U.make_ctx(cfg, "f32", 128, spec)
    ctx.load_weights(U.dev_weights(w))
    om = oracle.Model(cfg, w)
    ot = oracle.build_tree_buffers(oracle.default_tree_paths(**spec))
    prompt = I.make_prompt(32, cfg["vocab"], 1)
    G = 48
    got = ctx.generate(prompt, G, B.AcceptParams(mode=B.GREEDY))
    ref = oracle.generate(om, ot, prompt, G, 128, mode=oracle.GREEDY)
    plain = oracle.generate_plain(om, prompt, G, 128)
    assert ref["tokens"].tolist() == plain["tokens"].tolist()
    assert got["tokens"].tolist() == ref["tokens"].tolist()
    assert got["emitted_per_step"].tolist() == ref["emitted_per_step"].tolist()
    assert got["steps"] < G
    ctx.close()


@pytest.mark.parametrize("mode", ["greedy", "typical_gumbel", "rejection"])
def test_large_tree_bf16_decode_stagewise(oracle, mode):
    # a 256-node, depth-5 tree on the small bf16 model: integer stages bit-exact on the GPU's own tensors at every step
    torch, B, U = _gpu()
    spec = _spec("sparse256_d5")
    cfg = I.model_shape("tiny", d=512, n_heads=4, head_dim=128, ffn=1408, vocab=2048, n_medusa=5, n_layers=2, max_tree_nodes=256)
    L_max = 256
    w = I.make_weights(cfg, seed=6, dtype="bf16", head_init="lm_copy")
    ctx = U.make_ctx(cfg, "bf16", L_max, spec)
    ctx.load_weights(U.dev_weights(w))
    om = oracle.Model(cfg, w)
    ot = oracle.build_tree_buffers(oracle.default_tree_paths(**spec))
    V, d, T, K = cfg["vocab"], cfg["d"], ot["T"], ot["depth"]
    ctx.prefill(torch.from_numpy(I.make_prompt(40, V, 7)).cuda())
    tau, eps, delta = (0.0, 0.09, 0.3) if mode == "greedy" else (0.7, 0.09, 0.3)
    f32 = lambda x: float(np.float32(x))
    params = B.AcceptParams(mode=dict(greedy=B.GREEDY, rejection=B.REJECTION).get(mode, B.TYPICAL), temperature=tau, eps=eps,
                            delta=delta)
    steps = 10
    noise = I.gumbel_noise(steps, V, 52) if mode != "greedy" else None
    uni = I.uniform_noise(steps, T, 53) if mode == "rejection" else None  # one uniform per node: up to ten siblings are tried in turn
    L, multi = 40, 0
    NL, H, D = cfg["n_layers"], cfg["n_heads"], cfg["head_dim"]
    for s in range(steps):
        st0 = ctx.state()
        h_last = ctx.read_workspace(B.WS_H_LAST, (d,), np.float32)
        row = None if noise is None else (noise[s] if uni is None else np.concatenate([noise[s], uni[s]]))
        ctx.decode_step(params, None if row is None else torch.from_numpy(row).cuda(), max_commit=1 << 20)
        st = ctx.state()
        assert st["status"] == 0
        z = ctx.read_workspace(B.WS_HEAD_LOGITS, (K, V), np.float32)
        _, z_ref = oracle.medusa_heads(h_last, om.w["medusa_w1"][:K], om.w["medusa_w2"][:K])
        assert np.abs(z - z_ref).max() <= TOL_LOGIT_BF16
        ti = ctx.read_workspace(B.WS_TOPK_IDX, (K, ot["topk"]), np.int32)
        for k in range(K):
            assert ti[k].tolist() == oracle.topk(z[k], ot["topk"]).tolist()
        tok = ctx.read_workspace(B.WS_TREE_TOK, (T,), np.int32)
        assert tok.tolist() == oracle.expand_candidates(st0["root"], ti, ot)[0].tolist()
        lg = ctx.read_workspace(B.WS_LOGITS, (T, V), np.float32)
        ref = oracle.evaluate_posterior(lg, tok, ot, mode=params.mode, tau=f32(tau), eps=f32(eps), delta=f32(delta),
                                        gumbel=None if noise is None else noise[s], uniform=None if uni is None else uni[s])
        assert mode == "greedy" or ref["min_margin"] > 1e-9
        acc = ctx.read_workspace(B.WS_ACC_NODES, (K + 1,), np.int32)
        assert (st["best"], st["accept_len"], st["next_root"]) == (ref["best"], ref["accept_len"], ref["next_root"])
        assert acc.tolist() == ref["acc_nodes"].tolist()
        n = 1 + ref["accept_len"]
        assert st["cache_len"] == L + n and st["n_emitted"] == n
        tk = ctx.read_workspace(B.WS_TREE_K, (NL, 256, H, D), np.uint16)
        kc = ctx.read_workspace(B.WS_K_CACHE, (NL, H, L_max, D), np.uint16)
        for j in range(n):
            assert np.array_equal(kc[:, :, L + j], tk[:, acc[j]])
        L += n
        multi += n > 1
    assert multi > 0 or mode == "rejection"  # (a random-init backbone's flat distributions rarely accept under rejection sampling)
    ctx.close()


# ----------------------------------------------------------------------------- projections on a single activation plane

@pytest.mark.parametrize("tree_name,n_prompt", [("sparse64_d4", 70), ("sparse128_d4", 70), ("sparse256_d4", 150)])
def test_single_plane_projections_report_their_accuracy(oracle, tree_name, n_prompt):
    """MEDUSA_OPT_ACTIVATION_PLANES = 1: the projections read only the hi plane of every activation (half the tensor-core
    work; four token tiles per weight stream).  This is an opt-in trade OUTSIDE the parity bar of the default path: the
    inputs of every projection carry a bfloat16 rounding (2^-9 relative), and three layers deep the normalised hidden
    state is off by 2.1e-2 .. 2.5e-2 instead of ~1e-2 -- just above the 2e-2 the default two-plane path is held to.  The
    bound asserted here is the documented one of this mode (4e-2 hidden, 5e-2 logits); the measured values are printed."""
    torch, B, U = _gpu()
    spec = _spec(tree_name)
    cfg = I.model_shape("tiny", d=512, n_heads=4, head_dim=128, ffn=1408, vocab=2048, n_medusa=4, n_layers=3,
                        max_tree_nodes=spec["n_nodes"])
    L_max = 512
    w = I.make_weights(cfg, seed=3, dtype="bf16", gain_std=0.1)
    ctx = U.make_ctx(cfg, "bf16", L_max, spec)
    ctx.set_option(B.OPT_ACTIVATION_PLANES, 1)
    ctx.load_weights(U.dev_weights(w))
    om = oracle.Model(cfg, w, kv_bf16=True)
    ot = oracle.build_tree_buffers(oracle.default_tree_paths(**spec))
    prompt = I.make_prompt(n_prompt, cfg["vocab"], 4)
    ctx.prefill(torch.from_numpy(prompt).cuda())
    kc = np.zeros(om.cache_shape(L_max))
    vc = np.zeros_like(kc)
    L = 0
    while L < n_prompt:
        n = min(64, n_prompt - L)
        last = oracle.tree_pass(om, prompt[L:L + n], oracle.chain_tree(n), L, kc, vc, want_logits=False)
        oracle.accept_and_update_kv(last["tree_k"], last["tree_v"], kc, vc, np.arange(n), n - 1, n, L, last["hidden"], prompt[L:L + n])
        L += n
    T, d, V = ot["T"], cfg["d"], cfg["vocab"]
    tok = I.rng(5, "treetok").integers(0, V, size=T).astype(np.int32)
    ctx.tree_pass(torch.from_numpy(tok).cuda())
    ref = oracle.tree_pass(om, tok, ot, n_prompt, kc, vc)
    hid = ctx.read_workspace(B.WS_HIDDEN, (T, d), np.float32)
    lgt = ctx.read_workspace(B.WS_LOGITS, (T, V), np.float32)
    eh, el = np.abs(hid - ref["hidden"]).max(), np.abs(lgt - ref["logits"]).max()
    print("single plane, %s: hidden max |err| %.3g, logits %.3g" % (tree_name, eh, el))
    assert eh <= 2 * TOL_HIDDEN_BF16, "hidden max |err| %.3g" % eh
    assert el <= TOL_LOGIT_BF16, "logits max |err| %.3g" % el
    assert ctx.device_status() == 0
    ctx.close()
