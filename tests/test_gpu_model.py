"""GPU parity of the backbone tree pass and the whole decode loop against the CPU oracle (through the C ABI)."""
import numpy as np
import pytest

from paper_2401_10774_b200 import inputs as I

pytestmark = pytest.mark.gpu

TOL_HIDDEN_BF16 = 2e-2
TOL_LOGIT_BF16 = 5e-2
TOL_F32 = 5e-4


def _gpu():
    import torch
    from paper_2401_10774_b200 import binding as B
    from tests import gpu_util as U
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    return torch, B, U


def _setup(oracle, cfg, dt, tree_name, L_max, seed, head_init="normal", std=0.02, gain_std=0.0):
    torch, B, U = _gpu()
    w = I.make_weights(cfg, seed=seed, dtype=dt, head_init=head_init, std=std, gain_std=gain_std)
    ctx = U.make_ctx(cfg, dt, L_max, I.TREE_SPECS[tree_name])
    ctx.load_weights(U.dev_weights(w))
    om = oracle.Model(cfg, w)
    ot = oracle.build_tree_buffers(oracle.default_tree_paths(**I.TREE_SPECS[tree_name]))
    return ctx, om, ot


def _oracle_prefill(oracle, om, prompt, L_max):
    kc = np.zeros(om.cache_shape(L_max))
    vc = np.zeros_like(kc)
    L = 0
    last = None
    while L < len(prompt):
        T = min(64, len(prompt) - L)
        last = oracle.tree_pass(om, prompt[L:L + T], oracle.chain_tree(T), L, kc, vc)
        oracle.accept_and_update_kv(last["tree_k"], last["tree_v"], kc, vc, np.arange(T), T - 1, T, L, last["hidden"],
                                    prompt[L:L + T])
        L += T
    return kc, vc, last


PASS_CASES = [
    # name, model override, dtype, tree, n_prompt, tolerances (hidden, logits)
    ("tiny_f32", dict(), "f32", "dense22", 32, TOL_F32, TOL_F32),
    ("tiny_f32_long_prompt", dict(), "f32", "dense22", 150, TOL_F32, TOL_F32),
    ("small_bf16_d128", dict(d=512, n_heads=4, head_dim=128, ffn=1408, vocab=2048, n_medusa=4, n_layers=3), "bf16",
     "sparse64_d4", 70, TOL_HIDDEN_BF16, TOL_LOGIT_BF16),
    # grouped-query attention: two key/value heads for four query heads (the k and v projections become a second launch)
    ("tiny_f32_gqa", dict(n_kv_heads=2), "f32", "dense22", 70, TOL_F32, TOL_F32),
    ("small_bf16_d128_gqa", dict(d=512, n_heads=4, n_kv_heads=2, head_dim=128, ffn=1408, vocab=2048, n_medusa=4, n_layers=3),
     "bf16", "sparse64_d4", 70, TOL_HIDDEN_BF16, TOL_LOGIT_BF16),
    ("small_bf16_d64_5heads", dict(d=256, n_heads=4, head_dim=64, ffn=688, vocab=1000, n_medusa=5, n_layers=2), "bf16",
     "sparse64_d5", 9, TOL_HIDDEN_BF16, TOL_LOGIT_BF16),
]


@pytest.mark.parametrize("case", PASS_CASES, ids=[c[0] for c in PASS_CASES])
def test_prefill_and_tree_pass_parity(oracle, case):
    torch, B, U = _gpu()
    name, over, dt, tree_name, n_prompt, tol_h, tol_l = case
    cfg = I.model_shape("tiny", **over)
    L_max = 256
    ctx, om, ot = _setup(oracle, cfg, dt, tree_name, L_max, seed=3, gain_std=0.1)
    prompt = I.make_prompt(n_prompt, cfg["vocab"], 4)
    ctx.prefill(torch.from_numpy(prompt).cuda())
    st = ctx.state()
    assert st["cache_len"] == n_prompt and st["status"] == 0
    kc, vc, last = _oracle_prefill(oracle, om, prompt, L_max)
    NL, H, D, d, V = cfg["n_layers"], I.kv_heads(cfg), cfg["head_dim"], cfg["d"], cfg["vocab"]  # H: key/value heads
    g_kc = U.read_act(ctx, B.WS_K_CACHE, (NL, H, L_max, D))
    g_vc = U.read_act(ctx, B.WS_V_CACHE, (NL, H, L_max, D))
    tol_kv = 5e-2 if dt == "bf16" else TOL_F32
    assert np.abs(g_kc[:, :, :n_prompt] - kc[:, :, :n_prompt]).max() <= tol_kv
    assert np.abs(g_vc[:, :, :n_prompt] - vc[:, :, :n_prompt]).max() <= tol_kv
    assert not g_kc[:, :, n_prompt:].any(), "positions beyond the cache length stay untouched"
    T_last = (n_prompt - 1) % 64 + 1
    hid_last = ctx.read_workspace(B.WS_HIDDEN, (d,), np.float32, offset_elems=(T_last - 1) * d)
    assert np.abs(hid_last - last["hidden"][-1]).max() <= tol_h
    assert np.array_equal(ctx.read_workspace(B.WS_H_LAST, (d,), np.float32), hid_last)
    # root = argmax of the GPU's own last logits row (integer stage: judged on the GPU's tensor)
    lg = ctx.read_workspace(B.WS_LOGITS, (V,), np.float32, offset_elems=(T_last - 1) * V)
    assert np.abs(lg - last["logits"][-1]).max() <= tol_l
    assert st["root"] == int(oracle.topk(lg, 1)[0])
    # tree pass on arbitrary tokens, against the oracle on ITS cache (end-to-end float parity)
    tok = I.rng(5, "treetok").integers(0, V, size=ot["T"]).astype(np.int32)
    ctx.tree_pass(torch.from_numpy(tok).cuda())
    ref = oracle.tree_pass(om, tok, ot, n_prompt, kc, vc)
    T = ot["T"]
    hid = ctx.read_workspace(B.WS_HIDDEN, (T, d), np.float32)
    lgt = ctx.read_workspace(B.WS_LOGITS, (T, V), np.float32)
    tk = U.read_act(ctx, B.WS_TREE_K, (NL, 64, H, D))[:, :T]
    tv = U.read_act(ctx, B.WS_TREE_V, (NL, 64, H, D))[:, :T]
    eh, el = np.abs(hid - ref["hidden"]).max(), np.abs(lgt - ref["logits"]).max()
    assert eh <= tol_h, "hidden max |err| %.3g" % eh
    assert el <= tol_l, "logits max |err| %.3g" % el
    assert np.abs(tk - ref["tree_k"]).max() <= tol_kv and np.abs(tv - ref["tree_v"]).max() <= tol_kv
    ctx.close()


@pytest.mark.parametrize("n_kv_heads", [0, 2], ids=["mha", "gqa"])
def test_tiny_fp32_medusa_greedy_token_exact(oracle, n_kv_heads):
    # the tiny fp32 reference model: 2 heads, dense (2,2) tree, 32-token prompt, 64 generated tokens
    # (also with two key/value heads for its four query heads)
    torch, B, U = _gpu()
    cfg = I.model_shape("tiny", n_kv_heads=n_kv_heads)
    ctx, om, ot = _setup(oracle, cfg, "f32", "dense22", 128, seed=0, head_init="lm_copy")
    prompt = I.make_prompt(32, cfg["vocab"], 1)
    G = 64
    got = ctx.generate(prompt, G, B.AcceptParams(mode=B.GREEDY))
    ref = oracle.generate(om, ot, prompt, G, 128, mode=oracle.GREEDY)
    plain = oracle.generate_plain(om, prompt, G, 128)
    assert ref["tokens"].tolist() == plain["tokens"].tolist()
    assert got["tokens"].tolist() == ref["tokens"].tolist(), "greedy token stream differs from the oracle"
    assert got["emitted_per_step"].tolist() == ref["emitted_per_step"].tolist()
    e = got["emitted_per_step"]
    assert e.sum() == G and e.min() >= 1 and e.max() <= ot["depth"] + 1
    assert got["steps"] < G, "LM-head-initialised heads must get speculated tokens accepted"
    assert ctx.state()["cache_len"] == 32 + G
    # plain greedy decoding through the same library (root-only tree) gives the same stream
    ctx1 = U.make_ctx(cfg, "f32", 128, paths=np.zeros((0, 1), dtype=np.int32))
    ctx1.load_weights(ctx._keep[0])
    p1 = ctx1.generate(prompt, G, B.AcceptParams(mode=B.GREEDY))
    assert p1["tokens"].tolist() == got["tokens"].tolist() and p1["steps"] == G
    ctx.close()
    ctx1.close()


@pytest.mark.parametrize("mode", ["greedy", "typical", "typical_gumbel", "rejection"])
def test_small_bf16_decode_stagewise(oracle, mode):
    # bf16 model: float stages against the oracle end to end for the first step; integer stages against the
    # oracle fed the GPU's own tensors at every step.
    torch, B, U = _gpu()
    cfg = I.model_shape("tiny", d=512, n_heads=4, head_dim=128, ffn=1408, vocab=2048, n_medusa=5, n_layers=2)
    L_max = 160
    ctx, om, ot = _setup(oracle, cfg, "bf16", "sparse64_d5", L_max, seed=6, head_init="lm_copy")
    V, d, T, K = cfg["vocab"], cfg["d"], ot["T"], ot["depth"]
    prompt = I.make_prompt(40, V, 7)
    ctx.prefill(torch.from_numpy(prompt).cuda())
    tau, eps, delta = (0.0, 0.09, 0.3) if mode == "greedy" else (0.7, 0.09, 0.3)
    f32 = lambda x: float(np.float32(x))
    params = B.AcceptParams(mode=dict(greedy=B.GREEDY, rejection=B.REJECTION).get(mode, B.TYPICAL), temperature=tau, eps=eps,
                            delta=delta)
    steps = 12
    noise = I.gumbel_noise(steps, V, 52) if mode in ("typical_gumbel", "rejection") else None
    uni = I.uniform_noise(steps, T, 53) if mode == "rejection" else None  # rejection sampling: one uniform per node and step
    L = 40
    multi = 0
    for s in range(steps):
        st0 = ctx.state()
        h_last = ctx.read_workspace(B.WS_H_LAST, (d,), np.float32)
        g = None if noise is None else torch.from_numpy(noise[s] if uni is None else np.concatenate([noise[s], uni[s]])).cuda()
        ctx.decode_step(params, g, max_commit=1 << 20)
        st = ctx.state()
        assert st["status"] == 0
        # heads: float parity on the GPU's h_last, integer parity on the GPU's logits
        z = ctx.read_workspace(B.WS_HEAD_LOGITS, (K, V), np.float32)
        _, z_ref = oracle.medusa_heads(h_last, om.w["medusa_w1"][:K], om.w["medusa_w2"][:K])
        assert np.abs(z - z_ref).max() <= TOL_LOGIT_BF16
        ti = ctx.read_workspace(B.WS_TOPK_IDX, (K, ot["topk"]), np.int32)
        for k in range(K):
            assert ti[k].tolist() == oracle.topk(z[k], ot["topk"]).tolist()
        tok = ctx.read_workspace(B.WS_TREE_TOK, (T,), np.int32)
        assert tok.tolist() == oracle.expand_candidates(st0["root"], ti, ot)[0].tolist()
        # acceptance on the GPU's logits: bit-exact
        lg = ctx.read_workspace(B.WS_LOGITS, (T, V), np.float32)
        ref = oracle.evaluate_posterior(lg, tok, ot, mode=params.mode, tau=f32(tau), eps=f32(eps), delta=f32(delta),
                                        gumbel=None if noise is None else noise[s], uniform=None if uni is None else uni[s])
        assert mode == "greedy" or ref["min_margin"] > 1e-9
        acc = ctx.read_workspace(B.WS_ACC_NODES, (ot["depth"] + 1,), np.int32)
        assert (st["best"], st["accept_len"], st["next_root"]) == (ref["best"], ref["accept_len"], ref["next_root"])
        assert acc.tolist() == ref["acc_nodes"].tolist()
        # commit: cache rows L..L+n-1 are exactly the tree rows of the accepted nodes
        n = 1 + ref["accept_len"]
        assert st["cache_len"] == L + n and st["n_emitted"] == n and st["root"] == ref["next_root"]
        NL, H, D = cfg["n_layers"], cfg["n_heads"], cfg["head_dim"]
        tk = ctx.read_workspace(B.WS_TREE_K, (NL, 64, H, D), np.uint16)
        kc = ctx.read_workspace(B.WS_K_CACHE, (NL, H, L_max, D), np.uint16)
        tv = ctx.read_workspace(B.WS_TREE_V, (NL, 64, H, D), np.uint16)
        vc = ctx.read_workspace(B.WS_V_CACHE, (NL, H, L_max, D), np.uint16)
        for j in range(n):
            assert np.array_equal(kc[:, :, L + j], tk[:, acc[j]]) and np.array_equal(vc[:, :, L + j], tv[:, acc[j]])
        em = ctx.read_workspace(B.WS_EMITTED, (n,), np.int32)
        assert em.tolist() == tok[acc[:n]].tolist()
        hid = ctx.read_workspace(B.WS_HIDDEN, (T, d), np.float32)
        assert np.array_equal(ctx.read_workspace(B.WS_H_LAST, (d,), np.float32), hid[acc[n - 1]])
        L += n
        multi += n > 1
    # (a random-init backbone's distributions are nearly flat, so rejection sampling, which accepts a candidate with
    # its own probability, rarely accepts one here; its longer paths are exercised on planted logits at operator level)
    assert multi > 0 or mode == "rejection", "LM-head-initialised heads must get speculated tokens accepted"
    ctx.close()


def test_cache_full_is_reported_not_overrun(oracle):
    torch, B, U = _gpu()
    cfg = I.model_shape("tiny")
    ctx, om, ot = _setup(oracle, cfg, "f32", "dense22", 40, seed=0, head_init="lm_copy")
    prompt = I.make_prompt(38, cfg["vocab"], 1)
    with pytest.raises(B.MedusaError) as e:
        ctx.prefill(torch.from_numpy(I.make_prompt(41, cfg["vocab"], 1)).cuda())
    assert e.value.code == B.ERR_CACHE_FULL
    ctx.prefill(torch.from_numpy(prompt).cuda())
    # generate clamps the commit to the remaining capacity: exactly 2 more tokens fit
    r = ctx.generate(prompt, 10, B.AcceptParams(mode=B.GREEDY))
    assert r["emitted_per_step"].sum() == 2 and ctx.state()["cache_len"] == 40
    # a raw step without a budget on a full cache must refuse to write
    ctx.decode_step(B.AcceptParams(mode=B.GREEDY), None, max_commit=8)
    assert ctx.device_status() == B.ERR_CACHE_FULL and ctx.state()["cache_len"] == 40
    ctx.close()


@pytest.mark.parametrize("shape,n_layers,tree_name", [("7b", 32, "sparse64_d4"), ("13b", 40, "sparse64_d5")])
def test_full_size_7b_step_sampled_path_parity(oracle, shape, n_layers, tree_name):
    """The benchmark's configuration (7B shape, bf16, 64-node tree, the same kernels and launch shapes) at a
    short cache so that the oracle can follow: the oracle runs one root-to-leaf path as a chain -- by the
    tree-attention invariant that reproduces the tree pass's outputs for the nodes on the path.

    The float figures of this test are a REPORT: through N_L layers the rounding of the bf16 KV cache and of q and the
    attention probabilities injects an independent error per layer, and these add in quadrature, so the end-to-end
    error grows like sqrt(N_L).  The pass criterion for the floats lives in test_gpu_fullsize_layers.py, which holds
    every layer, on all 64 rows, to the flat tolerances on the layer's own input.  Here only a gross bound guards
    against a broken pass, and the integer stage is asserted bit-exact."""
    torch, B, U = _gpu()
    cfg = I.model_shape(shape, n_layers=n_layers)
    L_max, n_prompt = 4096, 16
    ctx, om, ot = _setup(oracle, cfg, "bf16", tree_name, L_max, seed=40)
    prompt = I.make_prompt(n_prompt, cfg["vocab"], 41)
    ctx.prefill(torch.from_numpy(prompt).cuda())
    kc = np.zeros(om.cache_shape(n_prompt + 8))
    vc = np.zeros_like(kc)
    last = oracle.tree_pass(om, prompt, oracle.chain_tree(n_prompt), 0, kc, vc)
    oracle.accept_and_update_kv(last["tree_k"], last["tree_v"], kc, vc, np.arange(n_prompt), n_prompt - 1, n_prompt, 0,
                                last["hidden"], prompt)
    d, V, T = cfg["d"], cfg["vocab"], ot["T"]
    hid_last = ctx.read_workspace(B.WS_HIDDEN, (d,), np.float32, offset_elems=(n_prompt - 1) * d)
    e_prefill = np.abs(hid_last - last["hidden"][-1]).max()
    tok = I.rng(5, "treetok").integers(0, V, size=T).astype(np.int32)
    ctx.tree_pass(torch.from_numpy(tok).cuda())
    row = [int(x) for x in ot["retrieve"][7] if x >= 0]
    ref = oracle.tree_pass(om, tok[row], oracle.chain_tree(len(row)), n_prompt, kc, vc)
    hid = ctx.read_workspace(B.WS_HIDDEN, (T, d), np.float32)[row]
    lg = ctx.read_workspace(B.WS_LOGITS, (T, V), np.float32)[row]
    eh, el = np.abs(hid - ref["hidden"]).max(), np.abs(lg - ref["logits"]).max()
    print("REPORT %s width, %d layers, end to end vs the oracle's own pass on one sampled path: prefill hidden err %.3g, "
          "tree hidden err %.3g, logits err %.3g (flat tolerances %.3g / %.3g apply per layer, see test_gpu_fullsize_layers.py)"
          % (shape, n_layers, e_prefill, eh, el, TOL_HIDDEN_BF16, TOL_LOGIT_BF16))
    assert max(e_prefill, eh) < 0.5 and el < 1.0, "the pass is broken, not merely rounded"
    # integer stage on the GPU's own logits: acceptance is bit-exact at full size too
    full = ctx.read_workspace(B.WS_LOGITS, (T, V), np.float32)
    p = B.AcceptParams(mode=B.TYPICAL, temperature=0.7, eps=0.09, delta=0.3)
    out = torch.full((3 + 9,), -7, dtype=torch.int32, device="cuda")
    lgd = torch.from_numpy(full).cuda()
    ctx.evaluate_posterior(lgd, torch.from_numpy(tok).cuda(), p, None, out[0:1], out[1:2], out[2:3], out[3:])
    o = out.cpu().numpy()
    f32 = lambda x: float(np.float32(x))
    r = oracle.evaluate_posterior(full, tok, ot, mode=oracle.TYPICAL, tau=f32(0.7), eps=f32(0.09), delta=f32(0.3))
    assert (int(o[0]), int(o[1]), int(o[2])) == (r["best"], r["accept_len"], r["next_root"])
    assert o[3:3 + ot["depth"] + 1].tolist() == r["acc_nodes"].tolist()
    assert ctx.device_status() == 0
    ctx.close()


def test_tiny_fp32_typical_sampled_generate_matches_oracle(oracle):
    """Typical acceptance with a Gumbel-max sampled root on the tiny fp32 model: the whole token stream and the
    tokens emitted per step must equal the oracle's replay of the same noise (the float32 path differs from the
    double oracle only in summation order, far below the decision margins of this seed)."""
    torch, B, U = _gpu()
    cfg = I.model_shape("tiny")
    ctx, om, ot = _setup(oracle, cfg, "f32", "dense22", 160, seed=0, head_init="lm_copy")
    prompt = I.make_prompt(32, cfg["vocab"], 1)
    G = 48
    noise = I.gumbel_noise(G, cfg["vocab"], 52)
    f32 = lambda x: float(np.float32(x))
    got = ctx.generate(prompt, G, B.AcceptParams(mode=B.TYPICAL, temperature=0.7, eps=0.09, delta=0.3), gumbel_host=noise)
    ref = oracle.generate(om, ot, prompt, G, 160, mode=oracle.TYPICAL, tau=f32(0.7), eps=f32(0.09), delta=f32(0.3),
                          gumbel=noise)
    assert got["tokens"].tolist() == ref["tokens"].tolist()
    assert got["emitted_per_step"].tolist() == ref["emitted_per_step"].tolist()
    assert got["emitted_per_step"].max() > 1, "typical acceptance should accept speculated tokens with these heads"
    ctx.close()


def test_tiny_fp32_rejection_sampling_generate_matches_an_oracle_loop(oracle):
    """Rejection sampling through the convenience loop (host noise rows of V + T floats per step) on the tiny fp32 model
    with sharpened heads: the token stream equals a loop over the oracle's stage functions fed the same noise."""
    torch, B, U = _gpu()
    cfg = I.model_shape("tiny")
    ctx, om, ot = _setup(oracle, cfg, "f32", "dense22", 160, seed=0, head_init="lm_copy")
    V, T, K = cfg["vocab"], ot["T"], ot["depth"]
    prompt = I.make_prompt(32, V, 1)
    G, tau = 40, 0.05   # a low temperature sharpens the random-init distributions, so that candidates do get accepted
    f32 = lambda x: float(np.float32(x))
    noise = np.concatenate([I.gumbel_noise(G, V, 54), I.uniform_noise(G, T, 55)], axis=1)
    got = ctx.generate(prompt, G, B.AcceptParams(mode=B.REJECTION, temperature=tau), gumbel_host=noise)
    # the same loop over the oracle's stages
    kc = np.zeros(om.cache_shape(160)); vc = np.zeros_like(kc)
    last = oracle.tree_pass(om, prompt, oracle.chain_tree(len(prompt)), 0, kc, vc)
    oracle.accept_and_update_kv(last["tree_k"], last["tree_v"], kc, vc, np.arange(len(prompt)), len(prompt) - 1, len(prompt), 0,
                                last["hidden"], prompt)
    L, h_last, root = len(prompt), last["hidden"][-1].copy(), int(oracle.topk(last["logits"][-1].astype(np.float32), 1)[0])
    out, per_step, step, min_margin = [], [], 0, np.inf
    while len(out) < G:
        _, z = oracle.medusa_heads(h_last, om.w["medusa_w1"][:K], om.w["medusa_w2"][:K])
        ti = np.stack([oracle.topk(z[k].astype(np.float32), ot["topk"]) for k in range(K)])
        tok = oracle.expand_candidates(root, ti, ot)[0]
        p = oracle.tree_pass(om, tok, ot, L, kc, vc)
        r = oracle.evaluate_posterior(p["logits"].astype(np.float32), tok, ot, mode=oracle.REJECTION, tau=f32(tau),
                                      gumbel=noise[step, :V], uniform=noise[step, V:])
        min_margin = min(min_margin, r["min_margin"])
        c = oracle.accept_and_update_kv(p["tree_k"], p["tree_v"], kc, vc, r["acc_nodes"], r["accept_len"], G - len(out), L,
                                        p["hidden"], tok)
        em = [int(t) for t in c["emitted"] if t >= 0]
        n = len(em)
        # a budget that cuts the accepted path short makes the path's next token the next root (as the library does)
        root = int(tok[r["acc_nodes"][n]]) if n < 1 + r["accept_len"] else r["next_root"]
        L, h_last = c["L"], c["h_last"]
        out += em
        per_step.append(n)
        step += 1
    assert min_margin > 2e-3, "a uniform too close to its acceptance probability for a float32-vs-double comparison: change the seed"
    assert got["tokens"].tolist() == out[:G]
    assert got["emitted_per_step"].tolist() == per_step
    assert max(per_step) > 1, "the sharpened distributions must let some candidates through"
    ctx.close()


@pytest.mark.parametrize("mode", ["greedy", "typical_gumbel"])
def test_step_graph_replay_matches_plain_launches(oracle, mode):
    # The library captures a decode step into a CUDA graph on the second use of a launch configuration.  The same
    # steps with the graphs switched off must leave bit-identical state behind, across a change of the attention
    # grid (the cache grows through several 64-key tiles) and with the host following the cache length without
    # synchronising.
    torch, B, U = _gpu()
    cfg = I.model_shape("tiny", d=512, n_heads=4, head_dim=128, ffn=1408, vocab=2048, n_medusa=4, n_layers=2)
    L_max, n_prompt, steps = 512, 100, 60
    w = I.make_weights(cfg, seed=11, dtype="bf16", head_init="lm_copy")
    prompt = torch.from_numpy(I.make_prompt(n_prompt, cfg["vocab"], 12)).cuda()
    params = B.AcceptParams(mode=B.GREEDY) if mode == "greedy" else B.AcceptParams(mode=B.TYPICAL, temperature=0.7, eps=0.09, delta=0.3)
    noise = torch.from_numpy(I.gumbel_noise(steps, cfg["vocab"], 52)).cuda() if mode != "greedy" else None
    pinned = torch.zeros(2 * steps * 8, dtype=torch.int32).pin_memory()
    runs = []
    for graphs in (1, 0):
        ctx = U.make_ctx(cfg, "bf16", L_max, I.TREE_SPECS["sparse64_d4"])
        ctx.set_option(B.OPT_STEP_GRAPHS, graphs)
        ctx.load_weights(U.dev_weights(w))
        ctx.prefill(prompt)
        lens = []
        for s in range(steps):
            # the first third of the steps syncs and reads the emitted tokens on the host, like a serving loop;
            # the others are enqueued back to back
            if s < steps // 3:
                ctx.decode_step(params, None if noise is None else noise[s], 1 << 20, pinned.data_ptr(), pinned.data_ptr() + 32)
                torch.cuda.synchronize()
                lens.append(int(pinned[8]))
            else:
                ctx.decode_step(params, None if noise is None else noise[s], 1 << 20)
        st = ctx.state()
        assert st["status"] == 0
        info = ctx.step_graph_info()
        NL, H, D = cfg["n_layers"], cfg["n_heads"], cfg["head_dim"]
        kc = ctx.read_workspace(B.WS_K_CACHE, (NL, H, L_max, D), np.uint16)
        h_last = ctx.read_workspace(B.WS_H_LAST, (cfg["d"],), np.float32)
        runs.append((st, lens, kc[:, :, : st["cache_len"]].copy(), h_last, info))
        ctx.close()
    (st1, lens1, kc1, h1, info1), (st0, lens0, kc0, h0, info0) = runs
    assert info0 == dict(graphs=0, replays=0)
    assert info1["graphs"] >= 2 and info1["replays"] >= steps // 2, info1
    assert st1 == st0 and lens1 == lens0
    assert st1["cache_len"] > n_prompt + steps, "LM-head-initialised heads must get speculated tokens accepted"
    assert np.array_equal(kc1, kc0) and np.array_equal(h1, h0)


@pytest.mark.parametrize("shape", ["small", "gqa_ragged_ffn", "7b_2layers"])
def test_packed_weights_give_the_same_bits_as_row_major_weights(shape):
    """By default a bf16 context streams its own tile-by-tile copy of the backbone matrices (MEDUSA_OPT_PACK_WEIGHTS);
    the arithmetic and its order are those of the row-major path, so prefill and decode steps must agree bit for bit.
    The shapes cover matrices whose rows / columns do not fill the last 128 x 64 tile (zero-padded in the packed copy)."""
    torch, B, U = _gpu()
    if shape == "small":
        cfg = I.model_shape("tiny", d=512, n_heads=4, head_dim=128, ffn=1408, vocab=2048, n_medusa=4, n_layers=2)
    elif shape == "gqa_ragged_ffn":  # ffn 1000: 7.8 tiles of 128 rows and 15.6 k blocks of 64; vocabulary 2000: 15.6 tiles
        cfg = I.model_shape("tiny", d=512, n_heads=4, n_kv_heads=2, head_dim=128, ffn=1000, vocab=2000, n_medusa=4, n_layers=2)
    else:
        cfg = I.model_shape("7b", n_layers=2)
    w = U.dev_weights(I.make_weights(cfg, seed=21, dtype="bf16", head_init="lm_copy"))
    prompt = torch.from_numpy(I.make_prompt(150, cfg["vocab"], 22)).cuda()
    params = B.AcceptParams(mode=B.TYPICAL, temperature=0.7, eps=0.09, delta=0.3)
    V, d = cfg["vocab"], cfg["d"]
    def five_steps(ctx):
        ctx.prefill(prompt)
        snaps = []
        for s in range(5):
            ctx.decode_step(params)
            snaps.append((ctx.read_workspace(B.WS_LOGITS, (64, V), np.float32).copy(),
                          ctx.read_workspace(B.WS_HIDDEN, (64, d), np.float32).copy(), ctx.state()))
        assert ctx.device_status() == 0
        return snaps

    runs = []
    for pack in (1, 0):
        ctx = U.make_ctx(cfg, "bf16", 512, I.TREE_SPECS["sparse64_d4"])
        ctx.set_option(B.OPT_PACK_WEIGHTS, pack)
        ctx.load_weights(w)
        runs.append(five_steps(ctx))
        if pack == 0:
            # the same context loads the weights anew, packed this time (its step graphs and earlier copies are dropped)
            ctx.set_option(B.OPT_PACK_WEIGHTS, 1)
            ctx.load_weights(w)
            runs.append(five_steps(ctx))
            ctx.load_weights(w)  # and once more: the previous packed copies are released
            runs.append(five_steps(ctx))
        ctx.close()
    for other in runs[1:]:
        for s in range(5):
            assert np.array_equal(runs[0][s][0].view(np.uint32), other[s][0].view(np.uint32)), "logits differ at step %d" % s
            assert np.array_equal(runs[0][s][1].view(np.uint32), other[s][1].view(np.uint32)), "hidden differs at step %d" % s
            assert runs[0][s][2] == other[s][2]


def test_bad_acceptance_mode_is_refused_and_leaves_the_step_graphs_on(oracle):
    torch, B, U = _gpu()
    cfg = I.model_shape("tiny")
    ctx, om, ot = _setup(oracle, cfg, "f32", "dense22", 128, seed=0, head_init="lm_copy")
    ctx.prefill(torch.from_numpy(I.make_prompt(20, cfg["vocab"], 1)).cuda())
    good = B.AcceptParams(mode=B.GREEDY)
    ctx.decode_step(good)
    with pytest.raises(B.MedusaError) as e:
        ctx.decode_step(B.AcceptParams(mode=7))
    assert e.value.code == B.ERR_INVALID_ARG
    for _ in range(4):
        ctx.decode_step(good)
    torch.cuda.synchronize()
    info = ctx.step_graph_info()
    assert info["graphs"] == 1 and info["replays"] >= 3 and ctx.device_status() == 0
    ctx.close()


def test_decode_with_commit_budget_of_one_continues_the_same_stream(oracle):
    """A caller that lets every step commit a single token (max_commit = 1) still walks the greedy token stream: after
    a truncated commit the next root is the accepted path's next token, not the token after the whole path."""
    torch, B, U = _gpu()
    cfg = I.model_shape("tiny")
    ctx, om, ot = _setup(oracle, cfg, "f32", "dense22", 128, seed=0, head_init="lm_copy")
    prompt = I.make_prompt(32, cfg["vocab"], 1)
    G = 40
    plain = oracle.generate_plain(om, prompt, G, 128)["tokens"].tolist()
    ctx.prefill(torch.from_numpy(prompt).cuda())
    got, truncated = [], 0
    for s in range(G):
        ctx.decode_step(B.AcceptParams(mode=B.GREEDY), None, max_commit=1)
        st = ctx.state()
        assert st["n_emitted"] == 1 and st["cache_len"] == 32 + s + 1 and st["status"] == 0
        got.append(int(ctx.read_workspace(B.WS_EMITTED, (1,), np.int32)[0]))
        truncated += st["accept_len"] > 0
    assert got == plain
    assert truncated > 0, "the budget must actually have cut accepted paths short for this test to mean anything"
    ctx.close()
