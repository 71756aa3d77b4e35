"""Batch > 1: a context that holds several independent sequences (own KV cache, cache length, root and last hidden state)
and steps them all in one backbone pass.  Every sequence must behave exactly as it would alone: against the oracle per
sequence, and against a single-sequence context of the same library."""
import numpy as np
import pytest

from paper_2401_10774_b200 import inputs as I

pytestmark = pytest.mark.gpu

TOL_LOGIT_BF16 = 5e-2
TOL_HIDDEN_BF16 = 2e-2


def _gpu():
    import torch
    from paper_2401_10774_b200 import binding as B
    from tests import gpu_util as U
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    return torch, B, U


def test_selected_sequences_are_independent_and_equal_to_single_contexts(oracle):
    """The single-sequence calls on a selected sequence of a 3-sequence context leave exactly the state a context of its
    own would have (same kernels, same rows): interleaved prefill and steps of three sequences of different lengths."""
    torch, B, U = _gpu()
    cfg = I.model_shape("tiny", d=512, n_heads=4, head_dim=128, ffn=1408, vocab=2048, n_medusa=4, n_layers=2)
    w = I.make_weights(cfg, seed=11, dtype="bf16", head_init="lm_copy")
    dw = U.dev_weights(w)
    L_max, steps = 256, 6
    prompts = [I.make_prompt(n, cfg["vocab"], 30 + i) for i, n in enumerate((17, 70, 129))]
    ctx = U.make_ctx(dict(cfg, max_batch=3), "bf16", L_max, I.TREE_SPECS["sparse64_d4"])
    ctx.load_weights(dw)
    params = B.AcceptParams(mode=B.GREEDY)
    for b, p in enumerate(prompts):
        ctx.select_sequence(b)
        ctx.prefill(torch.from_numpy(p).cuda())
    got = [[] for _ in prompts]
    for s in range(steps):
        for b in (2, 0, 1):  # interleaved, in an order of its own
            ctx.select_sequence(b)
            ctx.decode_step(params)
            st = ctx.state()
            got[b].append((st["cache_len"], st["root"], st["accept_len"], ctx.read_workspace(B.WS_EMITTED, (5,), np.int32).tolist()))
    for b, p in enumerate(prompts):
        one = U.make_ctx(cfg, "bf16", L_max, I.TREE_SPECS["sparse64_d4"])
        one.set_option(B.OPT_STEP_GRAPHS, 0)
        one.load_weights(dw)
        one.prefill(torch.from_numpy(p).cuda())
        ref = []
        for s in range(steps):
            one.decode_step(params)
            st = one.state()
            ref.append((st["cache_len"], st["root"], st["accept_len"], one.read_workspace(B.WS_EMITTED, (5,), np.int32).tolist()))
        assert got[b] == ref, b
        ctx.select_sequence(b)
        NL, H, D = cfg["n_layers"], cfg["n_heads"], cfg["head_dim"]
        L = ref[-1][0]
        kc_b = ctx.read_workspace(B.WS_K_CACHE, (NL, H, L_max, D), np.uint16)[:, :, :L]
        kc_1 = one.read_workspace(B.WS_K_CACHE, (NL, H, L_max, D), np.uint16)[:, :, :L]
        assert np.array_equal(kc_b, kc_1)
        one.close()
    with pytest.raises(B.MedusaError) as e:
        ctx.select_sequence(3)
    assert e.value.code == B.ERR_INVALID_ARG
    ctx.close()


def test_batched_greedy_decode_is_token_exact_on_the_tiny_model(oracle):
    """Three sequences stepped together on the fp32 model: each stream equals the oracle's (and plain greedy decoding's)."""
    torch, B, U = _gpu()
    cfg = I.model_shape("tiny")
    w = I.make_weights(cfg, seed=0, dtype="f32", head_init="lm_copy")
    ctx = U.make_ctx(dict(cfg, max_batch=3), "f32", 160, I.TREE_SPECS["dense22"])
    ctx.load_weights(U.dev_weights(w))
    om = oracle.Model(cfg, w)
    ot = oracle.build_tree_buffers(oracle.default_tree_paths(**I.TREE_SPECS["dense22"]))
    prompts = [I.make_prompt(n, cfg["vocab"], 40 + i) for i, n in enumerate((32, 9, 70))]
    G = 36
    for b, p in enumerate(prompts):
        ctx.select_sequence(b)
        ctx.prefill(torch.from_numpy(p).cuda())
    W = ot["depth"] + 1
    pinned = torch.zeros(3 * W + 3, dtype=torch.int32).pin_memory()
    streams = [[] for _ in prompts]
    per_step = [[] for _ in prompts]
    for s in range(G):  # at least one token per sequence and step: G steps are enough for G tokens
        ctx.decode_step_batch(B.AcceptParams(mode=B.GREEDY), None, 1 << 20, pinned.data_ptr(), pinned.data_ptr() + 4 * 3 * W)
        torch.cuda.synchronize()
        for b in range(3):
            n = int(pinned[3 * W + b])
            assert 1 <= n <= W
            streams[b] += pinned[b * W:b * W + n].tolist()
            per_step[b].append(n)
    assert ctx.device_status() == 0
    for b, p in enumerate(prompts):
        ref = oracle.generate(om, ot, p, G, 160, mode=oracle.GREEDY)
        plain = oracle.generate_plain(om, p, G, 160)
        assert ref["tokens"].tolist() == plain["tokens"].tolist()
        assert streams[b][:G] == ref["tokens"].tolist(), "sequence %d" % b
        k = len(ref["emitted_per_step"]) - 1  # (the oracle's last step may be cut by its budget of G tokens)
        assert per_step[b][:k] == ref["emitted_per_step"][:k].tolist()
    assert max(max(x) for x in per_step) > 1, "LM-head-initialised heads must get speculated tokens accepted"
    ctx.close()


@pytest.mark.parametrize("mode,n_seq", [("greedy", 2), ("typical_gumbel", 4), ("typical", 3), ("rejection", 3)])
def test_batched_bf16_decode_stagewise(oracle, mode, n_seq):
    """bf16 model, 2 to 4 sequences with prompts of different lengths: at every step and for every sequence the integer
    stages are bit-exact against the oracle fed the GPU's own tensors (the sequence's rows of the batched pass), and the
    float stages of the first step are within tolerance of the oracle's own pass on that sequence's cache."""
    torch, B, U = _gpu()
    cfg = I.model_shape("tiny", d=512, n_heads=4, n_kv_heads=2, head_dim=128, ffn=1408, vocab=2048, n_medusa=5, n_layers=2)
    L_max = 384
    w = I.make_weights(cfg, seed=6, dtype="bf16", head_init="lm_copy")
    ctx = U.make_ctx(dict(cfg, max_batch=n_seq), "bf16", L_max, I.TREE_SPECS["sparse64_d5"])
    ctx.load_weights(U.dev_weights(w))
    om = oracle.Model(cfg, w, kv_bf16=True)
    ot = oracle.build_tree_buffers(oracle.default_tree_paths(**I.TREE_SPECS["sparse64_d5"]))
    V, d, T, K = cfg["vocab"], cfg["d"], ot["T"], ot["depth"]
    NL, Hkv, D = cfg["n_layers"], I.kv_heads(cfg), cfg["head_dim"]
    lens = (40, 7, 200, 65)[:n_seq]
    prompts = [I.make_prompt(n, V, 50 + i) for i, n in enumerate(lens)]
    o_caches = []
    for b, p in enumerate(prompts):
        ctx.select_sequence(b)
        ctx.prefill(torch.from_numpy(p).cuda())
        kc = np.zeros(om.cache_shape(L_max)); vc = np.zeros_like(kc)
        L = 0
        while L < len(p):
            n = min(64, len(p) - L)
            last = oracle.tree_pass(om, p[L:L + n], oracle.chain_tree(n), L, kc, vc, want_logits=False)
            oracle.accept_and_update_kv(last["tree_k"], last["tree_v"], kc, vc, np.arange(n), n - 1, n, L, last["hidden"], p[L:L + n])
            L += n
        o_caches.append((kc, vc))
    tau, eps, delta = (0.0, 0.09, 0.3) if mode == "greedy" else (0.7, 0.09, 0.3)
    f32 = lambda x: float(np.float32(x))
    params = B.AcceptParams(mode=dict(greedy=B.GREEDY, rejection=B.REJECTION).get(mode, B.TYPICAL), temperature=tau, eps=eps,
                            delta=delta)
    steps = 8
    noise = I.gumbel_noise(steps * n_seq, V, 52).reshape(steps, n_seq, V) if mode in ("typical_gumbel", "rejection") else None
    # rejection sampling: every sequence's noise row is its Gumbel row followed by one uniform per tree node
    uni = I.uniform_noise(steps * n_seq, T, 53).reshape(steps, n_seq, T) if mode == "rejection" else None
    Ls = list(lens)
    multi = 0
    for s in range(steps):
        before = []
        for b in range(n_seq):
            ctx.select_sequence(b)
            before.append((ctx.state(), ctx.read_workspace(B.WS_H_LAST, (d,), np.float32)))
        rows = None if noise is None else (noise[s] if uni is None else np.concatenate([noise[s], uni[s]], axis=1))
        ctx.decode_step_batch(params, None if rows is None else torch.from_numpy(np.ascontiguousarray(rows)).cuda(), 1 << 20)
        lg_all = ctx.read_workspace(B.WS_LOGITS, (n_seq * 64, V), np.float32)
        tok_all = ctx.read_workspace(B.WS_TREE_TOK, (n_seq * 64,), np.int32)
        hid_all = ctx.read_workspace(B.WS_HIDDEN, (n_seq * 64, d), np.float32)
        tk_all = ctx.read_workspace(B.WS_TREE_K, (NL, n_seq * 64, Hkv, D), np.uint16)
        for b in range(n_seq):
            ctx.select_sequence(b)
            st = ctx.state()
            st0, h_last = before[b]
            assert st["status"] == 0
            z = ctx.read_workspace(B.WS_HEAD_LOGITS, (K, V), np.float32)
            _, z_ref = oracle.medusa_heads(h_last, om.w["medusa_w1"][:K], om.w["medusa_w2"][:K])
            assert np.abs(z - z_ref).max() <= TOL_LOGIT_BF16
            ti = ctx.read_workspace(B.WS_TOPK_IDX, (K, ot["topk"]), np.int32)
            for k in range(K):
                assert ti[k].tolist() == oracle.topk(z[k], ot["topk"]).tolist()
            tok = tok_all[b * 64:b * 64 + T]
            assert tok.tolist() == oracle.expand_candidates(st0["root"], ti, ot)[0].tolist()
            lg = lg_all[b * 64:b * 64 + T]
            if s == 0:
                ref_pass = oracle.tree_pass(om, tok, ot, Ls[b], *o_caches[b])
                eh = np.abs(hid_all[b * 64:b * 64 + T] - ref_pass["hidden"]).max()
                el = np.abs(lg - ref_pass["logits"]).max()
                assert eh <= TOL_HIDDEN_BF16 and el <= TOL_LOGIT_BF16, (b, eh, el)
            ref = oracle.evaluate_posterior(lg, tok, ot, mode=params.mode, tau=f32(tau), eps=f32(eps), delta=f32(delta),
                                            gumbel=None if noise is None else noise[s, b], uniform=None if uni is None else uni[s, b])
            assert mode == "greedy" or ref["min_margin"] > 1e-9
            acc = ctx.read_workspace(B.WS_ACC_NODES, (K + 1,), np.int32)
            assert (st["best"], st["accept_len"], st["next_root"]) == (ref["best"], ref["accept_len"], ref["next_root"]), (s, b)
            assert acc.tolist() == ref["acc_nodes"].tolist()
            n = 1 + ref["accept_len"]
            assert st["cache_len"] == Ls[b] + n and st["n_emitted"] == n and st["root"] == ref["next_root"]
            kc = ctx.read_workspace(B.WS_K_CACHE, (NL, Hkv, L_max, D), np.uint16)
            for j in range(n):
                assert np.array_equal(kc[:, :, Ls[b] + j], tk_all[:, b * 64 + acc[j]])
            assert ctx.read_workspace(B.WS_EMITTED, (n,), np.int32).tolist() == tok[acc[:n]].tolist()
            assert np.array_equal(ctx.read_workspace(B.WS_H_LAST, (d,), np.float32), hid_all[b * 64 + acc[n - 1]])
            Ls[b] += n
            multi += n > 1
    assert multi > 0 or mode == "rejection"  # (nearly flat distributions of a random-init backbone rarely accept under rejection sampling)
    ctx.close()


def test_batched_step_refuses_large_trees_and_too_many_sequences():
    torch, B, U = _gpu()
    cfg = dict(I.model_shape("tiny", n_medusa=3), max_batch=2, max_tree_nodes=100)
    ctx = U.make_ctx(cfg, "f32", 64, I.LARGE_TREE_SPECS["sparse100_d3"])
    w = I.make_weights(I.model_shape("tiny", n_medusa=3), seed=0, dtype="f32")
    ctx.load_weights(U.dev_weights(w))
    with pytest.raises(B.MedusaError) as e:
        ctx.decode_step_batch(B.AcceptParams(mode=B.GREEDY))
    assert e.value.code == B.ERR_SHAPE
    ctx.close()
    with pytest.raises(B.MedusaError) as e:
        B.Context(dict(I.model_shape("tiny"), max_batch=5), B.F32, 64)
    assert e.value.code == B.ERR_SHAPE
