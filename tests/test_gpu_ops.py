"""GPU parity of the per-operation entry points against the CPU oracle, element by element, through the C ABI."""
import numpy as np
import pytest

from paper_2401_10774_b200 import inputs as I

pytestmark = pytest.mark.gpu

TOL_ATTN_BF16 = 2e-2   # attention outputs / normalised hidden states, bf16 path vs fp64 oracle (max abs)
TOL_LOGIT_BF16 = 5e-2  # logits, bf16 path
TOL_F32 = 2e-4         # fp32 path: float accumulation order only


def _gpu():
    import torch
    from paper_2401_10774_b200 import binding as B
    from tests import gpu_util as U
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    return torch, B, U


# ------------------------------------------------------------------------------------------- tree attention
ATT_CASES = [
    # name, dtype, H, D, L, L_max, tree, apply_rope
    ("f32_d64_L0", "f32", 3, 64, 0, 16, "dense22", True),
    ("f32_d64_L37", "f32", 3, 64, 37, 48, "dense22", True),
    ("f32_d128_L70", "f32", 2, 128, 70, 96, "sparse64_d5", False),
    ("bf16_d128_L0", "bf16", 2, 128, 0, 64, "dense22", True),          # tree keys only, 7 query rows
    ("bf16_d128_L1", "bf16", 2, 128, 1, 64, "sparse64_d4", True),
    ("bf16_d128_L100", "bf16", 4, 128, 100, 128, "sparse64_d4", True),
    ("bf16_d128_L200_7rows", "bf16", 3, 128, 200, 256, "dense22", True),   # row-split form, second half has no rows
    ("bf16_d128_L500", "bf16", 5, 128, 500, 512, "sparse64_d5", True),     # row-split form, ragged last tile
    ("bf16_d128_L600", "bf16", 5, 128, 600, 640, "sparse64_d5", True),     # key ranges, ragged last tile
    ("bf16_d64_L333", "bf16", 3, 64, 333, 512, "sparse64_d5", True),
    ("bf16_7b_L1024", "bf16", 32, 128, 1024, 1024, "sparse64_d4", True),
    # grouped-query attention (9th field: key/value heads): row-split form, key-range form, generic kernel
    ("bf16_gqa_H8_kv2_L300", "bf16", 8, 128, 300, 320, "sparse64_d5", True, 2),
    ("bf16_gqa_H32_kv8_L1100", "bf16", 32, 128, 1100, 1152, "sparse64_d4", True, 8),
    ("f32_gqa_d64_H4_kv1_L37", "f32", 4, 64, 37, 48, "dense22", True, 1),
    ("bf16_7b_L4096", "bf16", 32, 128, 4096, 4096, "sparse64_d4", True),
]


def _run_attention_case(oracle, case, kernel=0, length_hint=None):
    torch, B, U = _gpu()
    name, dt, H, D, L, L_max, tree_name, rope = case[:8]
    Hkv = case[8] if len(case) > 8 else 0
    cfg = dict(n_layers=0, d=H * D, n_heads=H, n_kv_heads=Hkv, head_dim=D, ffn=8, vocab=8, n_medusa=5)
    ctx = U.make_ctx(cfg, dt, L_max, I.TREE_SPECS[tree_name])
    ctx.set_option(B.OPT_ATTENTION_KERNEL, kernel)
    if length_hint is not None:
        ctx.set_option(B.OPT_ATTENTION_LENGTH_HINT, length_hint)
    t = ctx.tree
    seed = 20 if L <= 1024 else 21
    a = I.attention_inputs(t["T"], H, D, L, L_max, seed, dtype=dt, Hkv=Hkv)
    dev = {k: U.to_dev(v) for k, v in a.items()}
    out = U.empty_act((t["T"], H, D), ctx.dtype)
    lse = torch.zeros((t["T"], H), dtype=torch.float32, device="cuda")
    cache_len = torch.tensor([L], dtype=torch.int32, device="cuda")
    ctx.tree_attention(dev["q"], dev["k_new"], dev["v_new"], dev["k_cache"], dev["v_cache"], cache_len, rope, out, lse)
    torch.cuda.synchronize()
    ot = oracle.build_tree_buffers(oracle.default_tree_paths(**I.TREE_SPECS[tree_name]))
    ref, ref_lse = oracle.tree_attention(*(I.as_f32(a[k]) for k in ("q", "k_new", "v_new", "k_cache", "v_cache")), L,
                                         ot["mask"], ot["pos"], apply_rope=rope)
    tol = TOL_ATTN_BF16 if dt == "bf16" else TOL_F32
    err = np.abs(U.to_host_f32(out) - ref).max()
    assert err <= tol, "max |err| %.3g > %.3g" % (err, tol)
    assert np.abs(U.to_host_f32(lse) - ref_lse).max() <= (5e-2 if dt == "bf16" else 1e-3)
    # input tensors are not modified (k_new is rotated into scratch, not in place)
    assert torch.equal(dev["k_new"], U.to_dev(a["k_new"]))
    assert ctx.device_status() == 0
    ctx.close()


@pytest.mark.parametrize("case", ATT_CASES, ids=[c[0] for c in ATT_CASES])
def test_tree_attention_parity(oracle, case):
    _run_attention_case(oracle, case)


TC_ATT_CASES = [c for c in ATT_CASES if c[1] == "bf16" and c[3] == 128] + [
    ("bf16_gqa_H16_kv4_L2500", "bf16", 16, 128, 2500, 2560, "sparse64_d4", True, 4),  # full TMA tiles of shared heads
    ("bf16_d128_L777", "bf16", 5, 128, 777, 1024, "sparse64_d5", True),  # ragged last tile, several key ranges
]


@pytest.mark.parametrize("case", TC_ATT_CASES, ids=[c[0] for c in TC_ATT_CASES])
def test_tree_attention_parity_tcgen05_kernel(oracle, case):
    """The tcgen05/TMEM variant of the attention kernel (selected with MEDUSA_OPT_ATTENTION_KERNEL) meets the same bar."""
    _run_attention_case(oracle, case, kernel=2)


@pytest.mark.parametrize("kernel", [1, 2], ids=["mma_sync", "tcgen05"])
@pytest.mark.parametrize("hint", [0, 300, 2500])
def test_tree_attention_length_hint_is_only_a_hint(oracle, kernel, hint):
    """A host-side length bound that is too small (or exact) changes the launch, never the result."""
    _run_attention_case(oracle, ("bf16_gqa_H16_kv4_L2500", "bf16", 16, 128, 2500, 2560, "sparse64_d4", True, 4),
                        kernel=kernel, length_hint=hint)


def _random_tree_paths(g, depth, target):
    """A random prefix-closed set of rank tuples with `target` nodes (root included), ranks below 5."""
    nodes = {()}
    for _ in range(4000):
        if len(nodes) >= target:
            break
        par = sorted(nodes)[int(g.integers(0, len(nodes)))]
        if len(par) < depth:
            nodes.add(par + (int(g.integers(0, 5)),))
    rows = [list(n) + [-1] * (depth - len(n)) for n in sorted(nodes) if n]
    return np.array(rows, dtype=np.int32).reshape(len(rows), depth)


@pytest.mark.parametrize("kernel", ["default", "tcgen05"])
@pytest.mark.parametrize("dt,D", [("bf16", 128), ("f32", 64)])
def test_tree_attention_random_trees(oracle, dt, D, kernel):
    """Irregular trees (any shape a caller may upload: chains, stars, lopsided ones, 2 to 64 nodes) at ragged cache
    lengths: the ancestor masks, positions and the tail tile must be right for every one of them."""
    if kernel == "tcgen05":
        if dt != "bf16":
            pytest.skip("the TMEM kernel exists for bf16, head dim 128")
    torch, B, U = _gpu()
    g = I.rng(61, "random-attention-trees")
    H = 3
    for trial in range(6):
        depth = int(g.integers(1, 6))
        T_target = [2, 64, 33, 17, 64, 5][trial]
        paths = _random_tree_paths(g, depth, T_target)
        depth = paths.shape[1]
        L = [0, 63, 64, 129, 200, 1][trial]
        L_max = 256
        cfg = dict(n_layers=0, d=H * D, n_heads=H, head_dim=D, ffn=8, vocab=8, n_medusa=5)
        ctx = U.make_ctx(cfg, dt, L_max, paths=paths)
        ctx.set_option(B.OPT_ATTENTION_KERNEL, 2 if kernel == "tcgen05" else 0)
        T = ctx.tree["T"]
        a = I.attention_inputs(T, H, D, L, L_max, 70 + trial, dtype=dt)
        dev = {k: U.to_dev(v) for k, v in a.items()}
        out = U.empty_act((T, H, D), ctx.dtype)
        cache_len = torch.tensor([L], dtype=torch.int32, device="cuda")
        ctx.tree_attention(dev["q"], dev["k_new"], dev["v_new"], dev["k_cache"], dev["v_cache"], cache_len, True, out, None)
        torch.cuda.synchronize()
        ot = oracle.build_tree_buffers(paths)
        ref, _ = oracle.tree_attention(*(I.as_f32(a[k]) for k in ("q", "k_new", "v_new", "k_cache", "v_cache")), L,
                                       ot["mask"], ot["pos"], apply_rope=True)
        err = np.abs(U.to_host_f32(out) - ref).max()
        assert err <= (TOL_ATTN_BF16 if dt == "bf16" else TOL_F32), (trial, T, L, err)
        assert ctx.device_status() == 0
        ctx.close()


def test_tree_attention_rejects_bad_arguments():
    torch, B, U = _gpu()
    cfg = dict(n_layers=0, d=128, n_heads=2, head_dim=64, ffn=8, vocab=8, n_medusa=2)
    ctx = B.Context(cfg, B.F32, 16)
    x = torch.zeros(7 * 2 * 64, device="cuda")
    cl = torch.zeros(1, dtype=torch.int32, device="cuda")
    with pytest.raises(B.MedusaError) as e:  # no tree yet
        ctx.tree_attention(x, x, x, x, x, cl, False, x)
    assert e.value.code == B.ERR_STATE
    ctx.build_tree_buffers(B.default_tree_paths((2, 2), 7))
    with pytest.raises(B.MedusaError) as e:
        ctx.tree_attention(None, x, x, x, x, cl, False, x)
    assert e.value.code == B.ERR_INVALID_ARG
    with pytest.raises(B.MedusaError) as e:  # misaligned
        ctx.tree_attention(x[1:], x, x, x, x, cl, False, x)
    assert e.value.code == B.ERR_INVALID_ARG
    with pytest.raises(B.MedusaError) as e:
        B.Context(dict(cfg, head_dim=80), B.F32, 16)
    assert e.value.code == B.ERR_SHAPE
    ctx.close()


# ------------------------------------------------------------------------------------------- heads + top-k + candidates
HEAD_CASES = [
    ("f32_small", "f32", 64, 300, 2, "dense22"),
    ("f32_tiny_shape", "f32", 256, 1024, 2, "dense22"),
    ("bf16_ragged", "bf16", 264, 1003, 4, "sparse64_d4"),
    ("bf16_7b", "bf16", 4096, 32000, 4, "sparse64_d4"),
    ("bf16_13b_5heads", "bf16", 5120, 32000, 5, "sparse64_d5"),
]


@pytest.mark.parametrize("case", HEAD_CASES, ids=[c[0] for c in HEAD_CASES])
def test_medusa_heads_parity(oracle, case):
    torch, B, U = _gpu()
    name, dt, d, V, K, tree_name = case
    cfg = dict(n_layers=0, d=d, n_heads=max(d // 128, 1), head_dim=128 if d >= 128 else 64, ffn=8, vocab=V, n_medusa=K)
    ctx = U.make_ctx(cfg, dt, 0, I.TREE_SPECS[tree_name])
    t = ctx.tree
    a = I.heads_inputs(d, V, K, 30, dtype=dt)
    h, W1, W2 = U.to_dev(a["h"]), U.to_dev(a["W1"]), U.to_dev(a["W2"])
    root = torch.tensor([a["root"]], dtype=torch.int32, device="cuda")
    topk_idx = torch.full((K, t["topk"]), -1, dtype=torch.int32, device="cuda")
    topk_val = torch.zeros((K, t["topk"]), dtype=torch.float32, device="cuda")
    logits = torch.zeros((K, V), dtype=torch.float32, device="cuda")
    tree_tok = torch.full((t["T"],), -1, dtype=torch.int32, device="cuda")
    ctx.medusa_heads(h, W1, W2, root, topk_idx, topk_val, logits, tree_tok)
    torch.cuda.synchronize()
    x_ref, z_ref = oracle.medusa_heads(I.as_f32(a["h"]), a["W1"], a["W2"])
    z = logits.cpu().numpy()
    tol = TOL_LOGIT_BF16 if dt == "bf16" else TOL_F32
    err = np.abs(z - z_ref).max()
    assert err <= tol, "head logits max |err| %.3g > %.3g" % (err, tol)
    # integer stages: bit-exact against the oracle fed the GPU's own logits
    ti = topk_idx.cpu().numpy()
    for k in range(K):
        assert ti[k].tolist() == oracle.topk(z[k], t["topk"]).tolist()
        assert topk_val[k].cpu().numpy().tolist() == z[k][ti[k]].tolist()
    ot = oracle.build_tree_buffers(oracle.default_tree_paths(**I.TREE_SPECS[tree_name]))
    tok_ref, _ = oracle.expand_candidates(a["root"], ti, ot)
    assert tree_tok.cpu().numpy().tolist() == tok_ref.tolist()
    ctx.close()


def test_topk_ties_go_to_lower_index(oracle):
    # heads whose logits contain exact duplicates: W2 rows repeated
    torch, B, U = _gpu()
    d, V, K = 64, 200, 2
    cfg = dict(n_layers=0, d=d, n_heads=1, head_dim=64, ffn=8, vocab=V, n_medusa=K)
    ctx = U.make_ctx(cfg, "f32", 0, I.TREE_SPECS["dense22"])
    a = I.heads_inputs(d, V, K, 31, dtype="f32")
    a["W2"][:, 100:200] = a["W2"][:, 0:100]  # every logit appears twice
    h, W1, W2 = U.to_dev(a["h"]), U.to_dev(a["W1"]), U.to_dev(a["W2"])
    root = torch.tensor([5], dtype=torch.int32, device="cuda")
    topk_idx = torch.zeros((K, 2), dtype=torch.int32, device="cuda")
    logits = torch.zeros((K, V), dtype=torch.float32, device="cuda")
    tree_tok = torch.zeros(7, dtype=torch.int32, device="cuda")
    ctx.medusa_heads(h, W1, W2, root, topk_idx, None, logits, tree_tok)
    z = logits.cpu().numpy()
    ti = topk_idx.cpu().numpy()
    for k in range(K):
        assert np.array_equal(z[k, :100], z[k, 100:])
        assert ti[k].tolist() == oracle.topk(z[k], 2).tolist()
        assert ti[k][0] < 100 and ti[k][1] == ti[k][0] + 100
    ctx.close()


# ------------------------------------------------------------------------------------------- acceptance
def _posterior_gpu(torch, B, ctx, logits, tok, mode, tau=0.0, eps=0.09, delta=0.3, gumbel=None):
    lg = torch.from_numpy(np.ascontiguousarray(logits, dtype=np.float32)).cuda()
    tk = torch.from_numpy(np.ascontiguousarray(tok, dtype=np.int32)).cuda()
    out = torch.full((3 + 16,), -7, dtype=torch.int32, device="cuda")
    g = None if gumbel is None else torch.from_numpy(np.ascontiguousarray(gumbel, dtype=np.float32)).cuda()
    p = B.AcceptParams(mode=mode, temperature=tau, eps=eps, delta=delta)
    ctx.evaluate_posterior(lg, tk, p, g, out[0:1], out[1:2], out[2:3], out[3:])
    o = out.cpu().numpy()
    W = ctx.tree["depth"] + 1
    return dict(best=int(o[0]), accept_len=int(o[1]), next_root=int(o[2]), acc_nodes=o[3:3 + W])


@pytest.mark.parametrize("tree_name", ["dense22", "sparse64_d4", "sparse64_d5"])
def test_evaluate_posterior_bit_exact(oracle, tree_name):
    torch, B, U = _gpu()
    V = 1000
    cfg = dict(n_layers=0, d=64, n_heads=1, head_dim=64, ffn=8, vocab=V, n_medusa=5)
    ctx = U.make_ctx(cfg, "f32", 0, I.TREE_SPECS[tree_name])
    ot = oracle.build_tree_buffers(oracle.default_tree_paths(**I.TREE_SPECS[tree_name]))
    g = I.rng(70, tree_name)
    f32 = lambda x: float(np.float32(x))
    n_multi = 0
    for trial in range(12):
        logits = (2.5 * g.standard_normal((ot["T"], V))).astype(np.float32)
        tok = g.integers(0, V, size=ot["T"]).astype(np.int32)
        # make some children likely: copy the parent's best tokens into the children
        for i in range(1, ot["T"]):
            if g.random() < 0.6:
                order = np.argsort(-logits[ot["parent"][i]], kind="stable")
                tok[i] = order[int(g.integers(0, 3))]
        noise = I.gumbel_noise(1, V, 100 + trial)[0]
        for mode, tau, eps, delta, gum in ((B.GREEDY, 0.0, 0.09, 0.3, None), (B.TYPICAL, 0.7, 0.09, 0.3, None),
                                           (B.TYPICAL, 1.3, 0.02, 0.14, noise), (B.TYPICAL, 0.0, 0.09, 0.3, None),
                                           (B.TYPICAL, 0.7, 0.0, 0.0, None), (B.TYPICAL, 0.7, 2.0, 1e30, noise)):
            ref = oracle.evaluate_posterior(logits, tok, ot, mode=mode, tau=f32(tau), eps=f32(eps), delta=f32(delta),
                                            gumbel=gum)
            assert mode == B.GREEDY or tau <= 0 or ref["min_margin"] > 1e-9, "ill-conditioned draw: change the seed"
            got = _posterior_gpu(torch, B, ctx, logits, tok, mode, tau, eps, delta, gum)
            for k in ("best", "accept_len", "next_root"):
                assert got[k] == ref[k], (trial, mode, tau, k, got, ref)
            assert got["acc_nodes"].tolist() == ref["acc_nodes"].tolist()
            n_multi += ref["accept_len"] > 0
    assert n_multi > 10, "the draws must exercise accepted paths"
    ctx.close()


def _distinct_sibling_tokens(g, ot, logits, V, likely=0.7):
    """Tree tokens as top-k picks give them: siblings distinct; with probability `likely` a child carries one of its
    parent's most probable tokens, so that rejection sampling accepts paths of every length."""
    T = ot["T"]
    tok = np.zeros(T, dtype=np.int32)
    tok[0] = int(g.integers(0, V))
    for n in range(T):
        kids = [c for c in range(T) if c != n and ot["parent"][c] == n]
        if not kids:
            continue
        order = np.argsort(-logits[n], kind="stable")
        pool = list(order[:len(kids)]) if g.random() < likely else list(g.permutation(V)[:len(kids)])
        tok[kids] = np.array(pool, dtype=np.int32)
    return tok


@pytest.mark.parametrize("tree_name", ["dense22", "sparse64_d4", "sparse64_d5", "sparse256_d5"])
def test_rejection_sampling_acceptance_bit_exact(oracle, tree_name):
    """Rejection sampling over the tree (Sec. 1 / Sec. 2.3.1, first paragraph; deterministic drafts): accepted path,
    row, and the token sampled from the residual equal the oracle's on identical logits, uniforms and Gumbel noise."""
    torch, B, U = _gpu()
    V = 1000
    spec = I.LARGE_TREE_SPECS[tree_name] if tree_name in I.LARGE_TREE_SPECS else I.TREE_SPECS[tree_name]
    cfg = dict(n_layers=0, d=64, n_heads=1, head_dim=64, ffn=8, vocab=V, n_medusa=5, max_tree_nodes=spec["n_nodes"])
    ctx = U.make_ctx(cfg, "f32", 0, spec)
    ot = oracle.build_tree_buffers(oracle.default_tree_paths(**spec))
    T = ot["T"]
    g = I.rng(71, tree_name)
    f32 = lambda x: float(np.float32(x))
    lens = []
    n_masked = 0
    for trial in range(16):
        logits = (2.5 * g.standard_normal((T, V))).astype(np.float32)
        tok = _distinct_sibling_tokens(g, ot, logits, V)
        noise = I.gumbel_noise(1, V, 300 + trial)[0]
        for tau in (0.7, 1.3, 0.05):
            u = g.random(T).astype(np.float32)
            if trial % 4 == 3:
                u[:] = np.float32(0.99999994)  # everything rejected: the residual sample excludes the root's children
            ref = oracle.evaluate_posterior(logits, tok, ot, mode=oracle.REJECTION, tau=f32(tau), gumbel=noise, uniform=u)
            assert ref["min_margin"] > 1e-9, "a uniform within rounding of its acceptance probability: change the seed"
            got = _posterior_gpu(torch, B, ctx, logits, tok, B.REJECTION, tau, 0.0, 0.0, np.concatenate([noise, u]))
            for k in ("best", "accept_len", "next_root"):
                assert got[k] == ref[k], (trial, tau, k, got, ref)
            assert got["acc_nodes"].tolist() == ref["acc_nodes"].tolist()
            lens.append(ref["accept_len"])
            # did the mask matter?  (the unmasked sample would have been a rejected token)
            last = ref["acc_nodes"][ref["accept_len"]]
            plain = int(np.argmax((logits[last] * np.float32(1.0 / f32(tau))).astype(np.float32) + noise))
            n_masked += plain != ref["next_root"]
    assert max(lens) >= min(3, ot["depth"]) and min(lens) == 0, "the draws must exercise short and long accepted paths"
    assert n_masked > 0, "the draws must exercise the exclusion of rejected tokens from the residual sample"
    assert ctx.device_status() == 0
    ctx.close()


def test_rejection_sampling_hand_vectors_and_refusals(oracle):
    import json
    import os
    torch, B, U = _gpu()
    fx = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "rejection_sampling_vectors.json")))["cases"]
    for c in fx:
        m = len(c["children_tokens"])
        paths = np.array([[i] for i in range(m)], dtype=np.int32)
        V = 8  # the fixture's four logits, padded with very unlikely tokens
        cfg = dict(n_layers=0, d=64, n_heads=1, head_dim=64, ffn=8, vocab=V, n_medusa=1)
        ctx = B.Context(cfg, B.F32, 0)
        ctx.build_tree_buffers(paths)
        row = np.full(V, -80.0, dtype=np.float32)
        row[:4] = c["logits"]
        logits = np.tile(row, (m + 1, 1))
        tok = np.array([0] + c["children_tokens"], dtype=np.int32)
        for tr in c["trials"]:
            u = np.array([0.0] + tr["uniform"], dtype=np.float32)
            got = _posterior_gpu(torch, B, ctx, logits, tok, B.REJECTION, c["tau"], 0.0, 0.0,
                                 np.concatenate([np.zeros(V, np.float32), u]))
            k = tr["accepted_child"]
            assert got["accept_len"] == (1 if k >= 0 else 0)
            assert got["acc_nodes"].tolist() == ([0, 1 + k] if k >= 0 else [0, -1])
            if k < 0:  # zero noise: the most probable token that was not rejected
                rest = [v for v in range(4) if v not in c["children_tokens"]]
                assert got["next_root"] == max(rest, key=lambda v: c["logits"][v])
        # refusals: no noise row, temperature zero
        lg = torch.from_numpy(logits).cuda()
        tk = torch.from_numpy(tok).cuda()
        out = torch.zeros(8, dtype=torch.int32, device="cuda")
        with pytest.raises(B.MedusaError):
            ctx.evaluate_posterior(lg, tk, B.AcceptParams(mode=B.REJECTION, temperature=0.7), None, out[0:1], out[1:2], out[2:3], out[3:])
        noise = torch.zeros(V + m + 1, device="cuda")
        with pytest.raises(B.MedusaError):
            ctx.evaluate_posterior(lg, tk, B.AcceptParams(mode=B.REJECTION, temperature=0.0), noise, out[0:1], out[1:2], out[2:3], out[3:])
        ctx.close()


def test_evaluate_posterior_planted_paths(oracle):
    torch, B, U = _gpu()
    V = 64
    cfg = dict(n_layers=0, d=64, n_heads=1, head_dim=64, ffn=8, vocab=V, n_medusa=5)
    ctx = U.make_ctx(cfg, "f32", 0, I.TREE_SPECS["sparse64_d5"])
    t = ctx.tree
    g = I.rng(71, "planted")
    for row_i in (0, 20, t["P"] - 1):
        row = [int(x) for x in t["retrieve"][row_i] if x >= 0]
        for n_ok in range(len(row)):
            logits = g.standard_normal((t["T"], V)).astype(np.float32)
            tok = np.zeros(t["T"], dtype=np.int32)
            for i in range(t["T"]):
                sib = [j for j in range(t["T"]) if t["parent"][j] == t["parent"][i]]
                tok[i] = 3 + sib.index(i)
            for j in range(1, len(row)):
                logits[row[j - 1], tok[row[j]] if j <= n_ok else 0] = 50.0
            got = _posterior_gpu(torch, B, ctx, logits, tok, B.GREEDY)
            assert got["accept_len"] == n_ok and got["acc_nodes"][: n_ok + 1].tolist() == row[: n_ok + 1]
            assert np.all(got["acc_nodes"][n_ok + 1:] == -1)
            assert got["next_root"] == int(np.argmax(logits[row[n_ok]]))
    ctx.close()


# ------------------------------------------------------------------------------------------- commit
@pytest.mark.parametrize("dt", ["f32", "bf16"])
def test_accept_and_update_kv_bit_exact(oracle, dt):
    torch, B, U = _gpu()
    NL, H, D, L_max, d = 3, 2, 64, 40, 128
    cfg = dict(n_layers=NL, d=d, n_heads=H, head_dim=D, ffn=8, vocab=8, n_medusa=2)
    ctx = U.make_ctx(cfg, dt, L_max, I.TREE_SPECS["dense22"])
    T = 7
    tk = I.normal((NL, 64, H, D), 1.0, 80, "tk", dt)
    tv = I.normal((NL, 64, H, D), 1.0, 80, "tv", dt)
    kc = I.normal((NL, H, L_max, D), 1.0, 80, "kc", dt)
    vc = I.normal((NL, H, L_max, D), 1.0, 80, "vc", dt)
    hidden = I.normal((T, d), 1.0, 80, "hid", "f32")
    tok = np.arange(100, 107, dtype=np.int32)
    cases = [([0, 2, 6], 2, 8, 5), ([0, 1, -1], 1, 8, 0), ([0, -1, -1], 0, 8, 37), ([0, 2, 5], 2, 2, 20),
             ([0, 2, 5], 2, 8, 38)]  # last one overflows L_max = 40
    for acc, alen, max_commit, L in cases:
        d_kc, d_vc = U.to_dev(kc), U.to_dev(vc)
        cl = torch.tensor([L], dtype=torch.int32, device="cuda")
        h_last = torch.zeros(d, dtype=torch.float32, device="cuda")
        emitted = torch.full((3,), -9, dtype=torch.int32, device="cuda")
        n_em = torch.full((1,), -9, dtype=torch.int32, device="cuda")
        ctx.reset()
        ctx.accept_and_update_kv(U.to_dev(tk), U.to_dev(tv), d_kc, d_vc, torch.tensor(acc, dtype=torch.int32, device="cuda"),
                                 torch.tensor([alen], dtype=torch.int32, device="cuda"), max_commit, cl, U.to_dev(hidden),
                                 h_last, torch.from_numpy(tok).cuda(), emitted, n_em)
        torch.cuda.synchronize()
        okc, ovc = I.as_f32(kc).astype(np.float64), I.as_f32(vc).astype(np.float64)
        ref = oracle.accept_and_update_kv(I.as_f32(tk)[:, :T].astype(np.float64), I.as_f32(tv)[:, :T].astype(np.float64),
                                          okc, ovc, acc, alen, max_commit, L, hidden.astype(np.float64), tok)
        if ref["L"] < 0:
            assert ctx.device_status() == B.ERR_CACHE_FULL
            assert int(cl.item()) == L and int(n_em.item()) == 0
            assert np.array_equal(U.to_host_f32(d_kc), I.as_f32(kc))
            continue
        assert ctx.device_status() == B.OK
        assert int(cl.item()) == ref["L"] and int(n_em.item()) == len(ref["emitted"])
        assert emitted.cpu().numpy()[: len(ref["emitted"])].tolist() == ref["emitted"].tolist()
        assert np.array_equal(U.to_host_f32(d_kc).astype(np.float64), okc), "K cache differs (gathered positions)"
        assert np.array_equal(U.to_host_f32(d_vc).astype(np.float64), ovc)
        assert np.array_equal(U.to_host_f32(h_last).astype(np.float64), ref["h_last"])
    ctx.close()


def test_non_finite_logits_still_give_valid_indices(oracle):
    # NaN logits are outside the contract, but they must never turn into an out-of-range token or node index
    torch, B, U = _gpu()
    V = 200
    cfg = dict(n_layers=0, d=64, n_heads=1, head_dim=64, ffn=8, vocab=V, n_medusa=2)
    ctx = U.make_ctx(cfg, "f32", 0, I.TREE_SPECS["dense22"])
    logits = np.full((7, V), np.nan, dtype=np.float32)
    tok = np.arange(7, dtype=np.int32)
    for mode, tau in ((B.GREEDY, 0.0), (B.TYPICAL, 0.7)):
        got = _posterior_gpu(torch, B, ctx, logits, tok, mode, tau)
        assert 0 <= got["next_root"] < V and 0 <= got["accept_len"] <= 2 and got["acc_nodes"][0] == 0
    a = I.heads_inputs(64, V, 2, 33, dtype="f32")
    a["h"][:] = np.nan
    topk_idx = torch.full((2, 2), -1, dtype=torch.int32, device="cuda")
    tree_tok = torch.full((7,), -1, dtype=torch.int32, device="cuda")
    ctx.medusa_heads(U.to_dev(a["h"]), U.to_dev(a["W1"]), U.to_dev(a["W2"]), torch.tensor([3], dtype=torch.int32, device="cuda"),
                     topk_idx, None, None, tree_tok)
    ti, tt = topk_idx.cpu().numpy(), tree_tok.cpu().numpy()
    assert ((ti >= 0) & (ti < V)).all() and ((tt >= 0) & (tt < V)).all()
    ctx.close()
