"""Pins of the CPU oracle against things fixed outside it: the paper's worked examples, closed forms,
library routines (numpy / torch / transformers on CPU), brute force on tiny inputs.  No GPU needed."""
import itertools
import json
import math
import os

import numpy as np
import pytest

from paper_2401_10774_b200 import inputs as I

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _popcount(x):
    return bin(int(x)).count("1")


# ----------------------------------------------------------------------------- trees (Sec. 2.1.2, 2.3.3)

@pytest.mark.parametrize("idx", [0, 1, 2])
def test_tree_pins(oracle, idx):
    pin = json.load(open(os.path.join(GOLD, "tree_pins.json")))["trees"][idx]
    paths = oracle.default_tree_paths(pin["per_depth_topk"], pin["n_nodes"])
    t = oracle.build_tree_buffers(paths)
    assert (t["T"], t["P"], t["depth"]) == (pin["T"], pin["P"], pin["depth"])
    assert np.bincount(t["pos"]).tolist() == pin["nodes_per_depth"]
    assert sum(_popcount(m) for m in t["mask"]) == pin["popcount_sum"]
    assert int(np.bitwise_xor.reduce(t["mask"])) == int(pin["mask_xor"], 16)
    assert t["retrieve"][0].tolist() == pin["first_row"]
    assert t["retrieve"][-1].tolist() == pin["last_row"]
    if "masks" in pin:
        assert [int(m) for m in t["mask"]] == [int(m, 16) for m in pin["masks"]]
        assert t["tree_idx"].tolist() == pin["tree_idx"]
        assert t["parent"].tolist() == pin["parent"]
    if "mask_last" in pin:
        assert int(t["mask"][-1]) == int(pin["mask_last"], 16)
    if "row20" in pin:
        assert t["retrieve"][20].tolist() == pin["row20"]
    tuples = {tuple(int(x) for x in p if x >= 0) for p in paths}
    for k in pin.get("kept", []):
        assert tuple(k) in tuples
    for k in pin.get("excluded", []):
        assert tuple(k) not in tuples
    if "score_sum" in pin:
        s = sum(1.0 / math.prod(i + 1 for i in tp) for tp in tuples)
        assert abs(s - pin["score_sum"]) < 1e-3


def test_tree_fig2_example(oracle):
    # Fig. 2: top-2 of head 1 and top-3 of head 2 -> 2*3 = 6 candidates, 2 + 6 = 8 new tokens
    paths = [(a, -1) for a in range(2)] + [(a, b) for a in range(2) for b in range(3)]
    t = oracle.build_tree_buffers(np.array(paths, dtype=np.int32))
    assert t["P"] == 6 and t["T"] - 1 == 8 and t["depth"] == 2 and t["topk"] == 3
    # every token sees exactly its predecessors: root, its depth-1 ancestor, itself
    for i in range(t["T"]):
        anc, v = set(), i
        while v >= 0:
            anc.add(v)
            v = int(t["parent"][v])
        assert {j for j in range(64) if (int(t["mask"][i]) >> j) & 1} == anc
        assert t["pos"][i] == len(anc) - 1


def test_tree_structural_invariants(oracle):
    for name, spec in I.TREE_SPECS.items():
        t = oracle.build_tree_buffers(oracle.default_tree_paths(spec["per_depth_topk"], spec["n_nodes"]))
        T = t["T"]
        for i in range(1, T):
            p = int(t["parent"][i])
            assert 0 <= p < i, "ancestors come first"
            assert int(t["mask"][i]) == int(t["mask"][p]) | (1 << i)
            assert t["pos"][i] == t["pos"][p] + 1
        assert all(int(t["mask"][i]) < (1 << (i + 1)) for i in range(T)), "mask is lower-triangular"
        assert np.all(np.diff(t["pos"]) >= 0)
        # every non-root node lies on at least one retrieve row; rows are root-to-leaf chains
        seen = set()
        for row in t["retrieve"]:
            row = [int(x) for x in row if x >= 0]
            assert row[0] == 0
            for a, b in zip(row, row[1:]):
                assert int(t["parent"][b]) == a
            seen |= set(row)
        assert seen == set(range(T))


def test_tree_rejects_bad_input(oracle):
    with pytest.raises(ValueError):
        oracle.build_tree_buffers(np.array([[0, 0]], dtype=np.int32))  # parent (0,) missing
    with pytest.raises(ValueError):
        oracle.build_tree_buffers(np.array([[0, -1], [0, -1]], dtype=np.int32))  # duplicate
    with pytest.raises(ValueError):
        oracle.build_tree_buffers(np.array([[-1, 0]], dtype=np.int32))  # hole


def test_greedy_tree_is_optimal_by_brute_force(oracle):
    # Sec. 2.3.3: greedy node adding maximises sum over nodes of prod_j a_j^(i_j) under a node budget.
    topk = (3, 2, 2)
    nodes = [()]
    for k in range(1, len(topk) + 1):
        nodes += list(itertools.product(*[range(s) for s in topk[:k]]))
    nonroot = nodes[1:]
    score = {n: 1.0 / math.prod(i + 1 for i in n) for n in nonroot}
    for budget in (2, 4, 6, 8):
        best = -1.0
        for sub in itertools.combinations(nonroot, budget - 1):
            s = set(sub)
            if all(len(n) == 1 or n[:-1] in s for n in sub):
                best = max(best, sum(score[n] for n in sub))
        got = oracle.default_tree_paths(topk, budget)
        got_score = sum(score[tuple(int(x) for x in p if x >= 0)] for p in got)
        assert abs(got_score - best) < 1e-12


def _acc_table(seed, depth, topk):
    """A plausible calibration table: accuracies fall with the rank and with the head's distance (Sec. 2.3.3)."""
    g = np.random.default_rng(seed)
    a = np.sort(g.random((depth, topk)), axis=1)[:, ::-1] * np.linspace(0.9, 0.4, depth)[:, None]
    return np.ascontiguousarray(a)


@pytest.mark.parametrize("idx", [0, 1, 2])
def test_tree_from_accuracies_reproduces_the_surrogate_trees(oracle, idx):
    # With acc[k][i] = 1/(i+1) inside the per-depth top-k and 0 outside, the accuracy-driven construction must
    # select exactly the node sets of the pinned default trees (same figures as tests/golden/tree_pins.json).
    pin = json.load(open(os.path.join(GOLD, "tree_pins.json")))["trees"][idx]
    tk = pin["per_depth_topk"]
    acc = np.zeros((len(tk), max(tk)))
    for k, s_k in enumerate(tk):
        acc[k, :s_k] = [1.0 / (i + 1) for i in range(s_k)]
    paths, expect = oracle.tree_paths_from_accuracies(acc, pin["n_nodes"])
    t = oracle.build_tree_buffers(paths)
    assert (t["T"], t["P"], t["depth"]) == (pin["T"], pin["P"], pin["depth"])
    assert np.bincount(t["pos"]).tolist() == pin["nodes_per_depth"]
    assert int(np.bitwise_xor.reduce(t["mask"])) == int(pin["mask_xor"], 16)
    assert t["retrieve"][0].tolist() == pin["first_row"] and t["retrieve"][-1].tolist() == pin["last_row"]
    if "score_sum" in pin:
        assert abs(expect - pin["score_sum"]) < 1e-3


def test_tree_from_accuracies_is_optimal_by_brute_force(oracle):
    # Sec. 2.3.3: the expected acceptance length of a tree is the sum over its nodes of prod_j a_j^(i_j); greedy node
    # adding attains the maximum over all connected trees of the same size.  Exhaustive check on small tables.
    for seed in range(4):
        depth, topk = 3, 3
        acc = _acc_table(seed, depth, topk)
        nonroot = [n for k in range(1, depth + 1) for n in itertools.product(range(topk), repeat=k)]
        score = {n: math.prod(acc[j, i] for j, i in enumerate(n)) for n in nonroot}
        for budget in (2, 3, 5, 7):
            best = max(sum(score[n] for n in sub) for sub in itertools.combinations(nonroot, budget - 1)
                       if all(len(n) == 1 or n[:-1] in set(sub) for n in sub))
            paths, expect = oracle.tree_paths_from_accuracies(acc, budget)
            got = [tuple(int(x) for x in p if x >= 0) for p in paths]
            assert len(set(got)) == budget - 1
            assert all(len(n) == 1 or n[:-1] in set(got) for n in got)
            assert abs(sum(score[n] for n in got) - best) < 1e-12
            assert abs(expect - best) < 1e-12


def test_tree_from_accuracies_special_cases(oracle):
    # one head: the tree is the top n-1 ranks by accuracy, whatever their order in the table
    acc = np.array([[0.1, 0.5, 0.2, 0.05]])
    paths, expect = oracle.tree_paths_from_accuracies(acc, 3)
    assert paths[:, 0].tolist() == [1, 2] and abs(expect - 0.7) < 1e-15
    # all-certain first ranks: a chain of depth K comes first (products stay 1), ties go to the shorter tuple
    acc = np.array([[1.0, 0.3], [1.0, 0.3], [1.0, 0.3]])
    paths, expect = oracle.tree_paths_from_accuracies(acc, 4)
    assert [[int(x) for x in p if x >= 0] for p in paths] == [[0], [0, 0], [0, 0, 0]] and expect == 3.0
    # a budget that takes every node of the Cartesian tree
    acc = _acc_table(7, 2, 2)
    paths, expect = oracle.tree_paths_from_accuracies(acc, 7)
    assert len(paths) == 6
    assert abs(expect - (acc[0].sum() + acc[0].sum() * acc[1].sum())) < 1e-12
    for bad in (np.array([[1.5, 0.1]]), np.array([[float("nan"), 0.1]]), np.array([[-0.1, 0.1]])):
        with pytest.raises(ValueError):
            oracle.tree_paths_from_accuracies(bad, 2)
    with pytest.raises(ValueError):
        oracle.tree_paths_from_accuracies(np.array([[0.5, 0.1]]), 4)  # only two nodes exist


# ----------------------------------------------------------------------------- heads, top-k (Sec. 2.1.1, 2.1.2)

def test_heads_init_identity(oracle):
    # W1 = 0 and W2 = LM head  =>  every head predicts exactly what the LM head predicts
    d, V, K = 48, 200, 3
    h = I.normal((d,), 1.0, 7, "h")
    lm = I.normal((V, d), 0.02, 7, "lm")
    W1 = np.zeros((K, d, d), dtype=np.float32)
    W2 = np.stack([lm] * K)
    x, z = oracle.medusa_heads(h, W1, W2)
    ref = lm.astype(np.float64) @ h.astype(np.float64)
    assert np.array_equal(x, np.stack([h.astype(np.float64)] * K)), "SiLU(0) = 0, residual only"
    for k in range(K):
        np.testing.assert_allclose(z[k], ref, rtol=0, atol=1e-13)
        assert oracle.topk(z[k].astype(np.float32), 1)[0] == int(np.argmax(ref.astype(np.float32)))


def test_heads_against_numpy(oracle):
    import torch

    d, V, K = 64, 300, 2
    inp = I.heads_inputs(d, V, K, 11, dtype="f32")
    x, z = oracle.medusa_heads(inp["h"], inp["W1"], inp["W2"])
    h = torch.from_numpy(inp["h"]).double()
    for k in range(K):
        xr = h + torch.nn.functional.silu(torch.from_numpy(inp["W1"][k]).double() @ h)
        zr = torch.from_numpy(inp["W2"][k]).double() @ xr
        np.testing.assert_allclose(x[k], xr.numpy(), rtol=0, atol=1e-13)
        np.testing.assert_allclose(z[k], zr.numpy(), rtol=0, atol=1e-13)


def test_heads_bf16_weights_are_widened_exactly(oracle):
    d, V, K = 32, 64, 2
    a = I.heads_inputs(d, V, K, 5, dtype="bf16")
    x1, z1 = oracle.medusa_heads(I.as_f32(a["h"]), a["W1"], a["W2"])
    x2, z2 = oracle.medusa_heads(I.as_f32(a["h"]), I.as_f32(a["W1"]), I.as_f32(a["W2"]))
    assert np.array_equal(z1, z2) and np.array_equal(x1, x2)


def test_silu_values(oracle):
    assert oracle.silu(0.0) == 0.0
    assert abs(oracle.silu(1.0) - 1.0 / (1.0 + math.exp(-1.0))) < 1e-15
    assert abs(oracle.silu(-2.0) + 2.0 / (1.0 + math.exp(2.0))) < 1e-15


def test_topk_equals_stable_sort(oracle):
    g = I.rng(3, "topk")
    for n, k in ((17, 4), (1000, 4), (5, 5)):
        v = g.standard_normal(n).astype(np.float32)
        v[g.integers(0, n, size=n // 3)] = v[0]  # plant exact duplicates
        ref = np.argsort(-v, kind="stable")[:k]
        assert oracle.topk(v, k).tolist() == ref.tolist()
    assert oracle.topk(np.zeros(9, dtype=np.float32), 3).tolist() == [0, 1, 2]


def test_expand_candidates(oracle):
    t = oracle.build_tree_buffers(oracle.default_tree_paths((2, 2), 7))
    topk_idx = np.array([[10, 11], [20, 21]], dtype=np.int32)
    tok, cand = oracle.expand_candidates(99, topk_idx, t)
    assert tok.tolist() == [99, 10, 11, 20, 21, 20, 21]
    assert cand.tolist() == [[99, 10, 20], [99, 10, 21], [99, 11, 20], [99, 11, 21]]


# ----------------------------------------------------------------------------- building blocks

def test_rope_properties(oracle):
    g = I.rng(4, "rope")
    D = 64
    q, k = g.standard_normal(D), g.standard_normal(D)
    assert np.array_equal(oracle.rope(q, 0), q), "position 0 is the identity"
    for pos in (1, 17, 4095):
        assert abs(np.linalg.norm(oracle.rope(q, pos)) - np.linalg.norm(q)) < 1e-12
    # relative-position property: <R_m q, R_n k> depends only on m - n
    a = oracle.rope(q, 100) @ oracle.rope(k, 90)
    b = oracle.rope(q, 15) @ oracle.rope(k, 5)
    assert abs(a - b) < 1e-10
    # one frequency by hand: D = 2 -> plain rotation by pos radians (theta^0 = 1)
    v = oracle.rope(np.array([1.0, 0.0]), 1)
    np.testing.assert_allclose(v, [math.cos(1.0), math.sin(1.0)], atol=1e-15)
    # second pair of D = 4 rotates by pos * theta^(-1/2)
    v = oracle.rope(np.array([0.0, 1.0, 0.0, 0.0]), 3, theta=1e4)
    np.testing.assert_allclose(v, [0.0, math.cos(0.03), 0.0, math.sin(0.03)], atol=1e-15)


def test_rmsnorm_properties(oracle):
    d = 40
    g = np.linspace(0.5, 1.5, d).astype(np.float32)
    y = oracle.rmsnorm(np.full(d, -3.0), g, eps=0.0)
    np.testing.assert_allclose(y, -g.astype(np.float64), atol=1e-15)  # constant vector -> g * sign(x)
    x = I.rng(5, "rms").standard_normal(d)
    y = oracle.rmsnorm(x, np.ones(d, dtype=np.float32), eps=0.0)
    assert abs(np.mean(y * y) - 1.0) < 1e-12
    y2 = oracle.rmsnorm(x, np.ones(d, dtype=np.float32), eps=1e-5)
    np.testing.assert_allclose(y2, x / np.sqrt(np.mean(x * x) + 1e-5), atol=1e-15)


# ----------------------------------------------------------------------------- tree attention (Sec. 2.1.2)

def _sdpa(q, k, v, causal):
    import torch

    o = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q)[None], torch.from_numpy(k)[None], torch.from_numpy(v)[None], is_causal=causal)
    return o[0].numpy()


@pytest.mark.parametrize("L", [0, 5, 37])
def test_tree_attention_equals_per_path_causal_attention(oracle, L):
    # For every root-to-leaf path, ordinary causal attention over [cache; path] (library routine)
    # reproduces the tree outputs of every node on the path.
    H, D, L_max = 3, 16, 48
    t = oracle.build_tree_buffers(oracle.default_tree_paths((3, 2, 2), 14))
    T = t["T"]
    a = I.attention_inputs(T, H, D, L, L_max, 21, dtype="f32")
    out, lse = oracle.tree_attention(a["q"], a["k_new"], a["v_new"], a["k_cache"], a["v_cache"], L, t["mask"],
                                     t["pos"], apply_rope=True)
    # rotate with the oracle's own rope (pinned separately), then hand everything to torch
    q = np.stack([[oracle.rope(a["q"][i, h], L + t["pos"][i]) for h in range(H)] for i in range(T)])
    k = np.stack([[oracle.rope(a["k_new"][i, h], L + t["pos"][i]) for h in range(H)] for i in range(T)])
    for row in t["retrieve"]:
        row = [int(x) for x in row if x >= 0]
        n = len(row)
        for h in range(H):
            kk = np.concatenate([a["k_cache"][h, :L].astype(np.float64), k[row, h]], axis=0)
            vv = np.concatenate([a["v_cache"][h, :L].astype(np.float64), a["v_new"][row, h].astype(np.float64)])
            # queries: pad with L dummy leading queries so that is_causal's lower-triangular mask lines up
            qq = np.concatenate([np.zeros((L, D)), q[row, h]], axis=0)
            ref = _sdpa(qq[None], kk[None], vv[None], causal=True)[0][L:]
            np.testing.assert_allclose(out[row, h], ref, rtol=0, atol=1e-12)
    assert np.all(np.isfinite(lse))


def test_tree_attention_single_query_is_decode_attention(oracle):
    H, D, L, L_max = 2, 32, 19, 19
    a = I.attention_inputs(1, H, D, L, L_max, 22, dtype="f32")
    out, lse = oracle.tree_attention(a["q"], a["k_new"], a["v_new"], a["k_cache"], a["v_cache"], L,
                                     np.array([1], dtype=np.uint64), np.array([0]), apply_rope=False)
    for h in range(H):
        kk = np.concatenate([a["k_cache"][h], a["k_new"][:, h]]).astype(np.float64)
        vv = np.concatenate([a["v_cache"][h], a["v_new"][:, h]]).astype(np.float64)
        ref = _sdpa(a["q"][:, h].astype(np.float64)[None], kk[None], vv[None], causal=False)[0]
        np.testing.assert_allclose(out[:, h], ref, rtol=0, atol=1e-12)
        s = (kk @ a["q"][0, h].astype(np.float64)) / math.sqrt(D)
        assert abs(lse[0, h] - (np.log(np.sum(np.exp(s - s.max()))) + s.max())) < 1e-12


def test_tree_attention_equal_keys_gives_mean_of_visible_values(oracle):
    H, D, L, L_max = 2, 8, 6, 8
    t = oracle.build_tree_buffers(oracle.default_tree_paths((2, 2), 7))
    T = t["T"]
    a = I.attention_inputs(T, H, D, L, L_max, 23, dtype="f32")
    a["k_new"][:] = 0.25
    a["k_cache"][:, :L] = 0.25
    out, _ = oracle.tree_attention(a["q"], a["k_new"], a["v_new"], a["k_cache"], a["v_cache"], L, t["mask"], t["pos"],
                                   apply_rope=False)
    for i in range(T):
        vis = [j for j in range(T) if (int(t["mask"][i]) >> j) & 1]
        for h in range(H):
            ref = (a["v_cache"][h, :L].astype(np.float64).sum(0) + a["v_new"][vis, h].astype(np.float64).sum(0)) / (
                L + len(vis))
            np.testing.assert_allclose(out[i, h], ref, atol=1e-13)


def test_grouped_query_attention_equals_full_attention_on_repeated_heads(oracle):
    # Grouped-query attention is ordinary multi-head attention whose key/value heads are each shared by H / Hkv
    # consecutive query heads: repeating every key/value head that many times must give the same numbers exactly.
    H, Hkv, D, L, L_max = 6, 2, 16, 11, 16
    t = oracle.build_tree_buffers(oracle.default_tree_paths((3, 2), 10))
    a = I.attention_inputs(t["T"], H, D, L, L_max, 24, dtype="f32", Hkv=Hkv)
    out, lse = oracle.tree_attention(a["q"], a["k_new"], a["v_new"], a["k_cache"], a["v_cache"], L, t["mask"],
                                     t["pos"], apply_rope=True)
    g = H // Hkv
    out_f, lse_f = oracle.tree_attention(a["q"], np.repeat(a["k_new"], g, axis=1), np.repeat(a["v_new"], g, axis=1),
                                         np.repeat(a["k_cache"], g, axis=0), np.repeat(a["v_cache"], g, axis=0), L,
                                         t["mask"], t["pos"], apply_rope=True)
    assert np.array_equal(out, out_f) and np.array_equal(lse, lse_f)
    # and the heads of one group really differ from each other (different queries), those of different groups too
    assert not np.allclose(out[:, 0], out[:, 1]) and not np.allclose(out[:, 0], out[:, g])


# ----------------------------------------------------------------------------- backbone (App. G Table 5)

def _hf_llama(cfg, w):
    import torch
    from transformers import LlamaConfig, LlamaForCausalLM

    hc = LlamaConfig(vocab_size=cfg["vocab"], hidden_size=cfg["d"], intermediate_size=cfg["ffn"],
                     num_hidden_layers=cfg["n_layers"], num_attention_heads=cfg["n_heads"],
                     num_key_value_heads=I.kv_heads(cfg), head_dim=cfg["head_dim"], rms_norm_eps=cfg["rms_eps"],
                     rope_theta=cfg["rope_theta"], max_position_embeddings=512, tie_word_embeddings=False,
                     attention_bias=False, mlp_bias=False)
    hc._attn_implementation = "eager"
    m = LlamaForCausalLM(hc).double().eval()
    sd = {"model.embed_tokens.weight": w["embed"], "model.norm.weight": w["final_norm"],
          "lm_head.weight": w["lm_head"]}
    names = dict(attn_norm="input_layernorm", wq="self_attn.q_proj", wk="self_attn.k_proj", wv="self_attn.v_proj",
                 wo="self_attn.o_proj", ffn_norm="post_attention_layernorm", w_gate="mlp.gate_proj",
                 w_up="mlp.up_proj", w_down="mlp.down_proj")
    for l, lw in enumerate(w["layers"]):
        for k, v in lw.items():
            sd["model.layers.%d.%s.weight" % (l, names[k])] = v
    missing = m.load_state_dict({k: torch.from_numpy(np.asarray(v)).double() for k, v in sd.items()}, strict=False)
    assert not [k for k in missing.missing_keys if "rotary" not in k]
    return m


@pytest.mark.parametrize("n_kv_heads", [0, 2, 1], ids=["mha", "gqa_2_kv_heads", "mqa_1_kv_head"])
def test_chain_pass_equals_library_llama(oracle, n_kv_heads):
    # A chain tree is ordinary causal decoding; the transformers Llama implementation (fp64, CPU) is the
    # independent statement of the block: RMSNorm, rotary pairing (i, i+D/2), SwiGLU, causal softmax attention,
    # and (with fewer key/value heads than query heads) which key/value head a query head reads.
    import torch

    cfg = I.model_shape("tiny", d=64, n_heads=4, n_kv_heads=n_kv_heads, head_dim=16, ffn=88, vocab=96, n_medusa=0)
    w = I.make_weights(cfg, seed=9, dtype="f32", gain_std=0.1, std=0.2)
    model = oracle.Model(cfg, w)
    hf = _hf_llama(cfg, w)
    toks = I.make_prompt(23, cfg["vocab"], 2)
    L_max = 32
    kc = np.zeros(model.cache_shape(L_max))
    vc = np.zeros_like(kc)
    # first 10 tokens as one chain, commit them, then 13 more against the cache
    r1 = oracle.tree_pass(model, toks[:10], oracle.chain_tree(10), 0, kc, vc)
    c = oracle.accept_and_update_kv(r1["tree_k"], r1["tree_v"], kc, vc, np.arange(10), 9, 10, 0, r1["hidden"],
                                    toks[:10])
    assert c["L"] == 10
    r2 = oracle.tree_pass(model, toks[10:], oracle.chain_tree(13), 10, kc, vc)
    with torch.no_grad():
        out = hf(torch.from_numpy(toks.astype(np.int64))[None], output_hidden_states=True)
    ref_logits = out.logits[0].numpy()
    got = np.concatenate([r1["logits"], r2["logits"]])
    # the library evaluates its rotary cos/sin tables in float32 whatever the model dtype, so agreement is
    # limited to float32 rounding of the angles (~1e-6 here); any structural mistake is orders above that
    np.testing.assert_allclose(got, ref_logits, rtol=0, atol=2e-5)
    ref_hidden = out.hidden_states[-1][0].numpy()  # after the final norm
    np.testing.assert_allclose(np.concatenate([r1["hidden"], r2["hidden"]]), ref_hidden, rtol=0, atol=2e-5)


def test_tree_pass_rows_equal_their_own_path(oracle):
    # each node's logits equal those of plain decoding along its root-to-node path (bit-for-bit in the oracle)
    cfg = I.model_shape("tiny", d=64, n_heads=4, head_dim=16, ffn=88, vocab=96, n_medusa=0)
    w = I.make_weights(cfg, seed=10, dtype="f32", std=0.2)
    model = oracle.Model(cfg, w)
    t = oracle.build_tree_buffers(oracle.default_tree_paths((2, 2), 7))
    prompt = I.make_prompt(9, cfg["vocab"], 3)
    L_max = 24
    kc = np.zeros(model.cache_shape(L_max))
    vc = np.zeros_like(kc)
    r0 = oracle.tree_pass(model, prompt, oracle.chain_tree(9), 0, kc, vc)
    oracle.accept_and_update_kv(r0["tree_k"], r0["tree_v"], kc, vc, np.arange(9), 8, 9, 0, r0["hidden"], prompt)
    tree_tok = I.rng(6, "tt").integers(0, cfg["vocab"], size=7).astype(np.int32)
    rt = oracle.tree_pass(model, tree_tok, t, 9, kc, vc)
    for row in t["retrieve"]:
        row = [int(x) for x in row]
        rc = oracle.tree_pass(model, tree_tok[row], oracle.chain_tree(len(row)), 9, kc, vc)
        assert np.array_equal(rc["logits"], rt["logits"][row])
        assert np.array_equal(rc["tree_k"], rt["tree_k"][:, row])


# ----------------------------------------------------------------------------- acceptance (Sec. 2.3.1)

def _single_child_tree(oracle):
    return oracle.build_tree_buffers(np.array([[0]], dtype=np.int32))


def test_typical_acceptance_hand_vectors(oracle):
    cases = json.load(open(os.path.join(GOLD, "typical_acceptance_vectors.json")))["cases"]
    t = _single_child_tree(oracle)
    for c in cases:
        lg = np.array(c["logits"], dtype=np.float32)
        V = lg.size
        # the fixture's own consistency (hand values)
        assert abs(sum(c["p"]) - 1.0) < 5e-6
        assert abs(c["threshold"] - min(c["eps"], c.get("delta_exp_negH", c["delta"] * math.exp(-c["H"])))) < 2e-6
        for x in range(V):
            logits = np.stack([lg, np.zeros(V, dtype=np.float32)])
            r = oracle.evaluate_posterior(logits, [0, x], t, mode=oracle.TYPICAL, tau=c["tau"], eps=c["eps"],
                                          delta=c["delta"])
            assert (r["accept_len"] == 1) == c["pass"][x], (c, x)
            assert r["acc_nodes"].tolist() == ([0, 1] if c["pass"][x] else [0, -1])
            # the three quantities of the criterion, as the oracle itself evaluates them, against the hand values
            st = oracle.typical_decision(lg, x, c["tau"], c["eps"], c["delta"])
            assert st["ok"] == c["pass"][x]
            assert abs(st["p"] - c["p"][x]) < 2e-6, (c, x, st)
            assert abs(st["H"] - c["H"]) < 2e-6, (c, st)
            assert abs(st["threshold"] - c["threshold"]) < 2e-6, (c, st)
            if "delta_exp_negH" in c:
                assert abs(c["delta"] * math.exp(-st["H"]) - c["delta_exp_negH"]) < 2e-6
        if c.get("entropy_branch_decides"):
            # the entropy term is what decides: some token sits between delta*exp(-H) and eps, clear of both
            # (>= 10 % above the threshold, >= 4 % below eps; >= 10 % on both sides in the tau = 1 cases)
            thr = c["threshold"]
            assert thr < c["eps"] / 1.1
            assert any(1.1 * thr <= q <= c["eps"] / (1.1 if c["tau"] == 1.0 else 1.04) for q in c["p"])


def _planted(oracle, t, path_row, n_ok, V=64, seed=0):
    """logits such that exactly the first n_ok speculated tokens of retrieve row path_row are greedy-correct"""
    g = I.rng(seed, "planted")
    logits = g.standard_normal((t["T"], V)).astype(np.float32)
    tok = np.zeros(t["T"], dtype=np.int32)
    # distinct tokens among siblings
    for i in range(t["T"]):
        sib = [j for j in range(t["T"]) if t["parent"][j] == t["parent"][i]]
        tok[i] = 3 + sib.index(i)
    row = [int(x) for x in t["retrieve"][path_row] if x >= 0]
    for j in range(1, len(row)):
        par, c = row[j - 1], row[j]
        if j <= n_ok:
            logits[par, tok[c]] = 50.0
        else:
            logits[par, 0] = 50.0  # token 0 is nobody's candidate
    return logits, tok, row


def test_greedy_acceptance_planted_paths(oracle):
    t = oracle.build_tree_buffers(oracle.default_tree_paths((4, 3, 2, 2), 64))
    for path_row in (0, 7, 29):
        for n_ok in range(0, 5):
            logits, tok, row = _planted(oracle, t, path_row, n_ok, seed=path_row * 10 + n_ok)
            r = oracle.evaluate_posterior(logits, tok, t, mode=oracle.GREEDY)
            assert r["accept_len"] == n_ok
            assert r["acc_nodes"][: n_ok + 1].tolist() == row[: n_ok + 1]
            assert np.all(r["acc_nodes"][n_ok + 1:] == -1)
            assert r["next_root"] == int(np.argmax(logits[row[n_ok]]))
            assert 1 <= 1 + r["accept_len"] <= t["depth"] + 1


def test_typical_reductions_and_bounds(oracle):
    t = oracle.build_tree_buffers(oracle.default_tree_paths((4, 3, 2, 2, 2), 64))
    g = I.rng(8, "typ")
    V = 50
    for trial in range(20):
        logits = (3.0 * g.standard_normal((t["T"], V))).astype(np.float32)
        tok = g.integers(0, 6, size=t["T"]).astype(np.int32)
        gr = oracle.evaluate_posterior(logits, tok, t, mode=oracle.GREEDY)
        # temperature -> 0+ reverts to greedy (Sec. 2.3.1); tau <= 0 is greedy by definition
        cold = oracle.evaluate_posterior(logits, tok, t, mode=oracle.TYPICAL, tau=1e-3, eps=0.09, delta=0.3)
        zero = oracle.evaluate_posterior(logits, tok, t, mode=oracle.TYPICAL, tau=0.0)
        for r in (cold, zero):
            assert r["accept_len"] == gr["accept_len"] and r["acc_nodes"].tolist() == gr["acc_nodes"].tolist()
        # for delta < 1 the argmax token always passes (p_max >= exp(-H)), so typical accepts at least as much
        ty = oracle.evaluate_posterior(logits, tok, t, mode=oracle.TYPICAL, tau=0.7, eps=0.09, delta=0.3)
        assert ty["accept_len"] >= gr["accept_len"]
        # eps = delta = 0: everything with p > 0 passes -> first row, full length (row 0 is unpadded)
        al = oracle.evaluate_posterior(logits, tok, t, mode=oracle.TYPICAL, tau=0.7, eps=0.0, delta=0.0)
        assert al["best"] == 0 and al["accept_len"] == t["depth"]
        assert al["acc_nodes"].tolist() == t["retrieve"][0].tolist()
        # threshold above 1: nothing passes, one token per step
        no = oracle.evaluate_posterior(logits, tok, t, mode=oracle.TYPICAL, tau=0.7, eps=2.0, delta=1e30)
        assert no["accept_len"] == 0 and no["acc_nodes"][0] == 0 and no["next_root"] == int(np.argmax(logits[0]))


def test_typical_padded_row_and_tie_rule(oracle):
    # sparse64_d5 has one leaf at depth 4 (row 20, -1 padded).  Make only that row pass.
    t = oracle.build_tree_buffers(oracle.default_tree_paths((4, 3, 2, 2, 2), 64))
    assert t["retrieve"][20, -1] == -1
    logits, tok, row = _planted(oracle, t, 20, 4, seed=99)
    r = oracle.evaluate_posterior(logits, tok, t, mode=oracle.TYPICAL, tau=1.0, eps=0.5, delta=0.5)
    assert r["accept_len"] == 4 and r["acc_nodes"].tolist() == row + [-1]
    # the lowest row index wins ties: rows sharing the accepted prefix
    sharing = [i for i, rr in enumerate(t["retrieve"]) if rr[:5].tolist() == row]
    assert r["best"] == min(sharing)


def test_gumbel_root_sampling(oracle):
    t = _single_child_tree(oracle)
    V = 16
    g = I.rng(12, "gum")
    logits = g.standard_normal((2, V)).astype(np.float32)
    noise = I.gumbel_noise(1, V, 13)[0]
    r = oracle.evaluate_posterior(logits, [0, 5], t, mode=oracle.TYPICAL, tau=0.7, eps=2.0, delta=1e30, gumbel=noise)
    inv = np.float32(1.0 / 0.7)
    ref = int(np.argmax((logits[0] * inv).astype(np.float32) + noise))
    assert r["accept_len"] == 0 and r["next_root"] == ref
    # zero noise -> argmax
    r0 = oracle.evaluate_posterior(logits, [0, 5], t, mode=oracle.TYPICAL, tau=0.7, eps=2.0, delta=1e30,
                                   gumbel=np.zeros(V, dtype=np.float32))
    assert r0["next_root"] == int(np.argmax(logits[0]))


# ----------------------------------------------------------------------------- commit + whole decode

def test_commit_moves_exact_rows(oracle):
    NL, T, H, D, L_max, L, d = 2, 7, 2, 4, 16, 5, 6
    g = I.rng(14, "commit")
    tk, tv = g.standard_normal((NL, T, H, D)), g.standard_normal((NL, T, H, D))
    kc, vc = g.standard_normal((NL, H, L_max, D)), g.standard_normal((NL, H, L_max, D))
    kc0, vc0 = kc.copy(), vc.copy()
    hidden = g.standard_normal((T, d))
    tok = np.arange(100, 107, dtype=np.int32)
    r = oracle.accept_and_update_kv(tk, tv, kc, vc, [0, 2, 6], 2, 8, L, hidden, tok)
    assert r["L"] == 8 and r["emitted"].tolist() == [100, 102, 106]
    assert r["moved_src"].tolist() == [5, 7, 11] and r["moved_dst"].tolist() == [5, 6, 7]
    for j, node in enumerate([0, 2, 6]):
        assert np.array_equal(kc[:, :, L + j], tk[:, node]) and np.array_equal(vc[:, :, L + j], tv[:, node])
    keep = np.ones(L_max, bool)
    keep[5:8] = False
    assert np.array_equal(kc[:, :, keep], kc0[:, :, keep]) and np.array_equal(vc[:, :, keep], vc0[:, :, keep])
    assert np.array_equal(r["h_last"], hidden[6])
    # max_commit truncates; a full cache refuses
    r = oracle.accept_and_update_kv(tk, tv, kc, vc, [0, 2, 6], 2, 1, 8, hidden, tok)
    assert r["L"] == 9 and r["emitted"].tolist() == [100] and np.array_equal(r["h_last"], hidden[0])
    r = oracle.accept_and_update_kv(tk, tv, kc, vc, [0, 2, 6], 2, 3, 14, hidden, tok)
    assert r["L"] == -1


@pytest.mark.parametrize("head_init", ["lm_copy", "normal"])
def test_medusa_greedy_equals_plain_greedy(oracle, head_init):
    # Medusa-1 with greedy acceptance is lossless: token for token the plain greedy continuation.
    cfg = I.model_shape("tiny", d=64, n_heads=4, head_dim=16, ffn=88, vocab=128)
    w = I.make_weights(cfg, seed=0, dtype="f32", head_init=head_init, std=0.1)
    model = oracle.Model(cfg, w)
    t = oracle.build_tree_buffers(oracle.default_tree_paths((2, 2), 7))
    prompt = I.make_prompt(11, cfg["vocab"], 1)
    G, L_max = 40, 64
    med = oracle.generate(model, t, prompt, G, L_max, mode=oracle.GREEDY, return_cache=True)
    pl = oracle.generate_plain(model, prompt, G, L_max, return_cache=True)
    assert med["tokens"].tolist() == pl["tokens"].tolist()
    e = med["emitted_per_step"]
    assert e.sum() == G and np.all(e >= 1) and np.all(e <= t["depth"] + 1)
    if head_init == "lm_copy":
        assert med["steps"] < G, "heads initialised near the LM head must get some speculated tokens accepted"
    # the committed cache equals the cache plain decoding built for the same tokens
    n = len(prompt) + G - 1  # plain decoding has not yet processed the last emitted token's successor
    n = min(n, pl["L"])
    assert np.array_equal(med["k_cache"][:, :, :n], pl["k_cache"][:, :, :n])
    assert np.array_equal(med["v_cache"][:, :, :n], pl["v_cache"][:, :, :n])


def test_typical_generate_accepts_more_and_is_deterministic(oracle):
    cfg = I.model_shape("tiny", d=64, n_heads=4, head_dim=16, ffn=88, vocab=128)
    w = I.make_weights(cfg, seed=0, dtype="f32", head_init="lm_copy", std=0.1)
    model = oracle.Model(cfg, w)
    t = oracle.build_tree_buffers(oracle.default_tree_paths((2, 2), 7))
    prompt = I.make_prompt(11, cfg["vocab"], 1)
    a = oracle.generate(model, t, prompt, 30, 64, mode=oracle.TYPICAL, tau=0.7, eps=0.09, delta=0.3)
    b = oracle.generate(model, t, prompt, 30, 64, mode=oracle.TYPICAL, tau=0.7, eps=0.09, delta=0.3)
    gr = oracle.generate(model, t, prompt, 30, 64, mode=oracle.GREEDY)
    assert a["tokens"].tolist() == b["tokens"].tolist()
    assert np.all(a["emitted_per_step"] >= 1) and np.all(a["emitted_per_step"] <= 3)
    assert a["steps"] <= gr["steps"]


# ----------------------------------------------------------------------------- single-layer entry (layer-by-layer parity checks)

def test_layer_entry_composes_to_the_tree_pass_and_bf16_storage_rounding(oracle):
    """ora_layer runs the same block the pass runs: chaining it over the layers from the embedding rows, then the closing
    norm and LM head, reproduces ora_tree_pass bit for bit.  With kv_bf16 the tree keys/values are the unrounded ones
    rounded to bfloat16 (checked against numpy's own float32 -> bfloat16 rounding)."""
    cfg = I.model_shape("tiny", n_kv_heads=2)
    w = I.make_weights(cfg, seed=3, dtype="f32", gain_std=0.1)
    om = oracle.Model(cfg, w)
    t = oracle.build_tree_buffers(oracle.default_tree_paths((2, 2), 7))
    L_max, L = 24, 9
    g = I.rng(77, "layer-entry")
    kc = g.standard_normal(om.cache_shape(L_max))
    vc = g.standard_normal(om.cache_shape(L_max))
    tok = g.integers(0, cfg["vocab"], size=t["T"]).astype(np.int32)
    ref = oracle.tree_pass(om, tok, t, L, kc, vc)
    x = I.as_f32(w["embed"])[tok].astype(np.float64)
    for l in range(cfg["n_layers"]):
        r = oracle.layer(om, l, x, t, L, np.ascontiguousarray(kc[l]), np.ascontiguousarray(vc[l]))
        assert np.array_equal(r["tree_k"], ref["tree_k"][l]) and np.array_equal(r["tree_v"], ref["tree_v"][l])
        rb = oracle.layer(om, l, x, t, L, np.ascontiguousarray(kc[l]), np.ascontiguousarray(vc[l]), kv_bf16=True)
        for name in ("tree_k", "tree_v"):
            want = I.bf16_bits_to_f32(I.to_bf16_bits(r[name].astype(np.float32)))
            assert np.array_equal(rb[name], want.astype(np.float64))
        assert np.abs(rb["x_out"] - r["x_out"]).max() < 1e-2  # storage rounding moves the output only slightly
        x = r["x_out"]
    fin = oracle.final_norm_lm_head(om, x=x)
    assert np.array_equal(fin["hidden"], ref["hidden"]) and np.array_equal(fin["logits"], ref["logits"])
    # the LM head alone on a given hidden state
    alone = oracle.final_norm_lm_head(om, hidden_in=ref["hidden"])
    assert np.array_equal(alone["logits"], ref["logits"])


# ----------------------------------------------------------------------------- trees of more than 64 nodes (Sec. 3.3.1, Fig. 4)

def _independent_top_n_tree(per_depth_topk, n_nodes):
    """The surrogate sparse tree worked out a second way: enumerate the Cartesian tree, sort every node by (integer
    denominator prod(i_j + 1) ascending, tuple ascending with a prefix before its extensions), keep the best n - 1.
    Scores never increase along a path and a prefix sorts first, so the cut is prefix-closed and equals what greedy
    node adding (Sec. 2.3.3) selects."""
    nodes = []
    for k in range(1, len(per_depth_topk) + 1):
        nodes += list(itertools.product(*[range(s) for s in per_depth_topk[:k]]))
    nodes.sort(key=lambda n: (math.prod(i + 1 for i in n), n))
    return set(nodes[: n_nodes - 1])


def _row_bits(mask_row):
    """Set bits of a multi-word mask row (word w holds nodes 64 w .. 64 w + 63)."""
    words = np.atleast_1d(mask_row)
    return {64 * w + b for w, word in enumerate(words) for b in range(64) if (int(word) >> b) & 1}


@pytest.mark.parametrize("topk,n_nodes", [((6, 4, 3, 2, 2), 128), ((10, 6, 4, 3, 2), 256), ((8, 8), 73)])
def test_large_tree_buffers_against_an_independent_construction(oracle, topk, n_nodes):
    paths = oracle.default_tree_paths(topk, n_nodes)
    got = {tuple(int(x) for x in p if x >= 0) for p in paths}
    assert got == _independent_top_n_tree(topk, n_nodes)
    t = oracle.build_tree_buffers(paths)
    T = t["T"]
    assert T == n_nodes and t["mask"].shape == (T, (T + 63) // 64)
    # node order: root first, then (depth, tuple); masks = the ancestor sets found by walking the parent pointers
    order = [()] + sorted(got, key=lambda n: (len(n), n))
    index = {n: i for i, n in enumerate(order)}
    for i, n in enumerate(order):
        anc = {index[n[:k]] for k in range(len(n) + 1)}
        assert _row_bits(t["mask"][i]) == anc
        assert t["pos"][i] == len(n)
        assert t["parent"][i] == (index[n[:-1]] if n else -1)
        assert t["tree_idx"][i] == (1 + (len(n) - 1) * t["topk"] + n[-1] if n else 0)
    leaves = sorted(n for n in order if not any(m[:-1] == n for m in got if m))
    assert t["P"] == len(leaves)
    for r, leaf in enumerate(leaves):
        want = [index[leaf[:k]] for k in range(len(leaf) + 1)]
        assert [int(x) for x in t["retrieve"][r] if x >= 0] == want


@pytest.mark.parametrize("topk,n_nodes,L", [((6, 4, 3, 2, 2), 128, 9), ((10, 6, 4, 3, 2), 256, 0), ((7, 5, 3), 100, 33)])
def test_large_tree_attention_equals_per_path_causal_attention(oracle, topk, n_nodes, L):
    # the invariant that defines tree attention, on trees whose masks span several 64-bit words: for every
    # root-to-leaf path, ordinary causal attention over [cache; path] reproduces the outputs of the path's nodes
    H, D, L_max = 2, 16, 40
    t = oracle.build_tree_buffers(oracle.default_tree_paths(topk, n_nodes))
    T = t["T"]
    a = I.attention_inputs(T, H, D, L, L_max, 24, dtype="f32")
    out, lse = oracle.tree_attention(a["q"], a["k_new"], a["v_new"], a["k_cache"], a["v_cache"], L, t["mask"],
                                     t["pos"], apply_rope=True)
    q = np.stack([[oracle.rope(a["q"][i, h], L + t["pos"][i]) for h in range(H)] for i in range(T)])
    k = np.stack([[oracle.rope(a["k_new"][i, h], L + t["pos"][i]) for h in range(H)] for i in range(T)])
    covered = set()
    for row in t["retrieve"]:
        row = [int(x) for x in row if x >= 0]
        covered |= set(row)
        for h in range(H):
            kk = np.concatenate([a["k_cache"][h, :L].astype(np.float64), k[row, h]], axis=0)
            vv = np.concatenate([a["v_cache"][h, :L].astype(np.float64), a["v_new"][row, h].astype(np.float64)])
            qq = np.concatenate([np.zeros((L, D)), q[row, h]], axis=0)
            ref = _sdpa(qq[None], kk[None], vv[None], causal=True)[0][L:]
            np.testing.assert_allclose(out[row, h], ref, rtol=0, atol=1e-12)
    assert covered == set(range(T)) and np.all(np.isfinite(lse))


def test_large_tree_medusa_greedy_equals_plain_greedy(oracle):
    # the exactness property of greedy acceptance does not depend on the tree's size: a 100-node tree on the tiny model
    cfg = I.model_shape("tiny", n_medusa=3)
    w = I.make_weights(cfg, seed=0, dtype="f32", head_init="lm_copy")
    om = oracle.Model(cfg, w)
    t = oracle.build_tree_buffers(oracle.default_tree_paths((7, 5, 3), 100))
    prompt = I.make_prompt(20, cfg["vocab"], 1)
    G = 24
    ref = oracle.generate(om, t, prompt, G, 64, mode=oracle.GREEDY)
    plain = oracle.generate_plain(om, prompt, G, 64)
    assert ref["tokens"].tolist() == plain["tokens"].tolist()
    assert ref["emitted_per_step"].sum() == G and ref["emitted_per_step"].max() <= t["depth"] + 1


# ----------------------------------------------------------------------------- rejection sampling (Sec. 1, Sec. 2.3.1 first paragraph)

def _flat_tree(oracle, n_children):
    """Root with n_children leaf children (nodes 1..n in rank order)."""
    return oracle.build_tree_buffers(np.array([[i] for i in range(n_children)], dtype=np.int32))


def _accept_probability(oracle, logits, tok, t, tau, child, reject_before):
    """The probability with which the oracle accepts node `child`, read off its decisions: the uniform at which the
    decision flips (bisection in float32), with every node of `reject_before` forced to be rejected first."""
    V = logits.shape[1]
    zero = np.zeros(V, dtype=np.float32)
    lo, hi = np.float32(0.0), np.float32(1.0)
    for _ in range(40):
        mid = np.float32((np.float64(lo) + np.float64(hi)) / 2)
        u = np.zeros(t["T"], dtype=np.float32)
        u[list(reject_before)] = np.float32(0.99999994)
        u[child] = mid
        r = oracle.evaluate_posterior(logits, tok, t, mode=oracle.REJECTION, tau=tau, gumbel=zero, uniform=u)
        if child in r["acc_nodes"].tolist():
            lo = mid
        else:
            hi = mid
    return float(hi)


def test_rejection_sampling_hand_vectors(oracle):
    fx = json.load(open(os.path.join(GOLD, "rejection_sampling_vectors.json")))["cases"]
    for c in fx:
        lg = np.array(c["logits"], dtype=np.float32)
        V, m = lg.size, len(c["children_tokens"])
        t = _flat_tree(oracle, m)
        tok = np.array([0] + c["children_tokens"], dtype=np.int32)
        logits = np.tile(lg, (t["T"], 1))
        assert abs(sum(c["p"]) - 1.0) < 5e-6
        # the acceptance probability of every sibling, as the oracle takes its decisions, against the hand values
        for i in range(m):
            a = _accept_probability(oracle, logits, tok, t, c["tau"], 1 + i, range(1, 1 + i))
            assert abs(a - c["accept_prob"][i]) < 3e-6, (c["children_tokens"], i, a)
        for tr in c["trials"]:
            u = np.array([0.0] + tr["uniform"], dtype=np.float32)
            r = oracle.evaluate_posterior(logits, tok, t, mode=oracle.REJECTION, tau=c["tau"], gumbel=np.zeros(V, np.float32),
                                          uniform=u)
            k = tr["accepted_child"]
            if k >= 0:
                assert r["accept_len"] == 1 and r["acc_nodes"].tolist() == [0, 1 + k], (tr, r)
                assert r["rejected"].tolist() == [] and r["best"] == k
                if tr.get("decides_by_renormalisation"):
                    x = c["children_tokens"][k]
                    assert c["p"][x] < tr["uniform"][k] < c["accept_prob"][k]
            else:
                assert r["accept_len"] == 0 and r["acc_nodes"].tolist() == [0, -1]
                assert sorted(r["rejected"].tolist()) == sorted(c["children_tokens"])
                # the next token comes from the residual: never a rejected token, frequencies as worked by hand
                noise = I.gumbel_noise(6000, V, 77)
                counts = np.zeros(V)
                for row in noise:
                    counts[oracle.evaluate_posterior(logits, tok, t, mode=oracle.REJECTION, tau=c["tau"], gumbel=row,
                                                     uniform=u)["next_root"]] += 1
                for x in c["children_tokens"]:
                    assert counts[x] == 0
                for key, q in tr["residual"].items():
                    f = counts[int(key)] / len(noise)
                    assert abs(f - q) < 4 * math.sqrt(max(q * (1 - q), 1e-4) / len(noise)) + 1e-9, (key, f, q)


def test_rejection_sampling_keeps_the_backbone_distribution(oracle):
    """Losslessness, the property the scheme is for: the probability that the step's first new token is x equals
    softmax(logits / tau)[x].  For a child x_i that probability is prod_{j<i}(1 - a_j) * a_i with the oracle's own
    acceptance probabilities a (read off its decisions); a wrong renormalisation, sibling order or temperature breaks it."""
    g = I.rng(31, "rej")
    V, m, tau = 12, 5, 0.8
    t = _flat_tree(oracle, m)
    lg = (g.standard_normal(V) * 2.0).astype(np.float32)
    logits = np.tile(lg, (t["T"], 1))
    tok = np.concatenate([[0], g.permutation(V)[:m]]).astype(np.int32)
    x = lg.astype(np.float64) / tau
    p = np.exp(x - x.max())
    p /= p.sum()
    reach = 1.0
    for i in range(m):
        a = _accept_probability(oracle, logits, tok, t, tau, 1 + i, range(1, 1 + i))
        assert abs(reach * a - p[tok[1 + i]]) < 2e-6, (i, reach * a, p[tok[1 + i]])
        reach *= 1.0 - a
    # what is left is the mass of the tokens that are no child, and the residual sample lands only there
    rest = [v for v in range(V) if v not in tok[1:].tolist()]
    assert abs(reach - p[rest].sum()) < 5e-6
    u = np.full(t["T"], 0.99999994, dtype=np.float32)
    noise = I.gumbel_noise(8000, V, 78)
    counts = np.zeros(V)
    for row in noise:
        r = oracle.evaluate_posterior(logits, tok, t, mode=oracle.REJECTION, tau=tau, gumbel=row, uniform=u)
        assert r["accept_len"] == 0
        counts[r["next_root"]] += 1
    assert counts[tok[1:]].sum() == 0
    for v in rest:
        q = p[v] / p[rest].sum()
        assert abs(counts[v] / len(noise) - q) < 4 * math.sqrt(max(q * (1 - q), 1e-4) / len(noise)), (v, counts[v] / len(noise), q)


def test_rejection_sampling_walks_the_tree_with_each_nodes_own_logits(oracle):
    g = I.rng(32, "rejtree")
    spec = I.TREE_SPECS["sparse64_d4"]
    t = oracle.build_tree_buffers(oracle.default_tree_paths(**spec))
    T, V, W = t["T"], 50, t["depth"] + 1
    logits = g.standard_normal((T, V)).astype(np.float32)
    tok = np.zeros(T, dtype=np.int32)
    for n in range(T):  # siblings carry distinct tokens, as top-k picks do
        kids = [c for c in range(T) if c != n and t["parent"][c] == n]
        tok[kids] = g.permutation(V)[:len(kids)]
    zero = np.zeros(V, dtype=np.float32)
    # uniforms of zero accept the first child everywhere: the all-rank-0 path, full depth, next token from the leaf's row
    r = oracle.evaluate_posterior(logits, tok, t, mode=oracle.REJECTION, tau=1.0, gumbel=zero, uniform=np.zeros(T, np.float32))
    assert r["accept_len"] == t["depth"] and r["acc_nodes"].tolist() == t["retrieve"][r["best"]][:W].tolist()
    assert all(t["parent"][r["acc_nodes"][j]] == r["acc_nodes"][j - 1] for j in range(1, W))
    assert r["next_root"] == int(np.argmax(logits[r["acc_nodes"][-1]]))
    # uniforms just below one reject everything: nothing accepted, the children's tokens struck out at the root
    r = oracle.evaluate_posterior(logits, tok, t, mode=oracle.REJECTION, tau=1.0, gumbel=zero,
                                  uniform=np.full(T, 0.99999994, np.float32))
    kids0 = [c for c in range(T) if c != 0 and t["parent"][c] == 0]
    assert r["accept_len"] == 0 and r["rejected"].tolist() == tok[kids0].tolist()
    masked = logits[0].copy()
    masked[tok[kids0]] = -np.inf
    assert r["next_root"] == int(np.argmax(masked))
    # brute force of the definition, node by node, on random uniforms
    for trial in range(20):
        u = g.random(T).astype(np.float32)
        noise = I.gumbel_noise(1, V, 100 + trial)[0]
        r = oracle.evaluate_posterior(logits, tok, t, mode=oracle.REJECTION, tau=0.9, gumbel=noise, uniform=u)
        n, path, struck = 0, [0], []
        while True:
            x = logits[n].astype(np.float64) / 0.9
            p = np.exp(x - x.max())
            p /= p.sum()
            R, nxt, struck = 0.0, -1, []
            for c in range(T):
                if c != n and t["parent"][c] == n:
                    if float(u[c]) < p[tok[c]] / (1.0 - R):
                        nxt = c
                        break
                    R += p[tok[c]]
                    struck.append(int(tok[c]))
            if nxt < 0:
                break
            n = nxt
            path.append(n)
        assert r["acc_nodes"][:len(path)].tolist() == path and r["accept_len"] == len(path) - 1
        assert r["rejected"].tolist() == struck
        assert t["retrieve"][r["best"]][:len(path)].tolist() == path
        sc = (logits[n] * np.float32(1.0 / 0.9)).astype(np.float32) + noise
        sc[struck] = -np.inf
        assert r["next_root"] == int(np.argmax(sc))
        assert r["min_margin"] > 0.0


def test_rejection_sampling_at_low_temperature_is_greedy(oracle):
    g = I.rng(33, "rejcold")
    spec = I.TREE_SPECS["sparse64_d4"]
    t = oracle.build_tree_buffers(oracle.default_tree_paths(**spec))
    T, V = t["T"], 40
    for trial in range(6):
        logits = g.standard_normal((T, V)).astype(np.float32)
        tok = g.integers(0, V, size=T).astype(np.int32)
        # plant the argmax token on a path so that greedy acceptance has something to accept
        row = t["retrieve"][trial % t["P"]]
        for j in range(1, t["depth"] + 1):
            if row[j] >= 0 and j <= 1 + trial % 3:
                tok[row[j]] = int(np.argmax(logits[row[j - 1]]))
        for n in range(T):  # keep siblings distinct without touching planted nodes
            kids = [c for c in range(T) if c != n and t["parent"][c] == n]
            seen = set()
            for c in kids:
                while int(tok[c]) in seen:
                    tok[c] = (tok[c] + 1) % V if c not in row else tok[c]
                    if c in row:
                        break
                seen.add(int(tok[c]))
        gr = oracle.evaluate_posterior(logits, tok, t, mode=oracle.GREEDY)
        u = g.random(T).astype(np.float32) * np.float32(0.98) + np.float32(0.01)
        rj = oracle.evaluate_posterior(logits, tok, t, mode=oracle.REJECTION, tau=1e-3, gumbel=np.zeros(V, np.float32), uniform=u)
        assert rj["accept_len"] == gr["accept_len"] and rj["next_root"] == gr["next_root"]
        assert rj["acc_nodes"].tolist() == gr["acc_nodes"].tolist()


# ----------------------------------------------------------------------------- Medusa-1 head training (Sec. 2.2.1, Eq. 1)

def _train_case(seed, N=24, d=16, V=40, K=3):
    g = I.rng(seed, "train")
    h = g.standard_normal((N, d))
    W1 = 0.3 * g.standard_normal((K, d, d))
    W2 = 0.3 * g.standard_normal((K, V, d))
    y = g.integers(0, V, size=(K, N))
    for k in range(K):  # the last k + 1 positions of a sequence have no token that far ahead
        y[k, N - (k + 1):] = -1
    return h, W1, W2, y


def test_medusa1_loss_matches_torch_cross_entropy_and_autograd(oracle):
    torch = pytest.importorskip("torch")
    h, W1, W2, y = _train_case(3)
    K = W1.shape[0]
    lam = [0.8 ** (k + 1) for k in range(K)]
    r = oracle.medusa1_loss_and_grads(h, W1, W2, y)
    th = torch.tensor(h, dtype=torch.float64)
    t1 = torch.tensor(W1, dtype=torch.float64, requires_grad=True)
    t2 = torch.tensor(W2, dtype=torch.float64, requires_grad=True)
    total = 0.0
    for k in range(K):
        x = th + torch.nn.functional.silu(th @ t1[k].T)
        lk = torch.nn.functional.cross_entropy(x @ t2[k].T, torch.tensor(y[k]), ignore_index=-1, reduction="mean")
        assert abs(float(lk.detach()) - r["loss_per_head"][k]) < 1e-12
        total = total + lam[k] * lk
    total.backward()
    assert abs(float(total.detach()) - r["loss"]) < 1e-12
    assert np.abs(t1.grad.numpy() - r["grad_w1"]).max() < 1e-12
    assert np.abs(t2.grad.numpy() - r["grad_w2"]).max() < 1e-12


def test_medusa1_gradient_by_finite_differences(oracle):
    h, W1, W2, y = _train_case(4, N=10, d=8, V=12, K=2)
    r = oracle.medusa1_loss_and_grads(h, W1, W2, y)
    g = I.rng(5, "fd")
    eps = 1e-6
    for which, W, grad in (("w1", W1, r["grad_w1"]), ("w2", W2, r["grad_w2"])):
        for _ in range(12):
            idx = tuple(int(g.integers(0, n)) for n in W.shape)
            Wp, Wm = W.copy(), W.copy()
            Wp[idx] += eps
            Wm[idx] -= eps
            a = (W1, Wp) if which == "w2" else (Wp, W2)
            b = (W1, Wm) if which == "w2" else (Wm, W2)
            fd = (oracle.medusa1_loss_and_grads(h, a[0], a[1], y)["loss"] - oracle.medusa1_loss_and_grads(h, b[0], b[1], y)["loss"]) / (2 * eps)
            assert abs(fd - grad[idx]) < 1e-7, (which, idx, fd, grad[idx])


def test_medusa1_closed_forms(oracle):
    # zero weights: every head predicts the uniform distribution, loss_k = log V, and the gradient of W2_k is
    # lambda_k * mean_n (1/V - onehot(y_n)) h_n^T; the gradient of W1 vanishes with W2
    h, W1, W2, y = _train_case(6)
    K, V, d = W2.shape
    r = oracle.medusa1_loss_and_grads(h, np.zeros_like(W1), np.zeros_like(W2), y)
    assert np.allclose(r["loss_per_head"], math.log(V), atol=1e-13)
    assert abs(r["loss"] - sum(0.8 ** (k + 1) for k in range(K)) * math.log(V)) < 1e-12
    assert np.abs(r["grad_w1"]).max() == 0.0
    for k in range(K):
        rows = np.nonzero(y[k] >= 0)[0]
        ref = np.zeros((V, d))
        for n in rows:
            ref += (1.0 / V) * h[n][None, :]
            ref[y[k][n]] -= h[n]
        ref *= 0.8 ** (k + 1) / len(rows)
        assert np.abs(r["grad_w2"][k] - ref).max() < 1e-13
    # lambda scales a head's loss and gradient and nothing else; ignored positions change nothing
    r1 = oracle.medusa1_loss_and_grads(h, W1, W2, y, lam=[1.0, 0.0, 0.5])
    r2 = oracle.medusa1_loss_and_grads(h, W1, W2, y, lam=[2.0, 0.0, 0.5])
    assert np.allclose(r2["grad_w1"][0], 2 * r1["grad_w1"][0]) and np.abs(r1["grad_w2"][1]).max() == 0.0
    assert np.allclose(r2["grad_w2"][2], r1["grad_w2"][2])
    h2 = h.copy()
    h2[-1] += 5.0  # the last position carries no label for any head
    r3 = oracle.medusa1_loss_and_grads(h2, W1, W2, y)
    r0 = oracle.medusa1_loss_and_grads(h, W1, W2, y)
    assert r3["loss"] == r0["loss"] and np.array_equal(r3["grad_w2"], r0["grad_w2"])
    # a head whose logits already put all mass on the labels has (almost) no loss and no gradient
    big = np.zeros_like(W2)
    hh = np.eye(d)[:8]
    yy = np.tile(np.arange(8), (K, 1))
    for k in range(K):
        big[k, np.arange(8), np.arange(8)] = 60.0
    rz = oracle.medusa1_loss_and_grads(hh, np.zeros_like(W1), big, yy)
    assert rz["loss"] < 1e-20 and np.abs(rz["grad_w2"]).max() < 1e-20
