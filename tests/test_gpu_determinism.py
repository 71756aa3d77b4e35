"""Run-to-run determinism: every reduction of the path has a fixed order (stream-K pieces are added in CTA order, key
ranges are combined in range order, no floating-point atomics), so the same call on the same state must give the same
bits.  A data race or an unordered reduction would show up here as drift between repetitions."""
import numpy as np
import pytest

from paper_2401_10774_b200 import inputs as I

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("shape,tree_name,n_prompt", [("small", "sparse64_d5", 200), ("7b_2layers", "sparse64_d4", 600),
                                                      ("small_large_tree", "sparse256_d5", 130)])
def test_three_repetitions_give_identical_bits(shape, tree_name, n_prompt):
    import torch
    from paper_2401_10774_b200 import binding as B
    from tests import gpu_util as U
    if shape == "7b_2layers":
        cfg = I.model_shape("7b", n_layers=2)
    else:
        cfg = I.model_shape("tiny", d=512, n_heads=4, n_kv_heads=2, head_dim=128, ffn=1408, vocab=2048, n_medusa=5, n_layers=2)
    spec = I.LARGE_TREE_SPECS[tree_name] if tree_name in I.LARGE_TREE_SPECS else I.TREE_SPECS[tree_name]
    cfg["max_tree_nodes"] = spec["n_nodes"]
    w = U.dev_weights(I.make_weights(cfg, seed=12, dtype="bf16", head_init="lm_copy"))
    V, d, T = cfg["vocab"], cfg["d"], spec["n_nodes"]
    rows = 64 * ((T + 63) // 64)
    prompt = torch.from_numpy(I.make_prompt(n_prompt, V, 13)).cuda()
    noise = torch.from_numpy(I.gumbel_noise(6, V, 14)).cuda()
    params = B.AcceptParams(mode=B.TYPICAL, temperature=0.7, eps=0.09, delta=0.3)
    runs = []
    for rep in range(3):
        ctx = U.make_ctx(cfg, "bf16", 1024, spec)
        ctx.load_weights(w)
        ctx.prefill(prompt)
        snap = []
        for s in range(6):
            ctx.decode_step(params, noise[s])
            snap.append((ctx.read_workspace(B.WS_LOGITS, (rows, V), np.float32)[:T].copy(),
                         ctx.read_workspace(B.WS_HIDDEN, (rows, d), np.float32)[:T].copy(),
                         ctx.read_workspace(B.WS_HEAD_LOGITS, (cfg["n_medusa"], V), np.float32).copy(),
                         ctx.state()))
        assert ctx.device_status() == 0
        runs.append(snap)
        ctx.close()
    for rep in (1, 2):
        for s in range(6):
            for a, b in zip(runs[0][s][:3], runs[rep][s][:3]):
                assert np.array_equal(a.view(np.uint32), b.view(np.uint32)), "repetition %d, step %d: bits differ" % (rep, s)
            assert runs[0][s][3] == runs[rep][s][3]
