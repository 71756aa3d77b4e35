"""The allocation-free tree-attention entry point against the regular one (GPU, through the C ABI).

Collected last on purpose: a run that stops at the first failure has then already run every other test.
The entry point is for callers that cannot allocate device memory at call time (their own memory pool owns
the budget, or an implicit device synchronisation is not acceptable, or they hold no context): its scratch is
a fixed array inside the library, shared by all calls, so two calls in a row must both be right."""
import numpy as np
import pytest

from paper_2401_10774_b200 import inputs as I

pytestmark = pytest.mark.gpu

TOL_ATTN_BF16 = 2e-2  # the tolerance the other attention parity tests use (max abs, bf16 outputs)


# (cache length, heads, capacity, length hint given to the call): the hint sizes the launch and may be exact, absent
# (-1: the capacity is assumed) or too small (the result must not change); 2000 and 3000 keys use several key ranges
# per head, i.e. the fixed scratch array really carries partial results between CTAs
CASES = [(0, 8, 1024, 0), (300, 8, 1024, 300), (1000, 8, 1024, 1000), (1000, 8, 1024, -1), (2000, 32, 2048, 2000),
         (2000, 32, 2048, 100), (3000, 64, 3072, -1)]


@pytest.mark.parametrize("L,H,L_max,hint", CASES)
def test_static_entry_matches_context_entry_twice(oracle, L, H, L_max, hint):
    import torch
    from paper_2401_10774_b200 import binding as B
    from tests import gpu_util as U

    assert torch.cuda.is_available(), "this test needs a CUDA device"
    D = 128
    cfg = dict(n_layers=0, d=H * D, n_heads=H, head_dim=D, ffn=8, vocab=8, n_medusa=4)
    ctx = U.make_ctx(cfg, "bf16", L_max, I.TREE_SPECS["sparse64_d4"])
    t = ctx.tree
    T = t["T"]
    a = I.attention_inputs(T, H, D, L, L_max, 90 + L, dtype="bf16")
    dev = {k: U.to_dev(v) for k, v in a.items()}
    cache_len = torch.tensor([L], dtype=torch.int32, device="cuda")
    mask = U.to_dev(t["mask"])
    ref = U.empty_act((T, H, D), B.BF16)
    ref_lse = torch.zeros((T, H), dtype=torch.float32, device="cuda")
    ctx.tree_attention(dev["q"], dev["k_new"], dev["v_new"], dev["k_cache"], dev["v_cache"], cache_len, False, ref, ref_lse)
    torch.cuda.synchronize()
    outs = []
    for call in range(2):
        out = torch.full((T, H, D), float("nan"), dtype=torch.bfloat16, device="cuda")
        lse = torch.full((T, H), float("nan"), dtype=torch.float32, device="cuda")
        B.tree_attention_static(dev["q"], dev["k_new"], dev["v_new"], dev["k_cache"], dev["v_cache"], cache_len, mask,
                                T, H, L_max, hint, out, lse)
        torch.cuda.synchronize()
        outs.append((out, lse))
    # against the oracle too (same bar as the other attention parity tests)
    ot = oracle.build_tree_buffers(oracle.default_tree_paths(**I.TREE_SPECS["sparse64_d4"]))
    o_ref, o_lse = oracle.tree_attention(*(I.as_f32(a[k]) for k in ("q", "k_new", "v_new", "k_cache", "v_cache")), L,
                                         ot["mask"], ot["pos"], apply_rope=False)
    for out, lse in outs:
        err = np.abs(U.to_host_f32(out) - o_ref).max()
        assert err <= TOL_ATTN_BF16, "max |err| %.3g vs the oracle" % err
        assert np.abs(U.to_host_f32(lse) - o_lse).max() <= 5e-2
    for out, lse in outs:
        err = (out.float() - ref.float()).abs().max().item()
        assert err <= TOL_ATTN_BF16, "max |err| %.3g vs the context entry point" % err
        assert (lse - ref_lse).abs().max().item() <= 1e-3
    assert torch.equal(outs[0][0], outs[1][0]), "two calls in a row on the shared scratch must agree bit for bit"
    # limits are enforced with an error, not a fault
    with pytest.raises(B.MedusaError) as e:
        B.tree_attention_static(dev["q"], dev["k_new"], dev["v_new"], dev["k_cache"], dev["v_cache"], cache_len, mask,
                                T, 65, L_max, L, outs[0][0], None)
    assert e.value.code == B.ERR_SHAPE
    with pytest.raises(B.MedusaError) as e:
        B.tree_attention_static(dev["q"], dev["k_new"], dev["v_new"], dev["k_cache"], dev["v_cache"], cache_len, mask,
                                65, H, L_max, L, outs[0][0], None)
    assert e.value.code == B.ERR_SHAPE
    ctx.close()
