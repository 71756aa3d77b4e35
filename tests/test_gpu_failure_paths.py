"""The bounded device-side waits of the tensor-core kernels, made to run out without hanging or faulting anything:
a test hook withholds every load of one CTA's producer (so nothing is in flight), the poll limit is lowered, the
consumers' waits expire, the launch returns, the device status reports the timeout, and after a reset the context
computes correct results again."""
import numpy as np
import pytest

from paper_2401_10774_b200 import inputs as I

pytestmark = pytest.mark.gpu


def _gpu():
    import torch
    from paper_2401_10774_b200 import binding as B
    from tests import gpu_util as U
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    return torch, B, U


def test_gemm_wait_expires_reports_timeout_and_context_recovers(oracle):
    torch, B, U = _gpu()
    cfg = I.model_shape("tiny", d=512, n_heads=4, head_dim=128, ffn=1408, vocab=2048, n_medusa=4, n_layers=2)
    w = I.make_weights(cfg, seed=11, dtype="bf16", head_init="lm_copy")
    ctx = U.make_ctx(cfg, "bf16", 256, I.TREE_SPECS["sparse64_d4"])
    ctx.load_weights(U.dev_weights(w))
    prompt = torch.from_numpy(I.make_prompt(40, cfg["vocab"], 12)).cuda()
    tok = torch.from_numpy(I.rng(5, "treetok").integers(0, cfg["vocab"], size=64).astype(np.int32)).cuda()
    ctx.prefill(prompt)
    ctx.tree_pass(tok)
    assert ctx.device_status() == B.OK
    good = ctx.read_workspace(B.WS_LOGITS, (64, cfg["vocab"]), np.float32)
    # one CTA of the next tensor-core GEMM gets no data; its waits give up after 20000 polls
    ctx.set_option(B.OPT_SPIN_LIMIT, 20000)
    ctx.set_option(B.OPT_WITHHOLD_LOAD, 1)
    ctx.tree_pass(tok)          # returns: nothing waits forever
    assert ctx.device_status() == B.ERR_TIMEOUT
    assert "status" in ctx.last_error()
    # the status is sticky until a reset; after it the same pass is correct again
    ctx.tree_pass(tok)
    assert ctx.device_status() == B.ERR_TIMEOUT
    ctx.set_option(B.OPT_SPIN_LIMIT, 0)
    ctx.reset()
    assert ctx.device_status() == B.OK
    ctx.prefill(prompt)
    ctx.tree_pass(tok)
    assert ctx.device_status() == B.OK
    again = ctx.read_workspace(B.WS_LOGITS, (64, cfg["vocab"]), np.float32)
    assert np.array_equal(again, good)
    ctx.close()


def test_tcgen05_attention_wait_expires_reports_timeout_and_context_recovers(oracle):
    torch, B, U = _gpu()
    H, D, L, L_max = 4, 128, 700, 768
    cfg = dict(n_layers=0, d=H * D, n_heads=H, head_dim=D, ffn=8, vocab=8, n_medusa=5)
    ctx = U.make_ctx(cfg, "bf16", L_max, I.TREE_SPECS["sparse64_d4"])
    ctx.set_option(B.OPT_ATTENTION_KERNEL, 2)
    T = ctx.tree["T"]
    a = I.attention_inputs(T, H, D, L, L_max, 20, dtype="bf16")
    dev = {k: U.to_dev(v) for k, v in a.items()}
    cache_len = torch.tensor([L], dtype=torch.int32, device="cuda")

    def run():
        out = U.empty_act((T, H, D), ctx.dtype)
        ctx.tree_attention(dev["q"], dev["k_new"], dev["v_new"], dev["k_cache"], dev["v_cache"], cache_len, False, out, None)
        torch.cuda.synchronize()
        return U.to_host_f32(out)

    good = run()
    assert ctx.device_status() == B.OK
    ctx.set_option(B.OPT_SPIN_LIMIT, 20000)
    ctx.set_option(B.OPT_WITHHOLD_LOAD, 2)
    run()                        # returns: the starved CTA's waits expire
    assert ctx.device_status() == B.ERR_TIMEOUT
    ctx.set_option(B.OPT_SPIN_LIMIT, 0)
    ctx.reset()
    assert ctx.device_status() == B.OK
    assert np.array_equal(run(), good)
    ot = oracle.build_tree_buffers(oracle.default_tree_paths(**I.TREE_SPECS["sparse64_d4"]))
    ref, _ = oracle.tree_attention(*(I.as_f32(a[k]) for k in ("q", "k_new", "v_new", "k_cache", "v_cache")), L,
                                   ot["mask"], ot["pos"], apply_rope=False)
    assert np.abs(good - ref).max() <= 2e-2
    ctx.close()
