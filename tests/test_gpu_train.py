"""Forward/backward of the Medusa-1 objective of the heads (Sec. 2.2.1, Eq. 1) on the GPU against the float64 oracle.

The GPU multiplies bf16 operands on the tensor cores with float accumulation; where an operand is a computed quantity
(h1, dz, da) it is either a split bf16 pair (about 16 mantissa bits) or, as the streamed operand of a projection, one
bf16 plane (8 bits).  A gradient entry is a sum over the positions of products with one such rounded factor, so its
error is about 2^-9 times the root-sum-square of the products: small against the matrix's largest entries, not against
an entry that happens to cancel.  The tests therefore bound |g - g_ref| by 2e-2 of the matrix's largest |g_ref|, the
relative Frobenius error by 1e-2, and the loss (float sums of float logits) by 2e-3 relative.
"""
import numpy as np
import pytest

from paper_2401_10774_b200 import inputs as I

pytestmark = pytest.mark.gpu

CASES = [
    # name, d, V, K, N (positions: chunks of up to 1024, a shorter batch is padded to a multiple of 256), weight std
    ("small_3heads_300", 512, 2048, 3, 300, 0.05),
    ("small_2heads_77", 256, 1024, 2, 77, 0.05),
    ("small_2heads_2chunks_1324", 512, 2048, 2, 1324, 0.05),
    ("7b_width_1head_300", 4096, 32000, 1, 300, 0.02),
    ("13b_width_2heads_2chunks_1100", 5120, 32000, 2, 1100, 0.02),
]


@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
def test_heads_loss_and_grads_against_the_oracle(oracle, case):
    import torch
    from paper_2401_10774_b200 import binding as B
    from tests import gpu_util as U
    name, d, V, K, N, std = case
    cfg = dict(n_layers=0, d=d, n_heads=max(d // 128, 1), head_dim=128, ffn=8, vocab=V, n_medusa=K, rms_eps=1e-5, rope_theta=1e4)
    w = I.make_weights(cfg, seed=90, dtype="bf16", std=std)
    ctx = B.Context(cfg, B.BF16, 64)
    ctx.load_weights(U.dev_weights(w))
    g = I.rng(91, name)
    h_bits = I.to_bf16_bits(g.standard_normal((N, d)).astype(np.float32))
    labels = g.integers(0, V, size=(K, N)).astype(np.int32)
    for k in range(K):
        labels[k, N - (k + 1):] = -1           # no token that far ahead at the end of the sequence
        labels[k, g.integers(0, N - 8, size=5)] = -1  # and a few unlabelled positions inside
    lam = [0.8 ** (k + 1) for k in range(K)]
    hd = torch.from_numpy(h_bits.view(np.int16)).cuda().view(torch.bfloat16)
    ld = torch.from_numpy(labels).cuda()
    loss = torch.full((K + 1,), -1.0, device="cuda")
    g1 = torch.full((K, d, d), 7.0, device="cuda")   # overwritten, not accumulated into
    g2 = torch.full((K, V, d), 7.0, device="cuda")
    ctx.heads_loss_and_grads(hd, ld, loss, g1, g2)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    ctx.heads_loss_and_grads(hd, ld, loss, g1, g2, lam=lam)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1)
    got_loss, got1, got2 = loss.cpu().numpy().astype(np.float64), g1.cpu().numpy(), g2.cpu().numpy()
    # twice the same bits (no atomics, fixed piece order)
    loss_b, g1_b, g2_b = torch.empty_like(loss), torch.empty_like(g1), torch.empty_like(g2)
    ctx.heads_loss_and_grads(hd, ld, loss_b, g1_b, g2_b, lam=lam)
    assert torch.equal(loss_b, loss) and torch.equal(g1_b, g1) and torch.equal(g2_b, g2)
    ref = oracle.medusa1_loss_and_grads(I.bf16_bits_to_f32(h_bits), I.as_f32(w["medusa_w1"]), I.as_f32(w["medusa_w2"]), labels, lam)
    assert np.all(np.abs(got_loss[:K] - ref["loss_per_head"]) <= 2e-3 * np.abs(ref["loss_per_head"])), (got_loss, ref["loss_per_head"])
    assert abs(got_loss[K] - ref["loss"]) <= 2e-3 * abs(ref["loss"])
    report = []
    for nm, got, want in (("W1", got1, ref["grad_w1"]), ("W2", got2, ref["grad_w2"])):
        for k in range(K):
            err = np.abs(got[k] - want[k])
            mx = float(np.abs(want[k]).max())
            fro = float(np.sqrt((err.astype(np.float64) ** 2).sum()) / np.sqrt((want[k] ** 2).sum()))
            report.append("%s[%d] max|err| %.3g of max|g| %.3g, rel. Frobenius %.3g" % (nm, k, float(err.max()), mx, fro))
            assert float(err.max()) <= 2e-2 * mx, report[-1]
            assert fro <= 1e-2, report[-1]
    flops = K * N * (4.0 * d * d + 6.0 * V * d)
    print("%s: loss %s (oracle %s); %s; %.2f ms per call = %.0f TFLOP/s"
          % (name, got_loss.round(5).tolist(), np.round(ref["loss_per_head"], 5).tolist(), "; ".join(report), ms, flops / ms / 1e9))
    ctx.close()


def test_heads_training_refuses_what_it_cannot_run():
    import torch
    from paper_2401_10774_b200 import binding as B
    from tests import gpu_util as U
    cfg = dict(n_layers=0, d=128, n_heads=1, head_dim=128, ffn=8, vocab=1024, n_medusa=1, rms_eps=1e-5, rope_theta=1e4)
    w = I.make_weights(cfg, seed=92, dtype="bf16")
    ctx = B.Context(cfg, B.BF16, 64)
    ctx.load_weights(U.dev_weights(w))
    h = torch.zeros(8, 128, dtype=torch.bfloat16, device="cuda")
    y = torch.zeros(1, 8, dtype=torch.int32, device="cuda")
    out = torch.zeros(2, device="cuda")
    g1, g2 = torch.zeros(1, 128, 128, device="cuda"), torch.zeros(1, 1024, 128, device="cuda")
    with pytest.raises(B.MedusaError):   # d is not a multiple of 256
        ctx.heads_loss_and_grads(h, y, out, g1, g2)
    ctx.close()
